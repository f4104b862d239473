/*
 * twa.h -- C ABI of the B200 (sm_100a) library for the subspace step of
 * Trainable Weight Averaging (TWA, arXiv 2205.13104).
 *
 * What the library computes (paper's notation, with the coefficients on the
 * basis vectors called alpha here instead of beta):
 *
 *   build      w_bar = (1/n) sum_i w_i                       Section 4.1, Algorithm 1
 *              P = [e_1 .. e_n], orthonormal, span P = span{w_i}
 *                                                            Section 4.1 (Schmidt
 *                                                            orthogonalisation of {w_i})
 *   quantise   P~ = low-bit codes of P plus scale factors    Section 4.6
 *   project    c = P~^T g                                    Section 4.2 (chain rule)
 *   update     alpha <- (1 - eta*lambda) alpha - eta c       Section 4.2, Algorithm 1
 *   lift       w = w_bar + P~ alpha                          Section 4.3, Algorithm 1
 *
 * General rules
 *  - Every pointer is a DEVICE pointer on the context's device unless its
 *    comment says "host".  The caller owns every buffer; the library
 *    allocates a few hundred bytes per context and nothing else.
 *  - Matrices are column-major: column j of a D x n matrix starts at
 *    data + j * col_stride (bytes).  Vectors are contiguous.
 *  - Alignment: data pointers of matrices, g, base, w and workspaces must be
 *    16-byte aligned; col_stride must be a multiple of 16 bytes.
 *  - Limits: 1 <= n <= TWA_MAX_N, 1 <= D <= TWA_MAX_LAUNCH_ROWS = 2^31 - 2^20 (the kernels
 *    count rows in 32-bit integers and round them up to whole tiles).  The per-column
 *    stepping calls (twa_project, twa_project_batch, twa_lift, twa_step, twa_step_adam,
 *    twa_step_host, twa_weighted_average), the row-chunked build (twa_build_begin / feed /
 *    end_pass) and twa_basis_export / twa_basis_import take D <= TWA_MAX_ROWS = 2^34.  Above
 *    TWA_MAX_LAUNCH_ROWS the stepping calls walk the basis in slabs of 2^30 rows, one launch
 *    per slab and kernel: the projection is the float64 sum of the slabs' projections in slab
 *    order (twa_project_batch: every slab after the first adds to C_out), the lift is
 *    independent per row; the calls stay capturable.  Every other call takes a view of at most
 *    TWA_MAX_LAUNCH_ROWS rows of such a basis (a twa_basis whose data points at a row on a
 *    512-byte segment of the columns).
 *  - Calls enqueue work on the context's stream and return without waiting
 *    for it.  Return value 0 = enqueued; a negative TWA_ERR_* = rejected on
 *    the host, nothing enqueued.  Errors found on the device (non-finite
 *    input, rank deficiency, a wait that ran out) are recorded in the
 *    context's status word and read with twa_get_status(), which
 *    synchronises the stream.  After a device-side error the outputs of that
 *    call are unspecified.
 *  - twa_project, twa_lift, twa_step, twa_step_adam, twa_project_batch and the twa_layered_*
 *    stepping calls only enqueue kernels on the context's stream: they may be captured into a
 *    CUDA graph (after one call of the same shape outside the capture, which raises the kernels'
 *    shared-memory limits) and replayed; pointers, sizes and scalar arguments are those of the
 *    captured call (the learning rate, and for the Adam steps the step count behind the bias
 *    corrections, are such scalars: a schedule needs one capture per value).
 *  - One context per stream; calls on one context must not overlap in time
 *    from several host threads.  Different contexts may be driven from different
 *    threads: the only state they share is a per-process cache of kernel attributes
 *    (shared-memory limits already raised), kept under a lock.
 *  - Results are run-to-run bit-identical for fixed arguments on one device
 *    model: every reduction is combined in a fixed order, no floating-point
 *    atomics are used.
 */
#ifndef TWA_H_
#define TWA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TWA_MAX_N 128
#define TWA_MAX_ROWS (1LL << 34) /* the stepping calls, the row-chunked build, export and import */
#define TWA_MAX_LAUNCH_ROWS ((1LL << 31) - (1LL << 20)) /* every other call; one launch of the stepping calls */

enum {
  TWA_OK = 0,
  TWA_ERR_INVALID_ARG = -1,    /* null pointer, size out of range                        */
  TWA_ERR_MISALIGNED = -2,     /* pointer or stride not 16-byte aligned                  */
  TWA_ERR_UNSUPPORTED = -3,    /* bits not in {32, 8, 4}, n > TWA_MAX_N, wrong device    */
  TWA_ERR_RANK_DEFICIENT = -4, /* device: candidate `detail` lies in the span of earlier */
  TWA_ERR_NONFINITE = -5,      /* device: NaN/Inf met in column `detail`                 */
  TWA_ERR_TIMEOUT = -6,        /* device: a bounded wait inside a kernel ran out         */
  TWA_ERR_CUDA = -7,           /* a CUDA runtime/driver call failed (twa_last_error)     */
  TWA_ERR_WORKSPACE = -8       /* workspace missing or smaller than twa_workspace_bytes  */
};

typedef enum { TWA_F32 = 0, TWA_BF16 = 1 } twa_dtype;

typedef struct twa_ctx twa_ctx;

/* Descriptor of a projection matrix P (D x n), held by the caller.
 *  bits == 32: data holds float32 values.
 *  bits == 8 : one two's-complement byte per element, code in [-127,127].
 *  bits == 4 : two elements per byte, row 2k in the low nibble and row 2k+1 in the high
 *              nibble, two's-complement nibbles, code in [-7,7].
 *  The represented value is scales[j] * code (Section 4.6, with one symmetric factor per
 *  column instead of two per layer).  The storage of codes is internal to the library: inside
 *  every aligned 512-byte segment of a column the 16-byte chunks are stored in a
 *  column-dependent order (conflict-free shared-memory reads), so only the library should
 *  produce or read `data` for bits 8 and 4; twa_basis_export / twa_basis_import convert to
 *  and from the canonical two's-complement image.  Bytes of a column beyond ceil(D*bits/8)
 *  up to col_stride are padding. */
typedef struct {
  void* data;         /* device, 16-byte aligned, n * col_stride bytes                 */
  float* scales;      /* device, n floats; ignored when bits == 32                     */
  int64_t D;          /* rows                                                          */
  int64_t col_stride; /* bytes between consecutive columns, multiple of 16             */
  int32_t n;          /* columns                                                       */
  int32_t bits;       /* 32, 8 or 4                                                    */
} twa_basis;

/* ---- context ------------------------------------------------------------------------ */

/* Creates a context bound to CUDA device `device` and to `cuda_stream` (a cudaStream_t
 * passed as void*, NULL = the legacy default stream).  Allocates the device status word.
 * Must not be called while the stream is being captured. */
int twa_create(twa_ctx** out, int device, void* cuda_stream);
void twa_destroy(twa_ctx* ctx);

/* Reads and keeps the first device-side error since the last twa_clear_status.  Waits for
 * the stream.  *code is TWA_OK or a TWA_ERR_*, *detail the offending column or -1. */
int twa_get_status(twa_ctx* ctx, int* code, int* detail);
int twa_clear_status(twa_ctx* ctx);
const char* twa_strerror(int code);
/* Host string describing the last failed CUDA call of this context ("" if none). */
const char* twa_last_error(const twa_ctx* ctx);

/* Tuning knobs for measurements; value 0 restores the built-in choice.
 *  TWA_TUNE_PROJECT_WARPS / TWA_TUNE_LIFT_WARPS: consumer warps per block (8..20; lift: even, >= 16)
 *  TWA_TUNE_STAGES: depth of the shared-memory ring (2..16)
 *  TWA_TUNE_WAIT_LIMIT_MS: bound of every in-kernel wait (default 2000 ms).  The limit is
 *      wall-clock time (%globaltimer), not time the kernel was running: where the GPU is
 *      time-sliced with other contexts, or a tool serialises kernels, a block that was off the
 *      GPU for longer reports TWA_ERR_TIMEOUT with nothing wrong -- raise the limit there.
 *  TWA_TUNE_DEQUANT_PATH: how 8/4-bit codes meet g and alpha: 0 = exact integer dot products
 *      on the tensor pipe against block-fixed-point digits of g / alpha (default),
 *      1 = code -> float32 conversion and float32 FMA.  The warp and stage knobs act on the
 *      float path and on 32-bit bases only.
 *  TWA_TUNE_TILE_SEGMENTS: tensor-pipe path, 512-byte segments of a column per tile: 1, 2 or 4
 *      (4 is honoured for n <= 32 only).  Default: per kernel and width, the tallest tile of which
 *      enough stages fit in shared memory.  Also the projection on a 32-bit basis (default 4 for
 *      n <= 32, 2 for n <= 64, else 1; 4 needs an even D and becomes 2 otherwise).
 *  TWA_TUNE_BUILD_PANEL: twa_build_basis: 0 = panels of 8 columns, the Gram-Schmidt coefficients
 *      inside a panel taken from the panel's Gram matrix (default); 1 = column by column;
 *      2 = panels of 8 columns with column-by-column sweeps inside a panel.
 *  TWA_TUNE_LIFT_VECTORS: lift on 8/4-bit codes, how the rows of `base` and of `w_out` travel:
 *      1 = every lane loads and stores its own rows; 2 = `base` comes through the shared-memory
 *      ring beside the codes; 3 = as 2, and the results leave through bulk stores from shared
 *      memory; 0 = built-in choice by the share of the two vectors in the bytes moved
 *      (n * bits <= 192: 2, <= 320: 3, else 1).
 *  TWA_TUNE_SLAB_ROWS: rows per launch of the per-column stepping calls (twa_project, twa_lift,
 *      twa_step, twa_step_adam, twa_weighted_average, twa_project_batch): a multiple of 65536, at most 2^30.  A basis
 *      of more rows is walked in slabs of that many rows (at most 16 of them, else the call
 *      returns TWA_ERR_INVALID_ARG), exactly as bases above TWA_MAX_LAUNCH_ROWS always are: shorter
 *      kernels where the GPU is shared and a long launch holds others up.  0 = one launch up to
 *      TWA_MAX_LAUNCH_ROWS, slabs of 2^30 rows above. */
enum { TWA_TUNE_PROJECT_WARPS = 1, TWA_TUNE_LIFT_WARPS = 2, TWA_TUNE_STAGES = 3,
       TWA_TUNE_WAIT_LIMIT_MS = 4, TWA_TUNE_DEQUANT_PATH = 5, TWA_TUNE_TILE_SEGMENTS = 6,
       TWA_TUNE_BUILD_PANEL = 7, TWA_TUNE_LIFT_VECTORS = 8, TWA_TUNE_SLAB_ROWS = 9 };
int twa_set_tuning(twa_ctx* ctx, int key, int value);

/* Exercises the bounded wait every streaming kernel uses, without any fault: enqueues one block
 * that waits (TWA_TUNE_WAIT_LIMIT_MS) for a barrier phase nothing completes.  The kernel then
 * returns normally and twa_get_status reports TWA_ERR_TIMEOUT; the context stays usable. */
int twa_selftest_wait(twa_ctx* ctx);

/* Per-kernel timing of twa_step for measurements.  twa_profile_enable(ctx, max_steps > 0)
 * creates CUDA events; from then on each twa_step records three of them (before the
 * projection kernel, between the two kernels, after the lift kernel) until max_steps steps
 * were recorded.  twa_profile_read waits for the stream, returns the summed durations in
 * milliseconds and the number of steps they cover, and starts a new series.
 * twa_profile_enable(ctx, 0) destroys the events. */
int twa_profile_enable(twa_ctx* ctx, int max_steps);
int twa_profile_read(twa_ctx* ctx, double* project_ms, double* lift_ms, int* steps);

/* ---- sizes -------------------------------------------------------------------------- */

/* Bytes between columns the library uses for a D-row basis of the given width:
 * ceil(D*bits/8) rounded up to 512 for bits 8 and 4, to 128 for bits 32. */
int64_t twa_basis_col_stride(int64_t D, int bits);
/* n * twa_basis_col_stride: size of the `data` buffer the caller must provide. */
size_t twa_basis_bytes(int64_t D, int n, int bits);
/* Size of the scratch buffer `ws` every call below takes (device, 16-byte aligned).  Its
 * contents need no initialisation and carry nothing between calls. */
size_t twa_workspace_bytes(int64_t D, int n, int bits);

/* ---- subspace construction (Section 4.1; Algorithm 1) ------------------------------- */

/* w_bar and the orthonormal basis of the n candidates.
 *  W        in/out: D x n float32 candidates, column i = w_i, column stride ldw ELEMENTS
 *           (ldw >= D, ldw % 4 == 0).  Overwritten by the basis: on return column j holds
 *           e_j, the j-th vector of the Gram-Schmidt orthonormalisation of the candidates in
 *           the given order (the factor Q of A = QR with positive diagonal).  Schedule: block
 *           classical Gram-Schmidt with one re-orthogonalisation -- panels of 8 columns are
 *           first made orthogonal to all earlier vectors, then orthonormalised among
 *           themselves from the panel's float64 Gram matrix (its Cholesky factor holds the
 *           Gram-Schmidt coefficients), and both steps are done a second time.  TWA_TUNE_BUILD_PANEL = 1 selects the literal
 *           column-after-column schedule (two projection passes per column); both give the
 *           same factor up to rounding.
 *  wbar_out out: D floats, the mean of the candidates (written before W is overwritten).
 *  P32_out  out (host struct): filled with {W, NULL, D, 4*ldw, n, 32}.
 * Device-side errors: TWA_ERR_NONFINITE, TWA_ERR_RANK_DEFICIENT (a column whose remainder
 * is below 1e-5 of its length; that column is set to zero). */
int twa_build_basis(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, float* wbar_out,
                    twa_basis* P32_out, void* ws, size_t ws_bytes);

/* twa_build_basis followed by twa_quantize_basis for each of `widths` storage widths (Sections
 * 4.1 and 4.6 in one call), with one pass over the float32 basis less: the largest magnitude
 * of every column is taken while the build writes the column for the last time, so each width
 * costs one encoding pass only.  Basis, scales and codes are those of the separate calls, bit
 * for bit.
 *  bits  host array of `widths` entries (1 <= widths <= 8), each 8 or 4.
 *  Pq    host array of `widths` descriptors; the caller sets data (twa_basis_bytes(D, n,
 *        bits[k]) bytes) and scales (n floats) of each, the call fills the rest.
 * Other arguments and device-side errors as for twa_build_basis and twa_quantize_basis. */
int twa_build_quantized(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw, float* wbar_out,
                        twa_basis* P32_out, const int* bits, int widths, twa_basis* Pq, void* ws,
                        size_t ws_bytes);

/* The same basis for candidate sets too large to be resident (e.g. 1.3 G rows x 32 columns =
 * 168 GB of float32): the caller feeds row chunks of the candidates, once per pass, and never
 * holds more than one chunk.  The orthonormal basis with span{e_1..e_j} = span{w_1..w_j} and
 * positive diagonal is unique, so it is computed in Gram form with every n x n quantity in
 * float64: G1 = A^T A, R1 = chol(G1); G2 = (A R1^-1)^T (A R1^-1), R2 = chol(G2);
 * Q = A (R1^-1 R2^-1) -- orthogonalise, then re-orthogonalise.  n <= 64.
 *
 *   twa_build_begin(ctx, D, n, wbar_out, bws, bws_bytes)
 *   pass 0: twa_build_feed(ctx, 0, chunk, ...) for every chunk   -> mean rows into wbar_out, G1
 *           twa_build_end_pass(ctx, 0, 0, NULL)
 *   pass 1: feed every chunk again                                -> G2
 *           twa_build_end_pass(ctx, 1, 0, NULL)
 *   pass 2: feed again (q32_out optional)                         -> column absmax of Q
 *           twa_build_end_pass(ctx, 2, bits, Pq)                  -> scales; fills *Pq
 *   pass 3: feed again with Pq                                    -> codes of Q (bits 8 / 4)
 *           twa_build_end_pass(ctx, 3, 0, NULL)
 *
 *  chunk   rows x n float32, column-major with column stride ldc elements: rows
 *          [row0, row0+rows) of the candidates.  row0 must be a multiple of 1024, rows a
 *          multiple of 1024 except for the chunk that ends at D.  Any order, each row range
 *          exactly once per pass, the same partition in every pass.
 *  q32_out passes 2 and 3, optional: rows x n float32 destination for the float32 basis rows
 *          of this chunk, column-major with column stride ldq >= rows elements (to assemble
 *          the whole basis pass base + row0 and the full column stride).  With bits == 32
 *          this is the only output and pass 3 is not run.
 *  Pq      the caller sets data (twa_basis_bytes) and scales before twa_build_end_pass(2).
 *          Several widths from one build: call twa_build_end_pass(ctx, 2, bits, Pq) once per
 *          width (each takes its scales from the same column absmax) and feed every chunk of
 *          pass 3 once per Pq; the rule "each row range once per pass" then holds per Pq.
 *  bws     device scratch of twa_build_workspace_bytes(n) bytes, alive until the last call.
 * Device-side errors: TWA_ERR_RANK_DEFICIENT (same 1e-5 rule as twa_build_basis),
 * TWA_ERR_NONFINITE.  Codes are exactly the quantiser applied to the float32 rows of pass 2. */
size_t twa_build_workspace_bytes(int n);
int twa_build_begin(twa_ctx* ctx, int64_t D, int n, float* wbar_out, void* bws, size_t bws_bytes);
int twa_build_feed(twa_ctx* ctx, int pass, const float* chunk, int64_t ldc, int64_t row0,
                   int64_t rows, const twa_basis* Pq, float* q32_out, int64_t ldq);
int twa_build_end_pass(twa_ctx* ctx, int pass, int bits, twa_basis* Pq);
/* Pass 3 for one or two widths at once: twa_build_feed(ctx, 3, ...) with a host array of `widths`
 * (1 or 2) quantised bases, e.g. the 8-bit and the 4-bit one of the same build.  The chunk's rows
 * of Q are formed once and encoded for every basis of the array; the codes are those of one
 * twa_build_feed per basis, bit for bit.  A chunk fed through this call counts as fed for each
 * of the bases. */
int twa_build_feed_codes(twa_ctx* ctx, const float* chunk, int64_t ldc, int64_t row0, int64_t rows,
                         const twa_basis* Pq, int widths, float* q32_out, int64_t ldq);

/* Mean only: wbar_out[r] = (1/n) sum_i W[r, i]. */
int twa_mean(twa_ctx* ctx, const float* W, int64_t D, int n, int64_t ldw, float* wbar_out);

/* ---- low-bit storage (Section 4.6, per-column symmetric variant) -------------------- */

/* Quantises a float32 basis.  For every column: s_j = absmax_j / qmax (IEEE float32
 * division), qmax = 127 (bits 8) or 7 (bits 4); code = clamp(rint(P[r,j] / s_j), -qmax,
 * qmax) with round-half-to-even; an all-zero column gets s_j = 0 and codes 0.
 *  P32  in: descriptor with bits == 32.
 *  Pq   in/out (host struct): the caller sets Pq->data (twa_basis_bytes(D, n, bits) bytes)
 *       and Pq->scales (n floats); the call fills D, col_stride, n, bits and the buffers.
 * Device-side error: TWA_ERR_NONFINITE. */
int twa_quantize_basis(twa_ctx* ctx, const twa_basis* P32, int bits, twa_basis* Pq, void* ws,
                       size_t ws_bytes);

/* Canonical image of a quantised basis, for parity checks and checkpoints:
 *  codes_out  device, n * ceil(D*bits/8) bytes, column after column without padding;
 *             bits 8: two's-complement int8; bits 4: row 2k low nibble, row 2k+1 high
 *             nibble, two's-complement nibbles, last high nibble 0 when D is odd.
 *  scales_out device, n floats. */
int twa_basis_export(twa_ctx* ctx, const twa_basis* Pq, void* codes_out, float* scales_out);
/* Inverse of twa_basis_export; Pq->data / Pq->scales set by the caller as for quantise. */
int twa_basis_import(twa_ctx* ctx, const void* codes, const float* scales, int64_t D, int n,
                     int bits, twa_basis* Pq);

/* ---- subspace step (Sections 4.2-4.3; loop body of Algorithm 1) --------------------- */

/* c_out[j] = s_j * sum_r code[r,j] * g[r]  (bits 32: sum_r P[r,j] g[r]).
 *  g      in: D elements of g_dtype (bfloat16 is widened exactly inside the kernel).
 *  c_out  out: n floats.
 * Products and partial sums are float32, the final combine over blocks is float64 in block
 * order. */
int twa_project(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype,
                float* c_out, void* ws, size_t ws_bytes);

/* The projection for `batch` gradients at once (Section 4.2's chain-rule equation for every row of
 * G): C_out[b*n + j] = s_j * sum_r code[r,j] * G[b*ldg + r].  P~ is read once per group of
 * twa_project_batch_group(ctx, P, g_dtype) gradients (8 when three stages of that shape fit in shared
 * memory, else 4; 1 for a float32 basis, which is projected gradient by gradient),
 * two gradients sharing every integer MMA.
 *  G      in: batch rows of ldg elements of g_dtype, ldg >= D; G and ldg*sizeof(element) 16-byte
 *         aligned.   C_out  out: batch x n floats.
 * Device-side errors: TWA_ERR_NONFINITE (detail = index of the gradient), TWA_ERR_TIMEOUT. */
int twa_project_batch(twa_ctx* ctx, const twa_basis* P, const void* G, int64_t ldg, int batch,
                      twa_dtype g_dtype, float* C_out, void* ws, size_t ws_bytes);
int twa_project_batch_group(twa_ctx* ctx, const twa_basis* P, twa_dtype g_dtype);

/* w_out[r] = base[r] + sum_j (s_j * alpha[j]) * code[r,j].
 *  alpha  in: n floats.   base  in: D floats, or NULL for 0.
 *  w_out  out: D floats; may be the same buffer as base, must not overlap P. */
int twa_lift(twa_ctx* ctx, const twa_basis* P, const float* alpha, const float* base,
             float* w_out, void* ws, size_t ws_bytes);

/* One training iteration of the subspace: c = P~^T g; alpha <- (1 - lr*lambda) alpha - lr c;
 * w = wbar + P~ alpha.  alpha (n floats) is updated in place; w (D floats) is overwritten and
 * may be the same buffer as wbar only if the caller wants wbar replaced.  c_out (n floats)
 * receives c and may be NULL.  alpha is state that outlives the call: when any coefficient of c is
 * not finite (TWA_ERR_NONFINITE) or a wait ran out in the projection (TWA_ERR_TIMEOUT) alpha is left
 * as it was (w is then lifted from the old alpha), so the step can be repeated after
 * twa_clear_status. */
int twa_step(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, float lr,
             float lambda, float* alpha, const float* wbar, float* w, float* c_out, void* ws,
             size_t ws_bytes);

/* The same iteration with Adam on the coefficients and decoupled weight decay (the base optimiser
 * of the paper's transformer runs, Section 5; Adam as published by Kingma & Ba):
 *   m <- beta1 m + (1-beta1) c;  v <- beta2 v + (1-beta2) c^2;
 *   alpha <- (1 - lr*weight_decay) alpha - lr (m / (1-beta1^step)) / (sqrt(v / (1-beta2^step)) + eps)
 * `opt` is read on the HOST at call time; `step` is the 1-based count of this update.  m, v: n floats
 * on the device, zero before the first step, updated in place.  A learning-rate schedule is the
 * caller's: pass the step's rate in opt->lr (twa_cosine_lr gives the cosine schedule). */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay;
  int32_t step;
} twa_adam;
int twa_step_adam(twa_ctx* ctx, const twa_basis* P, const void* g, twa_dtype g_dtype, const twa_adam* opt,
                  float* alpha, float* m, float* v, const float* wbar, float* w, float* c_out, void* ws,
                  size_t ws_bytes);
/* Host function: min_lr + (base_lr - min_lr) (1 + cos(pi step/total_steps)) / 2, step clamped to
 * [0, total_steps]. */
float twa_cosine_lr(float base_lr, int step, int total_steps, float min_lr);

/* Fixed-weight average of the candidates, w_out = sum_i weights[i] * w_i (Section 2's comparison
 * methods: SWA = equal weights, LAWA = equal weights on the last t, EMA = geometric weights), one
 * streaming pass over W.  W, ldw as for twa_build_basis (not modified); weights: n floats, device. */
int twa_weighted_average(twa_ctx* ctx, const float* W, int64_t D, int n, int64_t ldw, const float* weights,
                         float* w_out, void* ws, size_t ws_bytes);

/* The same iteration for a caller whose gradient and weights live in HOST memory (pinned
 * memory makes the copies asynchronous): g_host (D elements) goes to the device staging
 * buffer g_stage, the step runs into the device buffer w, and w goes back to w_host (D floats).
 * From 2^22 rows on the work is cut into up to 16 row chunks so that the three parts overlap:
 * the projection of a chunk starts when its rows of g have arrived, and every chunk of w leaves
 * for the host while the next one is lifted; the copies run on a second stream the context
 * creates at the first such call, ordered with the context's stream by events (work enqueued on
 * the context's stream after the call starts after the last copy).  The coefficients' gradient
 * is then the float64 sum of the chunks' projections in chunk order: equal to twa_step's within
 * the rounding of the float32 partial sums, not bit for bit.  Smaller problems run the three
 * operations back to back on the context's stream and give twa_step's result exactly. */
int twa_step_host(twa_ctx* ctx, const twa_basis* P, const void* g_host /* host */,
                  twa_dtype g_dtype, float lr, float lambda, float* alpha, const float* wbar,
                  float* w, float* w_host /* host */, void* g_stage, void* ws, size_t ws_bytes);

/* ---- the paper's default construction: layer-wise, affine B-bit codes -------------------- */

/* Layers are given as L+1 row offsets of the flat parameter vector on the HOST,
 * 0 = o_0 < o_1 < ... < o_L = D; layer l owns rows o_l .. o_{l+1}-1 (Section 4.5).
 *
 * A layered basis stores P~^l = a^l * code + b^l with unsigned B-bit codes and one (a^l, b^l)
 * pair per layer (Section 4.6: a^l = (max P^l - min P^l) / (2^B - 1), b^l = min P^l, code =
 * round((P - b^l) / a^l); here with float32 subtraction and division and round-half-to-even).
 * B is 1, 2, 3, 4, 8 or 16, the widths of the paper's ablation on quantisation bits (Section 5.5).
 * A code occupies a slot of 1, 2, 4 or 8 bits of a column byte (3-bit codes sit in 4-bit slots;
 * with S slots per byte, row S k + s of a column is in bits [s * slot, (s+1) * slot) of byte k);
 * 16-bit codes are stored as two 8-bit planes, the high bytes in columns 0..n-1 and the low bytes
 * in columns n..2n-1 of `codes` (so n <= 64 there).  Device memory per candidate and row: the slot
 * width, i.e. B bits except for B = 3 (4 bits).  The columns use the same column-major
 * chunk-permuted bytes as twa_basis, except that every layer starts on a 64-byte granule of the
 * column; `granules` maps each granule back to {layer, valid rows, first flat row, 0}.  All
 * pointers are device pointers into the one buffer `mem` the caller passed to twa_quantize_affine.
 * A layered basis holds at most TWA_MAX_LAUNCH_ROWS padded rows.  The layers' coefficients do not interact
 * (Section 4.5: one projection, one update and one lift per layer), so a model of more rows is
 * several layered bases over consecutive groups of layers, each stepped with its own rows of g,
 * wbar and w. */
typedef struct {
  twa_basis codes;            /* D = padded rows, bits = slot width 8, 4, 2 or 1, scales == NULL */
  float* a;                   /* L scaling factors                                              */
  float* b;                   /* L zero factors                                                 */
  int32_t* granules;          /* 4 ints per 64-byte granule of a column                         */
  int64_t* flat_offsets;      /* L+1 row offsets of the layers in the flat parameter vector     */
  int64_t* internal_offsets;  /* L+1 row offsets of the layers in the padded storage            */
  int64_t D;                  /* flat rows                                                      */
  int32_t L;                  /* layers                                                         */
  /* Work split of the step kernels, fixed when the basis is quantised (it depends on the GPU's
   * multiprocessor count and on the tile height in force then): block k owns tiles
   * k*tiles_per_cta .. of `tiles`, meets layers cta_first_layer[k] .. and keeps one row of
   * partial sums per layer it meets, rows cta_run_base[k] .. cta_run_base[k+1]-1. */
  int32_t cta_count, kt, tiles, tiles_per_cta, total_runs;
  int32_t* cta_first_layer;   /* cta_count ints                                                 */
  int32_t* cta_run_base;      /* cta_count + 1 ints                                             */
  int32_t code_bits;          /* B of the quantiser: 1, 2, 3, 4, 8 or 16 (codes.bits is the slot) */
  int32_t planes;             /* 1, or 2 for B = 16: codes.n = 2 n, columns 0..n-1 the high     */
                              /* bytes of the codes, columns n..2n-1 the low bytes              */
} twa_layered_basis;

/* Scratch for the two construction calls below (device, 16-byte aligned). */
size_t twa_layered_workspace_bytes(const int64_t* offsets_host, int L, int n);
/* Padded row count and size of `mem` for a layered basis. */
int64_t twa_layered_rows(const int64_t* offsets_host, int L, int bits);
size_t twa_layered_basis_bytes(const int64_t* offsets_host, int L, int n, int bits);

/* w_bar and, in place of the candidates, e_i^l = (w_i^l - w_bar^l) / ||w_i^l - w_bar^l||_2 for every
 * layer l and candidate i (Section 4.1 construction equation applied per layer, Section 4.5;
 * Algorithm 1).  A layer in which a candidate equals the mean gives a zero vector.  W, ldw,
 * wbar_out, P32_out as for twa_build_basis.  Synchronises the stream once (uploads the layer
 * tables from pageable host memory).  Device-side error: TWA_ERR_NONFINITE. */
int twa_build_centered(twa_ctx* ctx, float* W, int64_t D, int n, int64_t ldw,
                       const int64_t* offsets_host, int L, float* wbar_out, twa_basis* P32_out,
                       void* lws, size_t lws_bytes);

/* Per-layer min-max quantisation of a float32 basis (Section 4.6), bits = B in {1, 2, 3, 4, 8, 16}
 * (P32->n <= 64 for B = 16).
 *  mem  device buffer of twa_layered_basis_bytes, 256-byte aligned; *out points into it.
 * Device-side error: TWA_ERR_NONFINITE (detail = layer). */
int twa_quantize_affine(twa_ctx* ctx, const twa_basis* P32, const int64_t* offsets_host, int L,
                        int bits, void* mem, size_t mem_bytes, twa_layered_basis* out, void* lws,
                        size_t lws_bytes);

/* Row-chunked form of twa_build_centered + twa_quantize_affine (same Sections 4.1, 4.5, 4.6) for
 * candidate sets that do not fit in device memory: the caller feeds every row chunk of the
 * candidates once per pass, in any order inside a pass, and never holds more than one chunk.
 *   begin           carves `mem` (twa_layered_basis_bytes, 256-byte aligned), fills *out, clears the
 *                   accumulators in lws (twa_layered_workspace_bytes) and the codes; synchronises
 *                   the stream once (uploads the layer tables)
 *   pass 0: feed    w_bar rows of the chunk into wbar[row0 ..], sums of (w - w_bar)^2 per layer and
 *                   candidate;            end_pass(0): the norms
 *   pass 1: feed    min / max of e = (w - w_bar) / ||.|| per layer; q32_out (optional, rows x n,
 *                   column stride ldq) receives e as float32;   end_pass(1): the factors a, b
 *   pass 2: feed    codes of e (computed with the arithmetic of pass 1, so they are exactly the
 *                   quantiser applied to the float32 values of pass 1);   end_pass(2): nothing
 * chunk: rows x n float32, candidate i at chunk[i * ld + (r - row0)] for flat row r; 16-byte aligned,
 * ld and row0 multiples of 4.  offsets_host, lws: as passed to begin.  wbar: D floats, the same
 * buffer in every call.  The same chunking need not be used in every pass.  Errors as for the
 * resident calls (TWA_ERR_NONFINITE: detail = candidate in pass 0, layer in pass 1). */
int twa_layered_build_begin(twa_ctx* ctx, int64_t D, int n, const int64_t* offsets_host, int L, int bits,
                            void* mem, size_t mem_bytes, twa_layered_basis* out, void* lws, size_t lws_bytes);
int twa_layered_build_feed(twa_ctx* ctx, const twa_layered_basis* lb, const int64_t* offsets_host, int pass,
                           const float* chunk, int64_t ld, int64_t row0, int64_t rows, float* wbar,
                           float* q32_out, int64_t ldq, void* lws, size_t lws_bytes);
int twa_layered_build_end_pass(twa_ctx* ctx, const twa_layered_basis* lb, const int64_t* offsets_host,
                               int pass, void* lws, size_t lws_bytes);

/* Canonical image for parity checks and checkpoints: unsigned codes in flat row order, n rows of
 * ceil(D*slot/8) bytes (slot = 1, 2, 4, 8 as above: row S k + s in bits [s*slot, (s+1)*slot) of byte
 * k; B = 3 uses 4-bit slots, so its image has D/2 bytes per candidate; B = 16: 2 D bytes per
 * candidate, low byte first), and the L factors a, b.  Device pointers. */
int twa_layered_export(twa_ctx* ctx, const twa_layered_basis* lb, void* codes_out, float* a_out,
                       float* b_out);

/* Layer-wise subspace step (Algorithm 1 with the loop over layers of Section 4.5; quantised
 * basis of Section 4.6).  beta, c_out: L x n floats, layer-major (row l = coefficients of layer
 * l's n basis vectors).  g, wbar, base, w: D elements in flat row order.  sws: device scratch of
 * twa_layered_step_workspace_bytes, 256-byte aligned; it carries nothing between calls.
 *
 *   project: c^l_i   = sum_r (a^l code[r,i] + b^l) g[r]   over the rows r of layer l
 *   lift:    w_out[r] = base[r] + sum_i (a^l code[r,i] + b^l) beta^l_i   (base may be NULL)
 *   step:    c = project(g); beta <- (1 - lr*lambda) beta - lr c; w = lift(beta, wbar)
 *
 * Integer dot products are exact; float32 partial sums per warp and layer are combined in
 * float64 in a fixed order.  Device-side errors: TWA_ERR_NONFINITE (detail = layer),
 * TWA_ERR_TIMEOUT. */
size_t twa_layered_step_workspace_bytes(const twa_layered_basis* lb);
int twa_layered_project(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype,
                        float* c_out, void* sws, size_t sws_bytes);
int twa_layered_lift(twa_ctx* ctx, const twa_layered_basis* lb, const float* beta, const float* base,
                     float* w_out, void* sws, size_t sws_bytes);
int twa_layered_step(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype,
                     float lr, float lambda, float* beta, const float* wbar, float* w, float* c_out,
                     void* sws, size_t sws_bytes);

/* The layer-wise step with Adam on every layer's coefficients (m, v: L x n floats, as twa_step_adam). */
int twa_layered_step_adam(twa_ctx* ctx, const twa_layered_basis* lb, const void* g, twa_dtype g_dtype,
                          const twa_adam* opt, float* beta, float* m, float* v, const float* wbar, float* w,
                          float* c_out, void* sws, size_t sws_bytes);

/* ---- projection without any allocation ----------------------------------------------- */

/* (No counterpart in the paper: this entry point exists for the way some programs manage
 * GPU memory, not for the method.)
 *
 * c_out[j] = s_j * sum_r code[r,j] * g[r], exactly as twa_project, for callers that cannot
 * allocate device memory at the point of the call: a program whose caching allocator owns
 * the whole device, a loop that may not make calls which can synchronise the device, a
 * plug-in that is handed its input and output buffers and nothing else.  It takes no
 * context (twa_create allocates) and no workspace: the per-block partial sums, the
 * completion counter and the status word live in one fixed array of
 * twa_noalloc_scratch_bytes() = 131,328 bytes inside the library's device image, which every
 * GPU that loads the library holds until the process exits.  The call itself makes no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *
 *  device, cuda_stream  where to run (cudaStream_t as void*, NULL = legacy default stream).
 *  P, g, g_dtype, c_out as for twa_project; the caller still owns inputs and outputs.
 *  status_out           device, 2 ints, or NULL: receives {TWA_OK or the device-side error,
 *                       detail} when the kernel has run.
 * Limits: n <= TWA_MAX_N (128) columns and at most 256 blocks of partial sums; a larger n is
 * rejected with TWA_ERR_UNSUPPORTED.  twa_noalloc_last_error() gives the reason of the calling
 * thread's last rejected call; it is meaningful only right after a negative return value (a
 * call that is accepted clears it).
 * The first call on a device looks up the device address of the array and the driver entry
 * point it needs; make that first call before any stream capture begins.
 * All calls on one device share the array: the call clears the counter and the status on the
 * stream before the kernel, and calls that overlap on the GPU (different streams, or
 * different host threads without ordering) race on it -- serialise them. */
int twa_project_noalloc(int device, void* cuda_stream, const twa_basis* P, const void* g,
                        twa_dtype g_dtype, float* c_out, int* status_out);
const char* twa_noalloc_last_error(void);
size_t twa_noalloc_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* TWA_H_ */
