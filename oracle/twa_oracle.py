"""Float64 CPU oracle for the Trainable Weight Averaging (TWA) subspace path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
method computes.  It shares no code with the CUDA library, is never imported by
it, and must only be used by the tests, by the smoke check and by the CPU
baseline timing of the benchmark.  Nothing here is tuned.

Conventions
-----------
* A matrix of n vectors in R^D is a 2-D numpy array of shape (D, n): column j is
  vector j, as in the paper's P = [e_1, ..., e_n] (Section 4.2).  Any strides
  are accepted; passing ``arr.T`` of an (n, D) C-ordered array makes every
  column contiguous.
* Inputs carry the bytes the GPU sees (float32 candidates, float32 or widened
  bfloat16 gradients, int8 code values, float32 scales); all arithmetic widens
  them to float64 first.
* The paper writes beta for the coefficients on the basis vectors; the code
  calls them ``alpha`` like the library's interface does.

Every function is pinned by tests/test_oracle_*.py against closed forms,
library factorizations, brute force and the invariants the method fixes; no
function here is "parity unpinned".
"""

from __future__ import annotations

import numpy as np

QMAX = {8: 127, 4: 7}


# --------------------------------------------------------------------------- #
# Subspace construction
# --------------------------------------------------------------------------- #
def mean(W):
    """Centre point of the candidates, w_bar = (1/n) sum_i w_i.

    Section 4.1, the subspace-construction equation; Algorithm 1; Section 4.3
    uses it as the initial point w^(0).
    Summation runs over i in index order in float64.
    """
    W = np.asarray(W)
    D, n = W.shape
    acc = np.zeros(D, dtype=np.float64)
    for i in range(n):
        acc += W[:, i].astype(np.float64)
    return acc / float(n)


def cgs2(A, rel_tol=1e-10):
    """Schmidt orthogonalisation of the raw candidates, one vector after the
    other (Section 4.1, the paragraph on orthogonalising {w_i}), in the
    classical Gram-Schmidt form with one re-orthogonalisation ("CGS2").

    For j = 0..n-1:  v <- a_j;  exactly twice:  c_k = <q_k, v> for every k < j
    computed from the SAME v (classical, not modified), then
    v <- v - sum_k c_k q_k;  r_jj = ||v||_2;  q_j = v / r_jj.

    Returns (Q, R, deficient): Q is (D, n) float64 with orthonormal columns,
    R is the (n, n) upper-triangular factor with positive diagonal (A = Q R),
    deficient is None, or the index of the first column whose remainder
    satisfies r_jj <= rel_tol * ||a_j||_2 (columns from there on are left 0).
    """
    A = np.asarray(A)
    D, n = A.shape
    Q = np.zeros((D, n), dtype=np.float64, order="F")
    R = np.zeros((n, n), dtype=np.float64)
    for j in range(n):
        a = A[:, j].astype(np.float64)
        a_norm = float(np.sqrt(np.dot(a, a)))
        v = a.copy()
        for _pass in range(2):
            if j > 0:
                c = Q[:, :j].T @ v          # all coefficients from the same v
                v = v - Q[:, :j] @ c
                R[:j, j] += c
        r_jj = float(np.sqrt(np.dot(v, v)))
        if not (r_jj > rel_tol * a_norm):
            return Q, R, j
        R[j, j] = r_jj
        Q[:, j] = v / r_jj
    return Q, R, None


# --------------------------------------------------------------------------- #
# Low-bit storage of the projection matrix: per-column absmax, symmetric
# --------------------------------------------------------------------------- #
def absmax_scales(P32, bits):
    """Per-column scale s_j = fl32(max_r |P[r, j]| / qmax), qmax = 2^(bits-1)-1.

    This is the symmetric, per-column variant of the uniform quantiser of
    Section 4.6 (one factor per column instead of the paper's two per layer).
    Returns (scales float32 (n,), absmax float32 (n,)).
    """
    qmax = QMAX[bits]
    P32 = np.asarray(P32)
    assert P32.dtype == np.float32
    n = P32.shape[1]
    m = np.zeros(n, dtype=np.float32)
    for j in range(n):
        col = P32[:, j]
        m[j] = np.max(np.abs(col)) if col.size else np.float32(0)
    s = (m.astype(np.float64) / float(qmax)).astype(np.float32)
    return s, m


def encode(P32, scales, bits):
    """Codes for given scales: code = clamp(round_half_even(fl32(p / s_j)),
    -qmax, +qmax); a column with s_j == 0 is all zeros.

    The quotient is formed in float64 from the float32 operands and rounded
    once to float32, which equals the IEEE float32 division; rounding to the
    integer is ties-to-even (Section 4.6 leaves the rounding mode open).
    Returns an int8 array of shape (D, n) holding the code VALUES (also for
    bits == 4; packing is a separate step).
    """
    qmax = QMAX[bits]
    P32 = np.asarray(P32)
    assert P32.dtype == np.float32
    D, n = P32.shape
    codes = np.zeros((D, n), dtype=np.int8, order="F")
    for j in range(n):
        s = np.float32(scales[j])
        if s == 0:
            continue
        t = (P32[:, j].astype(np.float64) / np.float64(s)).astype(np.float32)
        q = np.rint(t)                      # numpy rint: ties to even
        q = np.clip(q, -qmax, qmax)
        codes[:, j] = q.astype(np.int8)
    return codes


def quantize(P32, bits):
    """Whole quantiser: scales from the column absmax, then codes."""
    s, _ = absmax_scales(P32, bits)
    return encode(P32, s, bits), s


def pack_codes(codes, bits):
    """Canonical byte image of the codes, one row of bytes per column.

    bits == 8: byte r of column j is code[r, j] (two's complement).
    bits == 4: byte k of column j holds row 2k in its low nibble and row 2k+1
    in its high nibble, both as two's-complement nibbles; an odd D leaves the
    last high nibble 0.  Returns uint8 of shape (n, ceil(D*bits/8)).
    """
    codes = np.asarray(codes)
    D, n = codes.shape
    if bits == 8:
        return np.ascontiguousarray(codes.T).view(np.uint8).copy()
    assert bits == 4
    nb = (D + 1) // 2
    out = np.zeros((n, nb), dtype=np.uint8)
    for j in range(n):
        col = codes[:, j].astype(np.int16)
        nib = (col & 0xF).astype(np.uint8)
        lo = nib[0::2]
        hi = nib[1::2]
        out[j, : lo.size] = lo
        out[j, : hi.size] |= (hi << 4).astype(np.uint8)
    return out


def unpack_codes(packed, D, bits):
    """Inverse of pack_codes: (n, bytes) uint8 -> int8 code values (D, n)."""
    packed = np.asarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    if bits == 8:
        return np.asfortranarray(packed.view(np.int8)[:, :D].T)
    assert bits == 4
    codes = np.zeros((D, n), dtype=np.int8, order="F")
    for j in range(n):
        b = packed[j]
        lo = (b & 0xF).astype(np.int8)
        hi = (b >> 4).astype(np.int8)
        lo = (lo ^ 8) - 8                    # two's-complement nibble -> its value in [-8, 7]
        hi = (hi ^ 8) - 8
        inter = np.empty(2 * b.size, dtype=np.int8)
        inter[0::2] = lo
        inter[1::2] = hi
        codes[:, j] = inter[:D]
    return codes


def storage_bytes(D, n, bits):
    """Bytes of the stored projection matrix in this per-column format:
    n columns of ceil(D*bits/8) code bytes plus one float32 scale per column
    (bits == 32: plain float32, 4nD).  Mirrors the accounting of the table
    "memory_projection" (Section 4.6): 4nD against nBD/8 plus the factors."""
    if bits == 32:
        return 4 * n * D
    return n * ((D * bits + 7) // 8) + 4 * n


def paper_storage_bytes(D, n, bits, L=1, k=1):
    """The table "memory_projection" of Section 4.6 as printed: 4*ceil(n/k)*D
    bytes at 32 bits, ceil(n/k)*B*D/8 + 8L bytes at B bits."""
    cols = -(-n // k)
    if bits == 32:
        return 4 * cols * D
    return cols * bits * D / 8 + 8 * L


# --------------------------------------------------------------------------- #
# Subspace step
# --------------------------------------------------------------------------- #
def project(codes, scales, g):
    """Coefficient gradient c = P~^T g with P~[r, j] = s_j * code[r, j]
    (Section 4.2, the chain-rule equation; Algorithm 1, the update of the
    variables).  c_j = s_j * sum_r code[r, j] * g[r], all in float64."""
    codes = np.asarray(codes)
    g64 = np.asarray(g).astype(np.float64)
    n = codes.shape[1]
    c = np.zeros(n, dtype=np.float64)
    for j in range(n):
        c[j] = np.float64(scales[j]) * np.dot(codes[:, j].astype(np.float64), g64)
    return c


def project_batch(codes, scales, G):
    """Coefficient gradients of several gradient vectors at once: column b of the
    result is P~^T g_b (Section 4.2, the chain-rule equation, applied to each
    column of G).  G has shape (D, B); returns (n, B) in float64."""
    codes = np.asarray(codes)
    G64 = np.asarray(G).astype(np.float64)
    n, B = codes.shape[1], G64.shape[1]
    C = np.zeros((n, B), dtype=np.float64)
    for b in range(B):
        for j in range(n):
            C[j, b] = np.float64(scales[j]) * np.dot(codes[:, j].astype(np.float64), G64[:, b])
    return C


def project_f32(P32, g):
    """c = P^T g for an unquantised float32 basis, in float64."""
    P32 = np.asarray(P32)
    g64 = np.asarray(g).astype(np.float64)
    n = P32.shape[1]
    c = np.zeros(n, dtype=np.float64)
    for j in range(n):
        c[j] = np.dot(P32[:, j].astype(np.float64), g64)
    return c


def sgd_update(alpha, c, lr, lam=0.0):
    """alpha <- (1 - lr*lam) * alpha - lr * c  (the gradient-descent update rule
    of Section 4.2; Algorithm 1 writes it with the factor (1 - eta*lambda))."""
    alpha = np.asarray(alpha, dtype=np.float64)
    c = np.asarray(c, dtype=np.float64)
    return (1.0 - float(lr) * float(lam)) * alpha - float(lr) * c


def adam_update(alpha, m, v, c, lr, t, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0):
    """One Adam step on the coefficients with decoupled weight decay (the base
    optimiser the paper uses on the coefficients of transformer models, Section 5
    training details; Adam as published by Kingma & Ba, the decay applied to the
    variable itself as in AdamW).  t is the 1-based step count.
        alpha <- (1 - lr*wd) alpha
        m <- beta1 m + (1-beta1) c ;  v <- beta2 v + (1-beta2) c^2
        alpha <- alpha - lr * (m / (1-beta1^t)) / (sqrt(v / (1-beta2^t)) + eps)
    Returns (alpha, m, v) in float64."""
    alpha = np.asarray(alpha, dtype=np.float64)
    m = np.asarray(m, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    c = np.asarray(c, dtype=np.float64)
    alpha = alpha * (1.0 - float(lr) * float(weight_decay))
    m = float(beta1) * m + (1.0 - float(beta1)) * c
    v = float(beta2) * v + (1.0 - float(beta2)) * c * c
    m_hat = m / (1.0 - float(beta1) ** int(t))
    v_hat = v / (1.0 - float(beta2) ** int(t))
    alpha = alpha - float(lr) * m_hat / (np.sqrt(v_hat) + float(eps))
    return alpha, m, v


def cosine_lr(base_lr, step, total_steps, min_lr=0.0):
    """Cosine learning-rate schedule (the schedule of the paper's TWA runs on
    transformers): base at step 0, min_lr at step total_steps."""
    x = min(max(float(step) / float(total_steps), 0.0), 1.0)
    return float(min_lr) + 0.5 * (float(base_lr) - float(min_lr)) * (1.0 + np.cos(np.pi * x))


def weighted_average(W, weights):
    """Fixed-weight average w = sum_i weights_i w_i of the candidates (SWA: equal
    weights; LAWA: equal weights on the last t; EMA: geometric weights -- the
    comparison methods of Section 2), in float64."""
    W = np.asarray(W)
    out = np.zeros(W.shape[0], dtype=np.float64)
    for i in range(W.shape[1]):
        out += np.float64(weights[i]) * W[:, i].astype(np.float64)
    return out


def lift(codes, scales, alpha, base=None):
    """w = base + P~ alpha (Section 4.3: w_twa = w_bar + P beta; Algorithm 1,
    the update of the weights).  base None means 0.
    w[r] = base[r] + sum_j (s_j * alpha_j) * code[r, j], in float64."""
    codes = np.asarray(codes)
    D, n = codes.shape
    w = np.zeros(D, dtype=np.float64) if base is None else np.asarray(base).astype(np.float64).copy()
    for j in range(n):
        a = np.float64(scales[j]) * np.float64(alpha[j])
        w += a * codes[:, j].astype(np.float64)
    return w


def lift_f32(P32, alpha, base=None):
    """w = base + P alpha for an unquantised float32 basis, in float64."""
    P32 = np.asarray(P32)
    D, n = P32.shape
    w = np.zeros(D, dtype=np.float64) if base is None else np.asarray(base).astype(np.float64).copy()
    for j in range(n):
        w += np.float64(alpha[j]) * P32[:, j].astype(np.float64)
    return w


def step(codes, scales, g, alpha, wbar, lr, lam=0.0):
    """One iteration of the loop body of Algorithm 1: project the gradient,
    update the coefficients, rebuild the weights from w_bar.
    Returns (alpha_new, w_new, c)."""
    c = project(codes, scales, g)
    alpha_new = sgd_update(alpha, c, lr, lam)
    w_new = lift(codes, scales, alpha_new, wbar)
    return alpha_new, w_new, c


def step_f32(P32, g, alpha, wbar, lr, lam=0.0):
    """Same iteration with an unquantised float32 basis."""
    c = project_f32(P32, g)
    alpha_new = sgd_update(alpha, c, lr, lam)
    w_new = lift_f32(P32, alpha_new, wbar)
    return alpha_new, w_new, c


# --------------------------------------------------------------------------- #
# The paper's default construction: decentralise + normalise, layer by layer,
# per-layer min-max (affine) B-bit codes, one coefficient per (layer, model).
# `layers` is the list of row offsets [0 = o_0 < o_1 < ... < o_L = D]: layer l
# owns rows o_l .. o_{l+1}-1 of the flat parameter vector (Section 4.5).
# --------------------------------------------------------------------------- #
def center_normalize(W, layers):
    """e_i^l = (w_i^l - w_bar^l) / ||w_i^l - w_bar^l||_2 for every layer l
    (Section 4.1, the subspace-construction equation, applied per layer as in
    Section 4.5; Algorithm 1).  A layer in which a candidate equals the mean
    gives a zero vector (the paper does not say; such a direction cannot move
    the weights).  Returns (P float64 (D, n), w_bar float64 (D,))."""
    W = np.asarray(W)
    D, n = W.shape
    wbar = mean(W)
    P = np.zeros((D, n), dtype=np.float64, order="F")
    for l in range(len(layers) - 1):
        a, b = layers[l], layers[l + 1]
        for i in range(n):
            v = W[a:b, i].astype(np.float64) - wbar[a:b]
            nv = float(np.sqrt(np.dot(v, v)))
            if nv > 0.0:
                P[a:b, i] = v / nv
    return P, wbar


def affine_factors(P32, layers, bits):
    """Per-layer factors of the uniform min-max quantiser (Section 4.6):
    b^l = min(P^l), a^l = fl32(fl32(max(P^l) - min(P^l)) / (2^B - 1)), over all
    n columns of the layer.  Returns (a float32 (L,), b float32 (L,))."""
    P32 = np.asarray(P32)
    assert P32.dtype == np.float32
    L = len(layers) - 1
    a = np.zeros(L, dtype=np.float32)
    b = np.zeros(L, dtype=np.float32)
    levels = float(2 ** bits - 1)
    for l in range(L):
        blk = P32[layers[l]:layers[l + 1], :]
        lo, hi = np.float32(blk.min()), np.float32(blk.max())
        span = np.float32(hi - lo)                               # float32 subtraction
        a[l] = np.float32(np.float64(span) / levels)             # = IEEE float32 division
        b[l] = lo
    return a, b


def affine_encode(P32, layers, a, b, bits):
    """code = clamp(round_half_even(fl32(fl32(p - b^l) / a^l)), 0, 2^B - 1); a
    layer with a^l == 0 (constant layer) is all zeros.  Section 4.6, with the
    subtraction and the division both rounded to float32 and ties to even (the
    paper leaves precision and rounding mode open).  Returns the code VALUES of
    shape (D, n), uint8 (uint16 for B = 16)."""
    P32 = np.asarray(P32)
    assert P32.dtype == np.float32
    D, n = P32.shape
    top = 2 ** bits - 1
    dt = np.uint16 if bits > 8 else np.uint8
    codes = np.zeros((D, n), dtype=dt, order="F")
    for l in range(len(layers) - 1):
        if a[l] == 0:
            continue
        r0, r1 = layers[l], layers[l + 1]
        d = (P32[r0:r1, :] - np.float32(b[l])).astype(np.float32)          # float32 subtraction
        t = (d.astype(np.float64) / np.float64(a[l])).astype(np.float32)    # float32 division
        codes[r0:r1, :] = np.clip(np.rint(t), 0, top).astype(dt)
    return codes


SLOT_BITS = {1: 1, 2: 2, 3: 4, 4: 4, 8: 8, 16: 16}


def pack_unsigned(codes, bits):
    """Canonical byte image of unsigned B-bit codes (Section 4.6 stores the quantised matrix
    as B-bit integers), one row of bytes per column.  A code occupies a slot of 1, 2, 4, 8 or
    16 bits (3-bit codes sit in 4-bit slots): with S slots per byte, byte k of column j holds
    rows S*k .. S*k+S-1, row S*k+s in bits [s*slot, (s+1)*slot); 16-bit codes take two bytes,
    low byte first.  Unused bits are 0.  Returns uint8 of shape (n, ceil(D*slot/8))."""
    codes = np.asarray(codes)
    D, n = codes.shape
    slot = SLOT_BITS[bits]
    if slot == 16:
        out = np.zeros((n, 2 * D), dtype=np.uint8)
        for j in range(n):
            col = codes[:, j].astype(np.uint32)
            out[j, 0::2] = (col & 0xFF).astype(np.uint8)
            out[j, 1::2] = (col >> 8).astype(np.uint8)
        return out
    per = 8 // slot
    nb = (D + per - 1) // per
    out = np.zeros((n, nb), dtype=np.uint8)
    for j in range(n):
        col = codes[:, j].astype(np.uint16)
        for s_ in range(per):
            part = col[s_::per]
            out[j, : part.size] |= (part << (s_ * slot)).astype(np.uint8)
    return out


def unpack_unsigned(packed, D, bits):
    """Inverse of pack_unsigned: (n, bytes) uint8 -> code values (D, n), uint16."""
    packed = np.asarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    slot = SLOT_BITS[bits]
    codes = np.zeros((D, n), dtype=np.uint16, order="F")
    if slot == 16:
        for j in range(n):
            b = packed[j].astype(np.uint16)
            codes[:, j] = (b[0::2] | (b[1::2] << 8))[:D]
        return codes
    per = 8 // slot
    mask = (1 << slot) - 1
    for j in range(n):
        b = packed[j].astype(np.uint16)
        inter = np.empty(per * b.size, dtype=np.uint16)
        for s_ in range(per):
            inter[s_::per] = (b >> (s_ * slot)) & mask
        codes[:, j] = inter[:D]
    return codes


def affine_quantize(P32, layers, bits):
    a, b = affine_factors(P32, layers, bits)
    return affine_encode(P32, layers, a, b, bits), a, b


def affine_dequantize(codes, layers, a, b):
    """P~^l = a^l * code + b^l in float64 (Section 4.6)."""
    codes = np.asarray(codes)
    out = np.zeros(codes.shape, dtype=np.float64, order="F")
    for l in range(len(layers) - 1):
        r0, r1 = layers[l], layers[l + 1]
        out[r0:r1, :] = np.float64(a[l]) * codes[r0:r1, :].astype(np.float64) + np.float64(b[l])
    return out


def project_layerwise(codes, layers, a, b, g):
    """c[l, i] = sum_{r in layer l} P~[r, i] g[r] with P~ = a^l code + b^l
    (Algorithm 1, the update of the variables of layer l).  Returns (L, n)."""
    codes = np.asarray(codes)
    g64 = np.asarray(g).astype(np.float64)
    L, n = len(layers) - 1, codes.shape[1]
    c = np.zeros((L, n), dtype=np.float64)
    for l in range(L):
        r0, r1 = layers[l], layers[l + 1]
        gl = g64[r0:r1]
        sg = float(np.sum(gl))
        for i in range(n):
            c[l, i] = np.float64(a[l]) * np.dot(codes[r0:r1, i].astype(np.float64), gl) + np.float64(b[l]) * sg
    return c


def lift_layerwise(codes, layers, a, b, beta, base=None):
    """w^l = base^l + P~^l beta^l (Algorithm 1, the update of the weights of layer
    l); beta has shape (L, n)."""
    codes = np.asarray(codes)
    D, n = codes.shape
    w = np.zeros(D, dtype=np.float64) if base is None else np.asarray(base).astype(np.float64).copy()
    for l in range(len(layers) - 1):
        r0, r1 = layers[l], layers[l + 1]
        for i in range(n):
            w[r0:r1] += np.float64(beta[l, i]) * (np.float64(a[l]) * codes[r0:r1, i].astype(np.float64)
                                                  + np.float64(b[l]))
    return w


def step_layerwise(codes, layers, a, b, g, beta, wbar, lr, lam=0.0):
    """One iteration of the loop body of Algorithm 1 with its inner loop over the
    layers.  Returns (beta_new (L, n), w_new, c (L, n))."""
    c = project_layerwise(codes, layers, a, b, g)
    beta_new = sgd_update(beta, c, lr, lam)
    w_new = lift_layerwise(codes, layers, a, b, beta_new, wbar)
    return beta_new, w_new, c


def paper_affine_storage_bytes(D, n, bits, L):
    """Table "memory_projection" (Section 4.6): n*B*D/8 code bytes plus two
    4-byte factors per layer."""
    return n * bits * D / 8 + 8 * L
