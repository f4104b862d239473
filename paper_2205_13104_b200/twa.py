"""ctypes binding of libtwa.so: one Python function per C entry point of include/twa.h,
with the same name.  The functions only marshal arguments (torch tensors -> device
pointers); every step of the computation runs in the CUDA library.  There is no CPU
fallback: if the library has not been built, loading it raises.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libtwa.so")
CSRC = os.path.join(_HERE, "csrc")
SOURCES = ["twa_api.cu", "twa_basis.cu", "twa_chunked.cu", "twa_layered_build.cu", "twa_layered_step.cu", "twa_project_batch.cu", "twa_panel.cu", "twa_stream.cu",
           "twa_stream_mma.cu", "twa_noalloc.cu"]

TWA_MAX_N = 128
TWA_OK = 0
TWA_ERR_INVALID_ARG = -1
TWA_ERR_MISALIGNED = -2
TWA_ERR_UNSUPPORTED = -3
TWA_ERR_RANK_DEFICIENT = -4
TWA_ERR_NONFINITE = -5
TWA_ERR_TIMEOUT = -6
TWA_ERR_CUDA = -7
TWA_ERR_WORKSPACE = -8
TWA_F32 = 0
TWA_BF16 = 1
TWA_TUNE_PROJECT_WARPS = 1
TWA_TUNE_LIFT_WARPS = 2
TWA_TUNE_STAGES = 3
TWA_TUNE_WAIT_LIMIT_MS = 4
TWA_TUNE_DEQUANT_PATH = 5
TWA_TUNE_TILE_SEGMENTS = 6
TWA_TUNE_BUILD_PANEL = 7
TWA_TUNE_LIFT_VECTORS = 8
TWA_TUNE_SLAB_ROWS = 9

EXPORTS = [
    "twa_create", "twa_destroy", "twa_get_status", "twa_clear_status", "twa_strerror",
    "twa_last_error", "twa_set_tuning", "twa_selftest_wait", "twa_profile_enable", "twa_profile_read",
    "twa_basis_col_stride", "twa_basis_bytes",
    "twa_workspace_bytes", "twa_build_basis", "twa_build_quantized", "twa_build_workspace_bytes", "twa_build_begin",
    "twa_build_feed", "twa_build_feed_codes", "twa_build_end_pass", "twa_mean", "twa_quantize_basis",
    "twa_basis_export", "twa_basis_import", "twa_project", "twa_lift", "twa_step",
    "twa_step_host", "twa_step_adam", "twa_cosine_lr", "twa_weighted_average", "twa_layered_step_adam", "twa_project_batch", "twa_project_batch_group", "twa_layered_workspace_bytes", "twa_layered_rows", "twa_layered_basis_bytes",
    "twa_build_centered", "twa_quantize_affine", "twa_layered_export",
    "twa_layered_build_begin", "twa_layered_build_feed", "twa_layered_build_end_pass",
    "twa_layered_step_workspace_bytes", "twa_layered_project", "twa_layered_lift", "twa_layered_step",
    "twa_project_noalloc", "twa_noalloc_last_error", "twa_noalloc_scratch_bytes",
]


class twa_basis(ctypes.Structure):
    """Mirror of the C struct twa_basis."""
    _fields_ = [("data", ctypes.c_void_p), ("scales", ctypes.c_void_p),
                ("D", ctypes.c_int64), ("col_stride", ctypes.c_int64),
                ("n", ctypes.c_int32), ("bits", ctypes.c_int32)]


class twa_adam(ctypes.Structure):
    """Mirror of the C struct twa_adam."""
    _fields_ = [("lr", ctypes.c_float), ("beta1", ctypes.c_float), ("beta2", ctypes.c_float),
                ("eps", ctypes.c_float), ("weight_decay", ctypes.c_float), ("step", ctypes.c_int32)]


class twa_layered_basis(ctypes.Structure):
    """Mirror of the C struct twa_layered_basis."""
    _fields_ = [("codes", twa_basis), ("a", ctypes.c_void_p), ("b", ctypes.c_void_p),
                ("granules", ctypes.c_void_p), ("flat_offsets", ctypes.c_void_p),
                ("internal_offsets", ctypes.c_void_p), ("D", ctypes.c_int64), ("L", ctypes.c_int32),
                ("cta_count", ctypes.c_int32), ("kt", ctypes.c_int32), ("tiles", ctypes.c_int32),
                ("tiles_per_cta", ctypes.c_int32), ("total_runs", ctypes.c_int32),
                ("cta_first_layer", ctypes.c_void_p), ("cta_run_base", ctypes.c_void_p),
                ("code_bits", ctypes.c_int32), ("planes", ctypes.c_int32)]


class TwaError(RuntimeError):
    def __init__(self, code, where, extra=""):
        self.code = code
        msg = f"{where}: {twa_strerror(code)} ({code})"
        if extra:
            msg += f" -- {extra}"
        super().__init__(msg)


def _nvcc():
    return os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")


NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", os.path.join(_ROOT, "include")]


def build_command(out=LIB_PATH):
    """The one-line form of the build (every source in one nvcc call)."""
    return [_nvcc()] + NVCC_FLAGS + ["-shared", "-o", out] + [os.path.join(CSRC, s) for s in SOURCES]


def build_library(force=False, verbose=False):
    """Compiles the CUDA library for sm_100a next to this file (nvcc cross-compiles without
    a GPU): one object per source, compiled side by side, then one link.  Skipped when the
    library is newer than every source; an object is reused while it is newer than every
    source and header."""
    from concurrent.futures import ThreadPoolExecutor
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(_ROOT, "include", "twa.h")]
    newest = max(os.path.getmtime(d) for d in deps)
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= newest:
        return LIB_PATH
    obj_dir = os.path.join(_HERE, "_build")
    os.makedirs(obj_dir, exist_ok=True)
    headers = [d for d in deps if not d.endswith(".cu")]
    newest_header = max(os.path.getmtime(h) for h in headers)

    def compile_one(src):
        obj = os.path.join(obj_dir, os.path.splitext(src)[0] + ".o")
        path = os.path.join(CSRC, src)
        if not force and os.path.exists(obj) and \
                os.path.getmtime(obj) >= max(os.path.getmtime(path), newest_header):
            return obj
        cmd = [_nvcc()] + NVCC_FLAGS + ["-c", path, "-o", obj]
        if verbose:
            print(" ".join(cmd), flush=True)
        subprocess.run(cmd, check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, SOURCES))
    link = [_nvcc(), "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB_PATH] + objs
    if verbose:
        print(" ".join(link), flush=True)
    subprocess.run(link, check=True)
    return LIB_PATH


_lib = None


def load():
    """Loads libtwa.so (once) and declares the argument types of every entry point."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -c 'import __graft_entry__ as g; g.build()'`; there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
    szt = ctypes.c_size_t
    bp = ctypes.POINTER(twa_basis)
    sig = {
        "twa_create": (i32, [ctypes.POINTER(vp), i32, vp]),
        "twa_destroy": (None, [vp]),
        "twa_get_status": (i32, [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]),
        "twa_clear_status": (i32, [vp]),
        "twa_strerror": (ctypes.c_char_p, [i32]),
        "twa_last_error": (ctypes.c_char_p, [vp]),
        "twa_set_tuning": (i32, [vp, i32, i32]),
        "twa_selftest_wait": (i32, [vp]),
        "twa_profile_enable": (i32, [vp, i32]),
        "twa_profile_read": (i32, [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                   ctypes.POINTER(i32)]),
        "twa_basis_col_stride": (i64, [i64, i32]),
        "twa_basis_bytes": (szt, [i64, i32, i32]),
        "twa_workspace_bytes": (szt, [i64, i32, i32]),
        "twa_build_basis": (i32, [vp, vp, i64, i32, i64, vp, bp, vp, szt]),
        "twa_build_quantized": (i32, [vp, vp, i64, i32, i64, vp, bp, ctypes.POINTER(i32), i32, bp, vp, szt]),
        "twa_build_workspace_bytes": (szt, [i32]),
        "twa_build_begin": (i32, [vp, i64, i32, vp, vp, szt]),
        "twa_build_feed": (i32, [vp, i32, vp, i64, i64, i64, bp, vp, i64]),
        "twa_build_end_pass": (i32, [vp, i32, i32, bp]),
        "twa_build_feed_codes": (i32, [vp, vp, i64, i64, i64, bp, i32, vp, i64]),
        "twa_mean": (i32, [vp, vp, i64, i32, i64, vp]),
        "twa_quantize_basis": (i32, [vp, bp, i32, bp, vp, szt]),
        "twa_basis_export": (i32, [vp, bp, vp, vp]),
        "twa_basis_import": (i32, [vp, vp, vp, i64, i32, i32, bp]),
        "twa_project": (i32, [vp, bp, vp, i32, vp, vp, szt]),
        "twa_lift": (i32, [vp, bp, vp, vp, vp, vp, szt]),
        "twa_step": (i32, [vp, bp, vp, i32, f32, f32, vp, vp, vp, vp, vp, szt]),
        "twa_step_host": (i32, [vp, bp, vp, i32, f32, f32, vp, vp, vp, vp, vp, vp, szt]),
        "twa_step_adam": (i32, [vp, bp, vp, i32, ctypes.POINTER(twa_adam), vp, vp, vp, vp, vp, vp, vp, szt]),
        "twa_cosine_lr": (f32, [f32, i32, i32, f32]),
        "twa_weighted_average": (i32, [vp, vp, i64, i32, i64, vp, vp, vp, szt]),
        "twa_layered_step_adam": (i32, [vp, ctypes.POINTER(twa_layered_basis), vp, i32, ctypes.POINTER(twa_adam), vp, vp,
                                        vp, vp, vp, vp, vp, szt]),
        "twa_project_batch": (i32, [vp, bp, vp, i64, i32, i32, vp, vp, szt]),
        "twa_project_batch_group": (i32, [vp, bp, i32]),
        "twa_layered_workspace_bytes": (szt, [ctypes.POINTER(ctypes.c_int64), i32, i32]),
        "twa_layered_rows": (i64, [ctypes.POINTER(ctypes.c_int64), i32, i32]),
        "twa_layered_basis_bytes": (szt, [ctypes.POINTER(ctypes.c_int64), i32, i32, i32]),
        "twa_build_centered": (i32, [vp, vp, i64, i32, i64, ctypes.POINTER(ctypes.c_int64), i32, vp, bp, vp, szt]),
        "twa_quantize_affine": (i32, [vp, bp, ctypes.POINTER(ctypes.c_int64), i32, i32, vp, szt,
                                      ctypes.POINTER(twa_layered_basis), vp, szt]),
        "twa_layered_export": (i32, [vp, ctypes.POINTER(twa_layered_basis), vp, vp, vp]),
        "twa_layered_build_begin": (i32, [vp, i64, i32, ctypes.POINTER(ctypes.c_int64), i32, i32, vp, szt,
                                          ctypes.POINTER(twa_layered_basis), vp, szt]),
        "twa_layered_build_feed": (i32, [vp, ctypes.POINTER(twa_layered_basis), ctypes.POINTER(ctypes.c_int64), i32,
                                         vp, i64, i64, i64, vp, vp, i64, vp, szt]),
        "twa_layered_build_end_pass": (i32, [vp, ctypes.POINTER(twa_layered_basis), ctypes.POINTER(ctypes.c_int64),
                                             i32, vp, szt]),
        "twa_layered_step_workspace_bytes": (szt, [ctypes.POINTER(twa_layered_basis)]),
        "twa_layered_project": (i32, [vp, ctypes.POINTER(twa_layered_basis), vp, i32, vp, vp, szt]),
        "twa_layered_lift": (i32, [vp, ctypes.POINTER(twa_layered_basis), vp, vp, vp, vp, szt]),
        "twa_layered_step": (i32, [vp, ctypes.POINTER(twa_layered_basis), vp, i32, f32, f32, vp, vp, vp, vp,
                                   vp, szt]),
        "twa_project_noalloc": (i32, [i32, vp, bp, vp, i32, vp, vp]),
        "twa_noalloc_last_error": (ctypes.c_char_p, []),
        "twa_noalloc_scratch_bytes": (szt, []),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


# --------------------------------------------------------------------------------------
# helpers
# --------------------------------------------------------------------------------------
def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _dtype_code(t):
    if t.dtype == torch.float32:
        return TWA_F32
    if t.dtype == torch.bfloat16:
        return TWA_BF16
    raise TypeError(f"gradient dtype {t.dtype} not supported (float32 or bfloat16)")


def _check(rc, where, ctx=None):
    if rc != TWA_OK:
        extra = ""
        if rc == TWA_ERR_CUDA and ctx is not None:
            extra = twa_last_error(ctx)
        raise TwaError(rc, where, extra)


class Basis:
    """A twa_basis descriptor together with the tensors that own its memory."""

    def __init__(self, desc, data, scales):
        self.desc = desc
        self.data = data          # keeps the device buffers alive
        self.scales = scales

    D = property(lambda self: self.desc.D)
    n = property(lambda self: self.desc.n)
    bits = property(lambda self: self.desc.bits)
    col_stride = property(lambda self: self.desc.col_stride)


# --------------------------------------------------------------------------------------
# entry points (same names as in include/twa.h)
# --------------------------------------------------------------------------------------
def twa_strerror(code):
    return load().twa_strerror(int(code)).decode()


def twa_last_error(ctx):
    return load().twa_last_error(ctx).decode()


def twa_create(device=0, stream=None):
    """Context on `device` bound to `stream` (a torch.cuda.Stream; None = the current one)."""
    lib = load()
    if stream is None:
        stream = torch.cuda.current_stream(device)
    handle = ctypes.c_void_p()
    rc = lib.twa_create(ctypes.byref(handle), int(device), ctypes.c_void_p(stream.cuda_stream))
    _check(rc, "twa_create")
    return handle


def twa_destroy(ctx):
    load().twa_destroy(ctx)


def twa_get_status(ctx):
    code, detail = ctypes.c_int(0), ctypes.c_int(-1)
    _check(load().twa_get_status(ctx, ctypes.byref(code), ctypes.byref(detail)), "twa_get_status", ctx)
    return code.value, detail.value


def twa_clear_status(ctx):
    _check(load().twa_clear_status(ctx), "twa_clear_status", ctx)


def twa_set_tuning(ctx, key, value):
    _check(load().twa_set_tuning(ctx, int(key), int(value)), "twa_set_tuning", ctx)


def twa_selftest_wait(ctx):
    _check(load().twa_selftest_wait(ctx), "twa_selftest_wait", ctx)


def twa_profile_enable(ctx, max_steps):
    _check(load().twa_profile_enable(ctx, int(max_steps)), "twa_profile_enable", ctx)


def twa_profile_read(ctx):
    """(project_ms, lift_ms, steps) summed over the steps recorded since the last read."""
    p, l, k = ctypes.c_double(0), ctypes.c_double(0), ctypes.c_int(0)
    _check(load().twa_profile_read(ctx, ctypes.byref(p), ctypes.byref(l), ctypes.byref(k)),
           "twa_profile_read", ctx)
    return p.value, l.value, k.value


def twa_basis_col_stride(D, bits):
    return int(load().twa_basis_col_stride(int(D), int(bits)))


def twa_basis_bytes(D, n, bits):
    return int(load().twa_basis_bytes(int(D), int(n), int(bits)))


def twa_workspace_bytes(D, n, bits):
    return int(load().twa_workspace_bytes(int(D), int(n), int(bits)))


def new_workspace(device, D=1, n=1, bits=8):
    return torch.empty(twa_workspace_bytes(D, n, bits), dtype=torch.uint8, device=device)


def twa_mean(ctx, W, D, wbar_out):
    n, ldw = W.shape
    _check(load().twa_mean(ctx, _ptr(W), int(D), int(n), int(ldw), _ptr(wbar_out)), "twa_mean", ctx)
    return wbar_out


def twa_build_basis(ctx, W, D, wbar_out, ws):
    """W: float32 CUDA tensor (n, ldw), row i = candidate w_i; overwritten by the basis."""
    assert W.dtype == torch.float32 and W.is_contiguous()
    n, ldw = W.shape
    desc = twa_basis()
    rc = load().twa_build_basis(ctx, _ptr(W), int(D), int(n), int(ldw), _ptr(wbar_out),
                                ctypes.byref(desc), _ptr(ws), ws.numel())
    _check(rc, "twa_build_basis", ctx)
    return Basis(desc, W, None)


def twa_build_quantized(ctx, W, D, wbar_out, bits_list, ws, out=None):
    """twa_build_basis and one quantised basis per entry of bits_list in one call; returns
    (P32, [Pq, ...]).  out: a list of Basis from new_quantised_basis to fill (None: allocated here)."""
    assert W.dtype == torch.float32 and W.is_contiguous()
    n, ldw = W.shape
    k = len(bits_list)
    if out is None:
        out = [new_quantised_basis(int(D), int(n), int(b), W.device) for b in bits_list]
    desc32 = twa_basis()
    descs = (twa_basis * k)()
    bits = (ctypes.c_int * k)(*[int(b) for b in bits_list])
    for i in range(k):
        descs[i].data, descs[i].scales = out[i].desc.data, out[i].desc.scales
    rc = load().twa_build_quantized(ctx, _ptr(W), int(D), int(n), int(ldw), _ptr(wbar_out),
                                    ctypes.byref(desc32), bits, k, descs, _ptr(ws), ws.numel())
    _check(rc, "twa_build_quantized", ctx)
    for i in range(k):
        ctypes.memmove(ctypes.byref(out[i].desc), ctypes.byref(descs[i]), ctypes.sizeof(twa_basis))
    return Basis(desc32, W, None), out


def twa_build_workspace_bytes(n):
    return int(load().twa_build_workspace_bytes(int(n)))


def twa_build_begin(ctx, D, n, wbar_out, bws):
    _check(load().twa_build_begin(ctx, int(D), int(n), _ptr(wbar_out), _ptr(bws), bws.numel()),
           "twa_build_begin", ctx)


def twa_build_feed(ctx, pass_index, chunk, row0, rows, Pq=None, q32_out=None):
    """chunk: float32 CUDA tensor view (n, >= rows) whose row i holds rows [row0, row0+rows) of
    candidate i (stride(0) = column stride); q32_out: None or a float32 view (n, >= rows) laid out
    the same way that receives the float32 basis rows of this chunk."""
    assert chunk.dtype == torch.float32 and chunk.stride(1) == 1
    rc = load().twa_build_feed(ctx, int(pass_index), _ptr(chunk), int(chunk.stride(0)), int(row0),
                               int(rows), ctypes.byref(Pq.desc) if Pq is not None else None,
                               _ptr(q32_out), int(q32_out.stride(0)) if q32_out is not None else 0)
    _check(rc, "twa_build_feed", ctx)


def twa_build_feed_codes(ctx, chunk, row0, rows, Pqs, q32_out=None):
    """Pass 3 of the row-chunked build for one or two quantised bases at once (Pqs: list of Basis)."""
    assert chunk.dtype == torch.float32 and chunk.stride(1) == 1
    arr = (twa_basis * len(Pqs))()
    for i, q in enumerate(Pqs):
        ctypes.memmove(ctypes.byref(arr[i]), ctypes.byref(q.desc), ctypes.sizeof(twa_basis))
    rc = load().twa_build_feed_codes(ctx, _ptr(chunk), int(chunk.stride(0)), int(row0), int(rows), arr, len(Pqs),
                                     _ptr(q32_out), int(q32_out.stride(0)) if q32_out is not None else 0)
    _check(rc, "twa_build_feed_codes", ctx)


def twa_build_end_pass(ctx, pass_index, bits=0, Pq=None):
    rc = load().twa_build_end_pass(ctx, int(pass_index), int(bits),
                                   ctypes.byref(Pq.desc) if Pq is not None else None)
    _check(rc, "twa_build_end_pass", ctx)


def basis_view(P, row0=0, rows=None, col0=0, cols=None):
    """Descriptor of a block of rows and columns of a basis, sharing its memory.  For 8/4-bit
    storage the block must respect the internal chunk order: col0 a multiple of 8 and row0 a
    multiple of one 512-byte segment (512 rows at 8 bits, 1024 at 4 bits)."""
    rows = P.D - row0 if rows is None else rows
    cols = P.n - col0 if cols is None else cols
    assert 0 <= row0 and row0 + rows <= P.D and 0 <= col0 and col0 + cols <= P.n
    if P.bits != 32:
        assert col0 % 8 == 0 and (row0 * P.bits // 8) % 512 == 0
    else:
        assert row0 % 4 == 0
    off = col0 * P.col_stride + row0 * P.bits // 8
    desc = twa_basis(P.desc.data + off, (P.desc.scales + 4 * col0) if P.desc.scales else None,
                     int(rows), P.col_stride, int(cols), P.bits)
    return Basis(desc, P.data, P.scales)


def new_quantised_basis(D, n, bits, device):
    """Empty Basis with library-sized buffers, for twa_build_end_pass(2) to fill."""
    desc, data, scales = _new_quantised(D, n, bits, device)
    return Basis(desc, data, scales)


def basis_from_tensor(P32, D):
    """Descriptor for a float32 CUDA tensor (n, ld) holding a basis column per row."""
    assert P32.dtype == torch.float32 and P32.is_contiguous()
    n, ld = P32.shape
    desc = twa_basis(P32.data_ptr(), None, int(D), 4 * int(ld), int(n), 32)
    return Basis(desc, P32, None)


def _new_quantised(D, n, bits, device):
    data = torch.empty(twa_basis_bytes(D, n, bits), dtype=torch.uint8, device=device)
    scales = torch.empty(n, dtype=torch.float32, device=device)
    desc = twa_basis(data.data_ptr(), scales.data_ptr(), 0, 0, 0, 0)
    return desc, data, scales


def twa_quantize_basis(ctx, P32, bits, ws, out=None):
    """out: a Basis from new_quantised_basis to fill (None: buffers are allocated here)."""
    if out is None:
        out = new_quantised_basis(P32.D, P32.n, bits, P32.data.device)
    rc = load().twa_quantize_basis(ctx, ctypes.byref(P32.desc), int(bits), ctypes.byref(out.desc),
                                   _ptr(ws), ws.numel())
    _check(rc, "twa_quantize_basis", ctx)
    return out


def twa_basis_export(ctx, Pq):
    """Canonical codes (n, ceil(D*bits/8)) uint8 and scales (n,) float32, on the device."""
    row_bytes = (Pq.D * Pq.bits + 7) // 8
    codes = torch.empty((Pq.n, row_bytes), dtype=torch.uint8, device=Pq.data.device)
    scales = torch.empty(Pq.n, dtype=torch.float32, device=Pq.data.device)
    rc = load().twa_basis_export(ctx, ctypes.byref(Pq.desc), _ptr(codes), _ptr(scales))
    _check(rc, "twa_basis_export", ctx)
    return codes, scales


def twa_basis_import(ctx, codes, scales, D, bits):
    n = codes.shape[0]
    assert codes.dtype == torch.uint8 and codes.is_contiguous()
    assert codes.shape[1] == (D * bits + 7) // 8
    desc, data, sc = _new_quantised(D, n, bits, codes.device)
    rc = load().twa_basis_import(ctx, _ptr(codes), _ptr(scales), int(D), int(n), int(bits),
                                 ctypes.byref(desc))
    _check(rc, "twa_basis_import", ctx)
    return Basis(desc, data, sc)


def twa_project(ctx, P, g, c_out, ws):
    rc = load().twa_project(ctx, ctypes.byref(P.desc), _ptr(g), _dtype_code(g), _ptr(c_out),
                            _ptr(ws), ws.numel())
    _check(rc, "twa_project", ctx)
    return c_out


def twa_project_batch(ctx, P, G, C_out, ws):
    """G: (batch, ldg) gradients, one per row; C_out: (batch, n) float32."""
    assert G.dim() == 2 and G.is_contiguous() and C_out.is_contiguous()
    rc = load().twa_project_batch(ctx, ctypes.byref(P.desc), _ptr(G), int(G.shape[1]), int(G.shape[0]),
                                  _dtype_code(G), _ptr(C_out), _ptr(ws), ws.numel())
    _check(rc, "twa_project_batch", ctx)
    return C_out


def twa_project_batch_group(ctx, P, g_dtype=torch.bfloat16):
    code = _dtype_code(torch.empty(0, dtype=g_dtype))
    return int(load().twa_project_batch_group(ctx, ctypes.byref(P.desc), code))


def twa_lift(ctx, P, alpha, base, w_out, ws):
    rc = load().twa_lift(ctx, ctypes.byref(P.desc), _ptr(alpha), _ptr(base), _ptr(w_out),
                         _ptr(ws), ws.numel())
    _check(rc, "twa_lift", ctx)
    return w_out


def twa_step(ctx, P, g, lr, lam, alpha, wbar, w, ws, c_out=None):
    rc = load().twa_step(ctx, ctypes.byref(P.desc), _ptr(g), _dtype_code(g), float(lr), float(lam),
                         _ptr(alpha), _ptr(wbar), _ptr(w), _ptr(c_out), _ptr(ws), ws.numel())
    _check(rc, "twa_step", ctx)
    return w


def twa_step_host(ctx, P, g_host, lr, lam, alpha, wbar, w, w_host, g_stage, ws):
    """g_host / w_host: CPU tensors (pinned for asynchronous copies)."""
    assert not g_host.is_cuda and not w_host.is_cuda
    rc = load().twa_step_host(ctx, ctypes.byref(P.desc), _ptr(g_host), _dtype_code(g_host),
                              float(lr), float(lam), _ptr(alpha), _ptr(wbar), _ptr(w),
                              _ptr(w_host), _ptr(g_stage), _ptr(ws), ws.numel())
    _check(rc, "twa_step_host", ctx)
    return w_host


def twa_noalloc_last_error():
    return load().twa_noalloc_last_error().decode()


def twa_noalloc_scratch_bytes():
    return int(load().twa_noalloc_scratch_bytes())


def twa_project_noalloc(device, stream, P, g, c_out, status_out=None):
    """Projection that needs neither a context nor a workspace: for callers that cannot
    allocate device memory when they call (see include/twa.h).  `stream` is a
    torch.cuda.Stream or None for the current one; status_out an int32 CUDA tensor of 2."""
    if stream is None:
        stream = torch.cuda.current_stream(device)
    rc = load().twa_project_noalloc(int(device), ctypes.c_void_p(stream.cuda_stream),
                                    ctypes.byref(P.desc), _ptr(g), _dtype_code(g), _ptr(c_out),
                                    _ptr(status_out))
    if rc != TWA_OK:
        raise TwaError(rc, "twa_project_noalloc", twa_noalloc_last_error())
    return c_out


# --------------------------------------------------------------------------------------
# the paper's default construction: layer-wise, affine B-bit codes
# --------------------------------------------------------------------------------------
def _offsets(layers):
    arr = (ctypes.c_int64 * len(layers))(*[int(x) for x in layers])
    return arr, len(layers) - 1


class LayeredBasis:
    """A twa_layered_basis descriptor with the tensor that owns its memory."""

    def __init__(self, desc, mem, layers):
        self.desc = desc
        self.mem = mem
        self.layers = list(layers)

    D = property(lambda self: self.desc.D)
    L = property(lambda self: self.desc.L)
    n = property(lambda self: self.desc.codes.n // max(1, self.desc.planes))     # candidates
    bits = property(lambda self: self.desc.code_bits)                            # B of the quantiser
    slot_bits = property(lambda self: 16 if self.desc.planes == 2 else self.desc.codes.bits)


def twa_layered_workspace_bytes(layers, n):
    arr, L = _offsets(layers)
    return int(load().twa_layered_workspace_bytes(arr, L, int(n)))


def twa_layered_rows(layers, bits):
    arr, L = _offsets(layers)
    return int(load().twa_layered_rows(arr, L, int(bits)))


def twa_layered_basis_bytes(layers, n, bits):
    arr, L = _offsets(layers)
    return int(load().twa_layered_basis_bytes(arr, L, int(n), int(bits)))


def new_layered_workspace(layers, n, device):
    return torch.empty(twa_layered_workspace_bytes(layers, n), dtype=torch.uint8, device=device)


def twa_build_centered(ctx, W, D, layers, wbar_out, lws):
    assert W.dtype == torch.float32 and W.is_contiguous()
    n, ldw = W.shape
    arr, L = _offsets(layers)
    desc = twa_basis()
    rc = load().twa_build_centered(ctx, _ptr(W), int(D), int(n), int(ldw), arr, L, _ptr(wbar_out),
                                   ctypes.byref(desc), _ptr(lws), lws.numel())
    _check(rc, "twa_build_centered", ctx)
    return Basis(desc, W, None)


def twa_quantize_affine(ctx, P32, layers, bits, lws, mem=None):
    """mem: a uint8 CUDA tensor of twa_layered_basis_bytes(layers, n, bits) bytes to hold the basis
    (None: allocated here)."""
    arr, L = _offsets(layers)
    if mem is None:
        mem = torch.empty(twa_layered_basis_bytes(layers, P32.n, bits), dtype=torch.uint8,
                          device=P32.data.device)
    desc = twa_layered_basis()
    rc = load().twa_quantize_affine(ctx, ctypes.byref(P32.desc), arr, L, int(bits), _ptr(mem),
                                    mem.numel(), ctypes.byref(desc), _ptr(lws), lws.numel())
    _check(rc, "twa_quantize_affine", ctx)
    return LayeredBasis(desc, mem, layers)


def twa_layered_build_begin(ctx, D, n, layers, bits, lws, device):
    """Starts a row-chunked layer-wise build; returns the (still empty) LayeredBasis."""
    arr, L = _offsets(layers)
    mem = torch.empty(twa_layered_basis_bytes(layers, n, bits), dtype=torch.uint8, device=device)
    desc = twa_layered_basis()
    rc = load().twa_layered_build_begin(ctx, int(D), int(n), arr, L, int(bits), _ptr(mem), mem.numel(),
                                        ctypes.byref(desc), _ptr(lws), lws.numel())
    _check(rc, "twa_layered_build_begin", ctx)
    return LayeredBasis(desc, mem, layers)


def twa_layered_build_feed(ctx, lb, pass_index, chunk, row0, rows, wbar, lws, q32_out=None):
    """chunk: (n, ld) float32 CUDA tensor, candidate i's rows row0 .. row0+rows-1 in chunk[i, :rows]."""
    assert chunk.dtype == torch.float32 and chunk.stride(1) == 1
    arr, _ = _offsets(lb.layers)
    ldq = q32_out.stride(0) if q32_out is not None else 0
    rc = load().twa_layered_build_feed(ctx, ctypes.byref(lb.desc), arr, int(pass_index), _ptr(chunk),
                                       int(chunk.stride(0)), int(row0), int(rows), _ptr(wbar), _ptr(q32_out),
                                       int(ldq), _ptr(lws), lws.numel())
    _check(rc, "twa_layered_build_feed", ctx)


def twa_layered_build_end_pass(ctx, lb, pass_index, lws):
    arr, _ = _offsets(lb.layers)
    rc = load().twa_layered_build_end_pass(ctx, ctypes.byref(lb.desc), arr, int(pass_index), _ptr(lws), lws.numel())
    _check(rc, "twa_layered_build_end_pass", ctx)


def twa_layered_export(ctx, lb):
    """Canonical unsigned codes (n, ceil(D*slot/8)) uint8 in flat row order (slot = 1, 2, 4, 8 or 16
    bits per code; 3-bit codes sit in 4-bit slots, 16-bit codes low byte first) and the factors a, b."""
    row_bytes = (lb.D * lb.slot_bits + 7) // 8
    dev = lb.mem.device
    codes = torch.empty((lb.n, row_bytes), dtype=torch.uint8, device=dev)
    a = torch.empty(lb.L, dtype=torch.float32, device=dev)
    b = torch.empty(lb.L, dtype=torch.float32, device=dev)
    _check(load().twa_layered_export(ctx, ctypes.byref(lb.desc), _ptr(codes), _ptr(a), _ptr(b)),
           "twa_layered_export", ctx)
    return codes, a, b


def twa_layered_step_workspace_bytes(lb):
    return int(load().twa_layered_step_workspace_bytes(ctypes.byref(lb.desc)))


def new_layered_step_workspace(lb):
    return torch.empty(twa_layered_step_workspace_bytes(lb), dtype=torch.uint8, device=lb.mem.device)


def twa_layered_project(ctx, lb, g, c_out, sws):
    """c_out: (L, n) float32, layer-major."""
    rc = load().twa_layered_project(ctx, ctypes.byref(lb.desc), _ptr(g), _dtype_code(g), _ptr(c_out),
                                    _ptr(sws), sws.numel())
    _check(rc, "twa_layered_project", ctx)
    return c_out


def twa_layered_lift(ctx, lb, beta, base, w_out, sws):
    rc = load().twa_layered_lift(ctx, ctypes.byref(lb.desc), _ptr(beta), _ptr(base), _ptr(w_out),
                                 _ptr(sws), sws.numel())
    _check(rc, "twa_layered_lift", ctx)
    return w_out


def twa_layered_step(ctx, lb, g, lr, lam, beta, wbar, w, sws, c_out=None):
    rc = load().twa_layered_step(ctx, ctypes.byref(lb.desc), _ptr(g), _dtype_code(g), float(lr), float(lam),
                                 _ptr(beta), _ptr(wbar), _ptr(w), _ptr(c_out), _ptr(sws), sws.numel())
    _check(rc, "twa_layered_step", ctx)
    return w


def _adam(lr, step, beta1, beta2, eps, weight_decay):
    return twa_adam(float(lr), float(beta1), float(beta2), float(eps), float(weight_decay), int(step))


def twa_step_adam(ctx, P, g, lr, step, alpha, m, v, wbar, w, ws, beta1=0.9, beta2=0.999, eps=1e-8,
                  weight_decay=0.0, c_out=None):
    opt = _adam(lr, step, beta1, beta2, eps, weight_decay)
    rc = load().twa_step_adam(ctx, ctypes.byref(P.desc), _ptr(g), _dtype_code(g), ctypes.byref(opt), _ptr(alpha),
                              _ptr(m), _ptr(v), _ptr(wbar), _ptr(w), _ptr(c_out), _ptr(ws), ws.numel())
    _check(rc, "twa_step_adam", ctx)
    return w


def twa_layered_step_adam(ctx, lb, g, lr, step, beta, m, v, wbar, w, sws, beta1=0.9, beta2=0.999, eps=1e-8,
                          weight_decay=0.0, c_out=None):
    opt = _adam(lr, step, beta1, beta2, eps, weight_decay)
    rc = load().twa_layered_step_adam(ctx, ctypes.byref(lb.desc), _ptr(g), _dtype_code(g), ctypes.byref(opt),
                                      _ptr(beta), _ptr(m), _ptr(v), _ptr(wbar), _ptr(w), _ptr(c_out), _ptr(sws),
                                      sws.numel())
    _check(rc, "twa_layered_step_adam", ctx)
    return w


def twa_cosine_lr(base_lr, step, total_steps, min_lr=0.0):
    return float(load().twa_cosine_lr(float(base_lr), int(step), int(total_steps), float(min_lr)))


def twa_weighted_average(ctx, W, D, weights, w_out, ws):
    """W: (n, ldw) float32 candidates, one per row; weights: (n,) float32 on the device."""
    assert W.dtype == torch.float32 and W.is_contiguous()
    rc = load().twa_weighted_average(ctx, _ptr(W), int(D), int(W.shape[0]), int(W.shape[1]), _ptr(weights),
                                     _ptr(w_out), _ptr(ws), ws.numel())
    _check(rc, "twa_weighted_average", ctx)
    return w_out
