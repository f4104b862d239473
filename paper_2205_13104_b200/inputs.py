"""Seeded synthetic inputs for the TWA subspace path.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no mean, no orthogonalisation, no quantisation, no
projection).  Both the CUDA tests and the CPU oracle tests take their inputs
from here, so the two sides always see the same bytes.

The candidates stand in for checkpoints sampled along SGD trajectories, whose
pairwise cosine similarity the paper reports as about 0.99 (Section 5.5,
the decoupling ablation): a correlated random walk

    w_0 ~ N(0, w0_std^2),   w_i = w_{i-1} + step * xi_i + drift * d,

with xi_i ~ N(0, 1) iid and one shared drift direction d ~ N(0, 1).

Layout: a set of n vectors in R^D is a torch tensor of shape (n, ld) with
ld >= D; row i is vector i, i.e. the D x n matrix in column-major order with
leading dimension ld.  Elements [D, ld) of every row are zero.

Random numbers are drawn per chunk of CHUNK_ROWS rows from a generator seeded
by (seed, stream, chunk index), so any row range that starts and ends on a
chunk boundary can be regenerated on its own, on any device of the same kind.
CPU and CUDA generators give different streams; a test generates once and
copies.
"""

from __future__ import annotations

from dataclasses import dataclass

import torch

CHUNK_ROWS = 1 << 22

_STREAM_TRAJECTORY = 1
_STREAM_SHARED_W0 = 2
_STREAM_INTEGERS = 9
_STREAM_GRADIENT = 3


def _mix(x):
    # splitmix64 finaliser: spreads (seed, stream, index) over all 64 bits, because
    # some generators only look at part of the seed
    x &= (1 << 64) - 1
    x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & ((1 << 64) - 1)
    x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & ((1 << 64) - 1)
    return x ^ (x >> 31)


def _generator(device, seed, stream, index):
    g = torch.Generator(device=device)
    key = _mix(_mix(_mix(int(seed)) + int(stream)) + int(index))
    g.manual_seed(key & 0x7FFFFFFFFFFFFFFF)
    return g


def padded_ld(D, multiple=128):
    """Smallest multiple of `multiple` elements that holds D."""
    return ((int(D) + multiple - 1) // multiple) * multiple


def _chunks(D, row0=0, rows=None):
    rows = D - row0 if rows is None else rows
    end = row0 + rows
    assert row0 % CHUNK_ROWS == 0, "row ranges must start on a chunk boundary"
    assert end == D or end % CHUNK_ROWS == 0, "row ranges must end on a chunk boundary or at D"
    r = row0
    while r < end:
        nr = min(CHUNK_ROWS, D - r)
        yield r // CHUNK_ROWS, r, nr
        r += nr


def trajectory_rows(D, n, step, drift, seed, device, row0=0, rows=None,
                    w0_std=0.05, out=None):
    """Rows [row0, row0+rows) of one trajectory's candidates w_0 .. w_{n-1}.

    Returns a float32 tensor (n, rows) (or fills `out[:, :rows]`).  Draw order
    inside a chunk: w_0, d, xi_1 .. xi_{n-1}.
    """
    rows = D - row0 if rows is None else rows
    if out is None:
        out = torch.zeros((n, rows), dtype=torch.float32, device=device)
    for ci, r, nr in _chunks(D, row0, rows):
        gen = _generator(device, seed, _STREAM_TRAJECTORY, ci)
        z = torch.randn((n + 1, nr), generator=gen, dtype=torch.float32, device=device)
        dst = out[:, r - row0: r - row0 + nr]
        dst[0] = z[0] * w0_std
        d = z[1] * drift
        for i in range(1, n):
            dst[i] = dst[i - 1] + z[i + 1] * step + d
        del z
    return out


def trajectory_candidates(D, n, step, drift, seed, device, ld=None, w0_std=0.05):
    """All candidates of one trajectory as an (n, ld) tensor, pad columns zero."""
    ld = padded_ld(D) if ld is None else ld
    W = torch.zeros((n, ld), dtype=torch.float32, device=device)
    trajectory_rows(D, n, step, drift, seed, device, out=W[:, :D], w0_std=w0_std)
    return W


def multi_trajectory_candidates(D, groups, per_group, step, drift, seed, device,
                                ld=None, w0_std=0.05):
    """groups x per_group candidates: every trajectory starts from one shared
    w_0 (which is not itself a candidate) and contributes w_{t,1..per_group};
    trajectory t draws its steps from seed + 1 + t; the drift direction d is
    shared by all trajectories."""
    ld = padded_ld(D) if ld is None else ld
    n = groups * per_group
    W = torch.zeros((n, ld), dtype=torch.float32, device=device)
    for ci, r, nr in _chunks(D):
        gen = _generator(device, seed, _STREAM_SHARED_W0, ci)
        z = torch.randn((2, nr), generator=gen, dtype=torch.float32, device=device)
        w0 = z[0] * w0_std
        d = z[1] * drift
        for t in range(groups):
            gt = _generator(device, seed + 1 + t, _STREAM_TRAJECTORY, ci)
            xi = torch.randn((per_group, nr), generator=gt, dtype=torch.float32,
                             device=device)
            prev = w0
            for i in range(per_group):
                cur = prev + xi[i] * step + d
                W[t * per_group + i, r: r + nr] = cur
                prev = cur
            del xi
    return W


def small_integers(out, low, high, seed):
    """Fills the rows of `out` (k, D) with integers drawn uniformly from [low, high]: sums of products of
    such values are exact in float32 whatever the order of the additions, so a result on them is
    one number, not a number within a bound."""
    k, D = out.shape
    for ci, r, nr in _chunks(D):
        gen = _generator(out.device, seed, _STREAM_INTEGERS, ci)
        z = torch.randint(low, high + 1, (k, nr), generator=gen, device=out.device)
        out[:, r: r + nr] = z.to(out.dtype)
    return out


def gradient(D, std, seed, step_index, dtype, device, out=None):
    """One gradient g ~ N(0, std^2) of length D in `dtype` (float32 or
    bfloat16; bfloat16 is rounded from the float32 draw)."""
    if out is None:
        out = torch.empty((D,), dtype=dtype, device=device)
    for ci, r, nr in _chunks(D):
        gen = _generator(device, seed, _STREAM_GRADIENT, step_index * 4096 + ci)
        z = torch.randn((nr,), generator=gen, dtype=torch.float32, device=device)
        out[r: r + nr] = (z * std).to(dtype)
    return out


@dataclass(frozen=True)
class Workload:
    """One synthetic configuration (shapes of flat parameter vectors of
    ResNet-18/50, ViT-B/16 and a 1.3 B decoder, plus a tiny case)."""
    name: str
    D: int
    n: int
    step: float
    drift: float
    g_std: float
    g_dtype: str          # "f32" | "bf16"
    bits: tuple           # storage widths of P exercised
    steps: int
    groups: int = 1       # >1: n = groups * (n // groups) trajectories from a shared w_0
    seed: int = 0
    chunked_build: bool = False

    def candidates(self, device, ld=None):
        if self.groups > 1:
            return multi_trajectory_candidates(self.D, self.groups, self.n // self.groups,
                                               self.step, self.drift, self.seed, device, ld)
        return trajectory_candidates(self.D, self.n, self.step, self.drift, self.seed,
                                     device, ld)

    def gradient(self, step_index, device, out=None):
        dt = torch.bfloat16 if self.g_dtype == "bf16" else torch.float32
        return gradient(self.D, self.g_std, self.seed, step_index, dt, device, out)


WORKLOADS = {
    "tiny": Workload("tiny", 1_048_576, 10, 0.01, 0.002, 1e-3, "f32", (32,), 1),
    "resnet18": Workload("resnet18", 11_173_962, 20, 0.005, 0.001, 1e-3, "f32", (32, 8), 100),
    "resnet50": Workload("resnet50", 25_557_032, 50, 0.005, 0.001, 1e-3, "f32", (8,), 100,
                         groups=5),
    "vitb16": Workload("vitb16", 86_567_656, 100, 0.003, 0.001, 1e-4, "bf16", (8, 4), 100),
    "decoder1p3b": Workload("decoder1p3b", 1_315_758_080, 32, 0.002, 0.0005, 1e-4, "bf16",
                            (8, 4), 50, chunked_build=True),
}


# --------------------------------------------------------------------------------------
# Layer partitions: the sizes of the parameter tensors of the architectures the workloads
# stand for, in definition order; each tensor is one "layer" of the layer-wise method.
# --------------------------------------------------------------------------------------
def _offsets_from_sizes(sizes):
    out = [0]
    for s in sizes:
        out.append(out[-1] + int(s))
    return out


def _vit_b16_sizes():
    d, mlp, patch, tokens, classes = 768, 3072, 16, 197, 1000
    s = [d, tokens * d, d * 3 * patch * patch, d]                # class token, positions, patch embedding
    for _ in range(12):
        s += [d, d, 3 * d * d, 3 * d, d * d, d, d, d, mlp * d, mlp, d * mlp, d]
    s += [d, d, d * classes, classes]
    return s


def _decoder_1p3b_sizes():
    d, ffn, vocab, positions = 2048, 8192, 50272, 2050
    s = [vocab * d, positions * d]
    for _ in range(24):
        s += [d * d, d] * 4 + [d, d, ffn * d, ffn, d * ffn, d, d, d]
    s += [d, d]
    return s


def _resnet18_sizes():
    # 3x3 stem, four stages of two basic blocks, 10 classes
    s = [64 * 3 * 9, 64, 64]
    cin = 64
    for cout, stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        for b in range(2):
            s += [cout * cin * 9, cout, cout, cout * cout * 9, cout, cout]
            if b == 0 and (stride != 1 or cin != cout):
                s += [cout * cin, cout, cout]
            cin = cout
    s += [512 * 10, 10]
    return s


def _resnet50_sizes():
    # 7x7 stem, bottleneck stages of 3, 4, 6, 3 blocks, 1000 classes
    s = [64 * 3 * 49, 64, 64]
    cin = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        cout = 4 * width
        for b in range(blocks):
            s += [width * cin, width, width, width * width * 9, width, width, cout * width, cout, cout]
            if b == 0:
                s += [cout * cin, cout, cout]
            cin = cout
    s += [2048 * 1000, 1000]
    return s


_LAYER_SIZES = {"vitb16": _vit_b16_sizes, "decoder1p3b": _decoder_1p3b_sizes,
                "resnet18": _resnet18_sizes, "resnet50": _resnet50_sizes}


def layer_offsets(name, D=None):
    """L+1 row offsets of the layers of workload `name`.  With D given and different from the
    workload's size (a cut-down run), the partition is cut at D (or its last layer extended)."""
    if name in _LAYER_SIZES:
        off = _offsets_from_sizes(_LAYER_SIZES[name]())
    else:
        total = WORKLOADS[name].D
        off = _offsets_from_sizes([total // 8] * 7 + [total - 7 * (total // 8)])
    if D is not None and D != off[-1]:
        off = [o for o in off if o < D] + [D]
    return off
