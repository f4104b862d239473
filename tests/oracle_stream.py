"""Test harness: the float64 oracle applied to matrices too large for one call.

The projection is a sum over rows, so the oracle's project() on consecutive row chunks, added
up in chunk order, is the oracle's projection of the whole matrix; the chunks are handed to a
few host threads (numpy releases the interpreter lock inside its array loops).  Nothing here
replaces the oracle: unpacking, the dot products and the scaling are oracle.unpack_codes /
oracle.project / oracle.project_f32 calls on slices.  What this module adds itself is only the
weighted sum of the gradients of a sequence.
"""

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from oracle import twa_oracle as orc

CHUNK = 1 << 18            # rows per call of the oracle: the float64 copy of a column slice stays in cache
THREADS = max(1, min(32, (os.cpu_count() or 1)))


def _pool():
    return ThreadPoolExecutor(max_workers=THREADS)


def _chunks(D, chunk=CHUNK):
    return [(r0, min(D, r0 + chunk)) for r0 in range(0, D, chunk)]


def project_packed(packed, scales, D, bits, gs):
    """oracle.project of the canonical code image `packed` (n x ceil(D*bits/8) uint8, host) with every
    gradient of the list gs ((D,) arrays) in one pass over the codes: returns C (n, len(gs))."""
    n = packed.shape[0]
    step = CHUNK * 16                      # a multiple of every code group

    def part(rng):
        r0, r1 = rng
        co = orc.unpack_codes(packed[:, r0 * bits // 8:(r1 * bits + 7) // 8], r1 - r0, bits)
        c = np.zeros((n, len(gs)))
        for q0, q1 in _chunks(r1 - r0):
            for b, g in enumerate(gs):
                c[:, b] += orc.project(co[q0:q1], scales, g[r0 + q0:r0 + q1])
        return c

    with _pool() as pool:
        parts = list(pool.map(part, _chunks(D, step)))
    c = np.zeros((n, len(gs)))
    for pc in parts:                         # chunk order
        c += pc
    return c


def project_f32_columns(cols, gs):
    """oracle.project_f32 of float32 columns (D x k, host) with every gradient of gs: (k, len(gs))."""
    D, k = cols.shape

    def part(rng):
        r0, r1 = rng
        return np.stack([orc.project_f32(cols[r0:r1], g[r0:r1]) for g in gs], axis=1)

    with _pool() as pool:
        parts = list(pool.map(part, _chunks(D)))
    c = np.zeros((k, len(gs)))
    for pc in parts:
        c += pc
    return c


class HostColumns:
    """Some columns of a basis on the host, unpacked once, for many projections in a row (the
    step-by-step oracle of a sequence of training steps).  bits 8 / 4: `values` are the code
    VALUES (D x k int8) with their scales; bits 32: the float32 columns (D x k)."""

    def __init__(self, values, scales, bits):
        self.values, self.scales, self.bits = values, scales, bits
        self.D, self.k = values.shape

    @classmethod
    def from_packed(cls, packed, scales, D, bits):
        return cls(orc.unpack_codes(packed, D, bits), np.asarray(scales), bits)

    def project(self, g_host):
        def part(rng):
            r0, r1 = rng
            if self.bits == 32:
                return orc.project_f32(self.values[r0:r1], g_host[r0:r1])
            return orc.project(self.values[r0:r1], self.scales, g_host[r0:r1])
        with _pool() as pool:
            parts = list(pool.map(part, _chunks(self.D)))
        c = np.zeros(self.k)
        for p in parts:
            c += p
        return c


class WeightedGradientSum:
    """G = sum_t (1 - lr*lam)^(T-1-t) g_t in float64, gradient after gradient.  By linearity of the
    projection, T steps alpha <- (1 - lr*lam) alpha - lr P~^T g_t from alpha = 0 end at
    alpha_T = -lr P~^T G (pinned against the step-by-step recursion in tests/test_oracle_step.py)."""

    def __init__(self, D, T, lr, lam):
        self.acc = np.zeros(D, dtype=np.float64)
        self.T, self.decay, self.t = T, 1.0 - lr * lam, 0

    def add(self, g_host):
        wgt = self.decay ** (self.T - 1 - self.t)
        self.t += 1

        def part(rng):
            r0, r1 = rng
            if wgt == 1.0:
                np.add(self.acc[r0:r1], g_host[r0:r1], out=self.acc[r0:r1])     # widened to float64 by the add
            else:
                self.acc[r0:r1] += wgt * g_host[r0:r1].astype(np.float64)
        with _pool() as pool:
            list(pool.map(part, _chunks(self.acc.shape[0])))

    def result(self):
        assert self.t == self.T
        return self.acc


def weighted_gradient_sum(grads, lr, lam):
    acc = WeightedGradientSum(grads[0].shape[0], len(grads), lr, lam)
    for g in grads:
        acc.add(np.asarray(g))
    return acc.result()
