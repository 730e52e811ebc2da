"""Seeded synthetic inputs for the FFT-convolution workloads.

This module holds shapes and random-number recipes only -- none of the
method's arithmetic -- so that the CUDA path and the CPU oracle can be fed the
very same arrays.  It imports neither of them.

The five workloads mirror the layer shapes the paper evaluates (its Table 2
"representative layers" and the parameter grid of Section 4.1): x is
[S, f, h, w], w is [f', f, kh, kw], dy is [S, f', h-kh+1, w-kw+1], all fp32.
Values: activations U(-1, 1); weights N(0, variance 1/(f*kh*kw)) (fan-in
scaling) for the three layer configs, U(-1, 1) for the tiny config and the
sweep; output gradients N(0, 1), U(-1, 1) in the sweep.
Seeds: numpy.random.default_rng([14127580, cfg, point, tensor]) with tensor
0 = x, 1 = w, 2 = dy.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

SEED_ROOT = 14127580


@dataclass(frozen=True)
class ConvShape:
    name: str
    S: int
    f: int
    fp: int
    h: int
    w: int
    kh: int
    kw: int
    n: int
    cfg: int = 0          # seed component: which config
    point: int = 0        # seed component: which sweep point
    w_dist: str = "uniform"   # "uniform" | "fan_in"
    dy_dist: str = "normal"   # "normal" | "uniform"

    @property
    def oh(self) -> int:
        return self.h - self.kh + 1

    @property
    def ow(self) -> int:
        return self.w - self.kw + 1

    @property
    def macs(self) -> int:
        """Equivalent time-domain multiply-adds of one pass (the paper's
        'equivalent time-domain reductions', Section 4.2)."""
        return self.S * self.f * self.fp * self.kh * self.kw * self.oh * self.ow

    def args(self):
        return (self.S, self.f, self.fp, self.h, self.w, self.kh, self.kw, self.n)


def next_pow2(v: int) -> int:
    n = 1
    while n < v:
        n *= 2
    return n


CONFIGS = {
    # index = position in the list of benchmark configs (0-based)
    0: ConvShape("tiny_S8_f4_fp8_16x16_k3", 8, 4, 8, 16, 16, 3, 3, 16, cfg=1,
                 w_dist="uniform", dy_dist="normal"),
    1: ConvShape("mid_S128_f96_fp256_31x31_k5", 128, 96, 256, 31, 31, 5, 5, 32, cfg=2,
                 w_dist="fan_in", dy_dist="normal"),
    2: ConvShape("largek_S128_f64_fp64_64x64_k11", 128, 64, 64, 64, 64, 11, 11, 64, cfg=3,
                 w_dist="fan_in", dy_dist="normal"),
    3: ConvShape("deep_S128_f384_fp384_13x13_k3", 128, 384, 384, 13, 13, 3, 3, 16, cfg=4,
                 w_dist="fan_in", dy_dist="normal"),
}

SWEEP_S = (1, 16, 64, 128)
SWEEP_F = (1, 16, 64, 128, 256, 384)
SWEEP_H = (13, 16, 27, 32, 57, 64, 120, 128)
SWEEP_K = (3, 5, 7, 9, 11, 13)


def sweep_grid():
    """The full sweep grid (config index 4), in a fixed order; every point has
    k <= h.  Point ids are positions in this list."""
    pts = []
    for S in SWEEP_S:
        for f in SWEEP_F:
            for fp in SWEEP_F:
                for h in SWEEP_H:
                    for k in SWEEP_K:
                        if k <= h:
                            pts.append((S, f, fp, h, k))
    return pts


def sweep_points(count: int = 1000, seed: int = SEED_ROOT):
    """`count` grid points drawn without replacement, seeded; returns ConvShapes."""
    grid = sweep_grid()
    rng = np.random.default_rng([seed, 5])
    idx = np.sort(rng.choice(len(grid), size=min(count, len(grid)), replace=False))
    out = []
    for p in idx:
        S, f, fp, h, k = grid[int(p)]
        out.append(ConvShape("sweep_%d_S%d_f%d_fp%d_h%d_k%d" % (p, S, f, fp, h, k),
                             S, f, fp, h, h, k, k, max(8, next_pow2(h)), cfg=5,
                             point=int(p), w_dist="uniform", dy_dist="uniform"))
    return out


def _rng(shape: ConvShape, tensor: int):
    return np.random.default_rng([SEED_ROOT, shape.cfg, shape.point, tensor])


def _uniform(rng, dims):
    return (rng.random(dims, dtype=np.float32) * np.float32(2.0) - np.float32(1.0))


def _normal(rng, dims, std=1.0):
    return (rng.standard_normal(dims, dtype=np.float32) * np.float32(std))


def make_x(s: ConvShape) -> np.ndarray:
    return _uniform(_rng(s, 0), (s.S, s.f, s.h, s.w))


def make_w(s: ConvShape) -> np.ndarray:
    dims = (s.fp, s.f, s.kh, s.kw)
    if s.w_dist == "fan_in":
        return _normal(_rng(s, 1), dims, std=(s.f * s.kh * s.kw) ** -0.5)
    return _uniform(_rng(s, 1), dims)


def make_dy(s: ConvShape) -> np.ndarray:
    dims = (s.S, s.fp, s.oh, s.ow)
    if s.dy_dist == "normal":
        return _normal(_rng(s, 2), dims)
    return _uniform(_rng(s, 2), dims)


def make_planes(batch: int, h: int, w: int, seed: int) -> np.ndarray:
    """Plain U(-1,1) planes for the bare-transform tests."""
    rng = np.random.default_rng([SEED_ROOT, 99, seed])
    return _uniform(rng, (batch, h, w))


def sample_coords(dims, count: int, seed: int) -> np.ndarray:
    """Seeded sample of coordinates of a 4-D tensor: its 16 corners, then
    uniform random points; int32 [count, 4]."""
    dims = tuple(int(d) for d in dims)
    rng = np.random.default_rng([SEED_ROOT, 77, seed])
    corners = np.array([[(d - 1) * ((c >> k) & 1) for k, d in enumerate(dims)]
                        for c in range(16)], dtype=np.int64)
    rnd = np.stack([rng.integers(0, d, size=max(count - 16, 0)) for d in dims], axis=1)
    out = np.concatenate([corners, rnd], axis=0)[:max(count, 1)]
    return np.ascontiguousarray(out, dtype=np.int32)


def shard_range(S: int, rank: int, world: int):
    """Contiguous slice [lo, hi) of the minibatch owned by `rank` when S samples are
    split over `world` data-parallel ranks (sizes differ by at most one)."""
    base, extra = divmod(int(S), int(world))
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def plane_coords(dims, seed: int) -> np.ndarray:
    """Three coordinates from every plane of a 4-D tensor [a, b, rows, cols]: one uniform
    random element, one in the last row and one in the last column (the edges that a
    mis-clipped tile would get wrong); int32 [3 * a * b, 4]."""
    a, b, rows, cols = (int(d) for d in dims)
    rng = np.random.default_rng([SEED_ROOT, 78, seed])
    pa, pb = np.meshgrid(np.arange(a), np.arange(b), indexing="ij")
    pa, pb = pa.ravel(), pb.ravel()
    n = pa.size
    parts = []
    for r, c in ((rng.integers(0, rows, n), rng.integers(0, cols, n)),
                 (np.full(n, rows - 1), rng.integers(0, cols, n)),
                 (rng.integers(0, rows, n), np.full(n, cols - 1))):
        parts.append(np.stack([pa, pb, r, c], axis=1))
    return np.ascontiguousarray(np.concatenate(parts, axis=0), dtype=np.int32)


def sweep_host_bytes(s: ConvShape) -> int:
    """Bytes of the three input tensors and three results of a sweep point on the host."""
    return 8 * (s.S * s.f * s.h * s.w + s.fp * s.f * s.kh * s.kw + s.S * s.fp * s.oh * s.ow)


def sweep_stratified(per_n_large: int = 8, per_n_other: int = 6, count: int = 1000,
                     max_host_bytes: int = 5 << 29):
    """A stratified, seeded slice of the `count`-point sweep: for every basis n in
    {16, 32, 64, 128}, `per_n_large` points whose S, f and f' are all >= 64 (many
    contraction tiles) and `per_n_other` points from the rest (small shapes, where the plan
    resolves to the FP32 contraction, included).  Points whose tensors exceed
    `max_host_bytes` on the host are passed over, so that a time-boxed run is dominated by
    the GPU and the oracle, not by drawing random numbers."""
    pts = sweep_points(count)
    order = np.random.default_rng([SEED_ROOT, 56]).permutation(len(pts))
    out = []
    for n in (16, 32, 64, 128):
        large, other = [], []
        for oi in order:
            s = pts[int(oi)]
            if s.n != n or sweep_host_bytes(s) > max_host_bytes:
                continue
            if min(s.S, s.f, s.fp) >= 64:
                if len(large) < per_n_large:
                    large.append(s)
            elif len(other) < per_n_other:
                other.append(s)
        out.append(large + other)
    # round robin over the bases, so that a run stopped early has still seen all of them
    mixed = []
    for i in range(max(len(g) for g in out)):
        mixed.extend(g[i] for g in out if i < len(g))
    return mixed
