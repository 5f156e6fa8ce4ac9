"""Seeded synthetic inputs shaped like the video-DiT workloads.

This module only manufactures DATA (token grids, cluster maps, Gaussian
centroid-plus-noise tensors, dtype rounding).  It holds none of the attention
method's arithmetic, so both the CUDA path and the independent CPU checker can
be fed the very same bytes from it.

Recipe: tokens live on a (T, Hg, Wg) latent grid, token index
n = (t*Hg + h)*Wg + w.  Every token belongs to a cluster c(n) given by a
spatiotemporal region map.  For each head a centroid table mu^X[n_c, d] and noise
eps ~ N(0,1) are drawn per tensor X in {Q, K, V}, and X_n = mu^X[c(n)] +
sigma(n) * eps_n.  mu^Q and mu^V are independent N(0,1) tables; the key table is
aligned with the query table, mu^K = c mu^Q + sqrt(1 - c^2) nu with nu ~ N(0,1)
independent and c = `qk_align` (0.7): a query's logit against the keys of its own
region is then c sqrt(d) above the zero-mean logits against other regions, so
that same-region pairs carry most of the softmax mass, as "3D-local clusters"
implies, while a broad background remains (with c = 0 attention on these inputs
is nearly uniform and no sparse support can represent it; with c = 1 it is
one-hot per region).  Q and K are then multiplied by d^(-1/4) (the symmetric
folding of the 1/sqrt(d) logit scale into the inputs; calls on these tensors
therefore use softmax_scale = 1), and everything is rounded to the workload's
storage type.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    grid: tuple            # (T, Hg, Wg)
    H: int
    d: int
    dtype: str             # "f32" | "bf16"
    cluster_map: str       # key into _CLUSTER_MAPS
    block: int
    density: float
    n_sample: int
    n_probe: int
    sigma: float = 0.5
    n_sink: int = 0
    softmax_scale: float = 1.0
    qk_align: float = 0.7  # correlation c of the key centroid table with the query centroid table

    @property
    def N(self) -> int:
        T, Hg, Wg = self.grid
        return T * Hg * Wg

    def scaled(self, **kw) -> "Workload":
        """A smaller copy (fewer frames / heads / probes) for tests."""
        return replace(self, **kw)


def _coords(grid):
    T, Hg, Wg = grid
    n = np.arange(T * Hg * Wg)
    return n // (Hg * Wg), (n // Wg) % Hg, n % Wg


def _map_tiny(grid, head, H):
    t, h, w = _coords(grid)
    return (h // 8) * 4 + (w // 8)                      # 16 regions of 1x8x8, same ids every frame


def _map_480p(grid, head, H):
    T, Hg, Wg = grid
    t, h, w = _coords(grid)
    return ((t // 3) * (-(-Hg // 6)) + (h // 6)) * (-(-Wg // 8)) + (w // 8)   # 3x6x8 regions


def _map_720p(grid, head, H):
    T, Hg, Wg = grid
    t, h, w = _coords(grid)
    if head < H // 2:                                   # temporal-local 7x5x5
        return ((t // 7) * (-(-Hg // 5)) + (h // 5)) * (-(-Wg // 5)) + (w // 5)
    return (t * (-(-Hg // 15)) + (h // 15)) * (-(-Wg // 16)) + (w // 16)      # spatial-local 1x15x16


def _map_world(grid, head, H):
    t, h, w = _coords(grid)
    return ((t // 2) % 4) * 64 + ((h // 4) % 8) * 8 + ((w // 8) % 8)          # table shared across segments


_CLUSTER_MAPS = {"tiny": _map_tiny, "480p": _map_480p, "720p": _map_720p, "world": _map_world}

TINY = Workload("tiny-f32", 0, (4, 32, 32), 2, 64, "f32", "tiny", 64, 0.25, 64, 32)
VIDEO_480P = Workload("video-dit-480p-like", 1, (21, 30, 52), 24, 128, "bf16", "480p", 128, 0.25, 256, 128, n_sink=4)
VIDEO_720P = Workload("video-dit-720p-like", 2, (21, 45, 80), 40, 128, "bf16", "720p", 128, 0.22, 256, 128)
WORLD = Workload("world-model-like", 3, (24, 32, 64), 32, 128, "bf16", "world", 128, 0.26, 256, 192)
CONFIGS = {w.name: w for w in (TINY, VIDEO_480P, VIDEO_720P, WORLD)}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); the result
    is returned as float32 holding exactly representable values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 storage of float32 values that are already bfloat16-exact."""
    return (np.ascontiguousarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def _sigma(wl: Workload):
    if wl.cluster_map != "world":
        return wl.sigma
    t, _, _ = _coords(wl.grid)
    T = wl.grid[0]
    return np.where(t < T // 3, 0.3, 1.0)[:, None]       # conditioning frames vs prediction frames


def make_head(wl: Workload, head: int, seed: int = 0, step: int = 0):
    """Q, K, V of one head as float32 arrays [N, d] whose values are exactly
    representable in the workload's storage type.  `step` > 0 keeps the centroid
    tables of (seed, head) and draws fresh noise: successive calls over the same
    scene, the stand-in for successive denoising steps."""
    cmap = _CLUSTER_MAPS[wl.cluster_map](wl.grid, head, wl.H)
    n_c = int(cmap.max()) + 1
    sig = _sigma(wl)
    out = []
    tables = []
    for tensor_id in range(3):
        rng = np.random.default_rng([seed, wl.cfg_id, head, tensor_id])
        mu = rng.standard_normal((n_c, wl.d), dtype=np.float32)
        eps = rng.standard_normal((wl.N, wl.d), dtype=np.float32)
        if step:
            eps = np.random.default_rng([seed, wl.cfg_id, head, tensor_id, step]).standard_normal((wl.N, wl.d), dtype=np.float32)
        if tensor_id == 1 and wl.qk_align != 0.0:       # keys: aligned with the query centroids
            c = np.float32(wl.qk_align)
            mu = c * tables[0] + np.sqrt(np.float32(1.0) - c * c) * mu
        tables.append(mu)
        out.append(mu[cmap] + np.asarray(sig, dtype=np.float32) * eps)
    Q, K, V = out
    if wl.n_sink:
        # a few global "sink" keys: direction of the summed query centroids,
        # norm = mean + 3 std of the other keys' norms
        norms = np.linalg.norm(K[wl.n_sink:], axis=1)
        u = tables[0].sum(axis=0)
        u = u / np.linalg.norm(u)
        K[:wl.n_sink] = (norms.mean() + 3.0 * norms.std()) * u
    s = np.float32(wl.d ** -0.25)
    Q = Q * s
    K = K * s
    if wl.dtype == "bf16":
        Q, K, V = round_to_bf16(Q), round_to_bf16(K), round_to_bf16(V)
    return Q.astype(np.float32), K.astype(np.float32), V.astype(np.float32)
