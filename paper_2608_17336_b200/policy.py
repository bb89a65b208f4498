"""Static, data-free routing templates (the paper's precision layouts, App. B "Precision Layouts")
and the host-side policy plumbing around them: automatic grouping factor, coverage accounting,
coverage matching and a template cache.

A template is a uint8 array R[m, g] over query-tile rows m and key-tile groups g (1 = INT8,
0 = FP16); entries of illegal groups are 0.  `broadcast()` turns it into the [nb, H_k, T_m, T_mask]
map that tilemix_pack_routing_mask takes (the paper shares one template over layers, batch and KV
heads).  Pure numpy, no GPU.
"""
from __future__ import annotations

from dataclasses import dataclass
from functools import lru_cache

import numpy as np


@dataclass(frozen=True)
class Geometry:
    """Tile geometry of one sequence length (paper notation BLOCK_M, BLOCK_N, g)."""
    seqlen: int
    tile_m: int
    tile_n: int
    group: int

    @property
    def T_m(self): return -(-self.seqlen // self.tile_m)
    @property
    def T_n(self): return -(-self.seqlen // self.tile_n)
    @property
    def block_mask(self): return self.group * self.tile_n          # BLOCK_N^mask
    @property
    def T_mask(self): return -(-self.seqlen // self.block_mask)


def grouping_rule(seqlen_k: int, tile_n: int) -> int:
    """Automatic grouping factor g so that one 64-bit word covers a row (App. B "Policy Construction
    and Sharing"): b64 = ceil(L_k/64), BLOCK_N^mask = BLOCK_N * ceil(max(b64, BLOCK_N)/BLOCK_N)."""
    b64 = -(-seqlen_k // 64)
    return -(-max(b64, tile_n) // tile_n)


def auto_geometry(seqlen: int, tile_m: int, tile_n: int) -> Geometry:
    return Geometry(seqlen, tile_m, tile_n, grouping_rule(seqlen, tile_n))


def legal_groups(geo: Geometry) -> np.ndarray:
    """bool [T_m, T_mask]: group g holds at least one causal (query, key) pair of tile row m."""
    m = np.arange(geo.T_m)[:, None]
    g = np.arange(geo.T_mask)[None, :]
    last_row = np.minimum((m + 1) * geo.tile_m, geo.seqlen) - 1
    return g * geo.block_mask <= last_row


def coverage(geo: Geometry, R: np.ndarray) -> float:
    """Realised INT8 coverage: INT8-routed legal groups / legal groups (App. B "Coverage Accounting")."""
    legal = legal_groups(geo)
    return float(R[legal].sum() / max(int(legal.sum()), 1))


def _from_fp16_set(geo: Geometry, fp16: np.ndarray) -> np.ndarray:
    legal = legal_groups(geo)
    return (legal & ~fp16).astype(np.uint8)


# ----------------------------------------------------------------------------------------- layouts

def one(geo: Geometry) -> np.ndarray:
    """All legal groups INT8."""
    return legal_groups(geo).astype(np.uint8)


def zero(geo: Geometry) -> np.ndarray:
    """All legal groups FP16 (the kernel's full-precision reference)."""
    return np.zeros((geo.T_m, geo.T_mask), np.uint8)


def _gamma(geo: Geometry) -> np.ndarray:
    return (np.arange(geo.T_m) * geo.tile_m) // geo.block_mask      # group aligned with the start of row m


def band_fp16(geo: Geometry, w: int) -> np.ndarray:
    g = np.arange(geo.T_mask)[None, :]
    return np.abs(g - _gamma(geo)[:, None]) <= w


def band(geo: Geometry, w: int) -> np.ndarray:
    """FP16 within half-width w (in groups) of the diagonal group gamma(m), INT8 elsewhere."""
    return _from_fp16_set(geo, band_fp16(geo, w))


def global_fp16(geo: Geometry, n_global: int) -> np.ndarray:
    g = np.arange(geo.T_mask)[None, :]
    return np.broadcast_to(g < n_global, (geo.T_m, geo.T_mask)).copy()


def global_(geo: Geometry, n_global: int) -> np.ndarray:
    """The first n_global key-tile groups (the designated global positions) stay FP16 for every row."""
    return _from_fp16_set(geo, global_fp16(geo, n_global))


def row_random_fp16(geo: Geometry, rho_int8: float, seed: int) -> np.ndarray:
    legal = legal_groups(geo)
    rng = np.random.default_rng(seed)
    u = rng.random((geo.T_m, geo.T_mask))
    u = np.where(legal, u, 2.0)
    k_m = np.rint((1.0 - rho_int8) * legal.sum(1)).astype(np.int64)
    rank = np.argsort(np.argsort(u, axis=1, kind="stable"), axis=1, kind="stable")
    return legal & (rank < k_m[:, None])


def row_random(geo: Geometry, rho_int8: float, seed: int = 0) -> np.ndarray:
    """Per row, k_m = round((1 - rho)|G_m|) legal groups drawn uniformly without replacement stay FP16."""
    return _from_fp16_set(geo, row_random_fp16(geo, rho_int8, seed))


def aligned_sparse(geo: Geometry, alpha: float, beta: float) -> np.ndarray:
    """A right-aligned FP16 region of a(m) = min(|G_m|, ceil(alpha + beta*m)) groups per row."""
    legal = legal_groups(geo)
    n_legal = legal.sum(1)
    a = np.minimum(n_legal, np.ceil(alpha + beta * np.arange(geo.T_m)).astype(np.int64))
    g = np.arange(geo.T_mask)[None, :]
    g_max = n_legal - 1
    return _from_fp16_set(geo, g >= (g_max - a + 1)[:, None])


def bigbird(geo: Geometry, w: int, n_global: int, rho_random: float, seed: int = 0) -> np.ndarray:
    """Union of a local band, global groups and a row-random component, all kept FP16."""
    fp16 = band_fp16(geo, w) | global_fp16(geo, n_global) | row_random_fp16(geo, rho_random, seed)
    return _from_fp16_set(geo, fp16)


def sptrans(geo: Geometry, stride: int, tail: int) -> np.ndarray:
    """Sparse-Transformer pattern: for query i the FP16 keys are its own stride [u*s, i] and the last
    `tail` positions of every earlier stride; a group is FP16 for row m if any query of the row
    selects any key of the group."""
    fp16 = np.zeros((geo.T_m, geo.T_mask), bool)
    gk = geo.block_mask
    for m in range(geo.T_m):
        i0, i1 = m * geo.tile_m, min((m + 1) * geo.tile_m, geo.seqlen) - 1
        # own strides of the row's queries: keys [u(i0)*s, i1]
        lo = (i0 // stride) * stride
        fp16[m, lo // gk:i1 // gk + 1] = True
        # tails of the strides that precede some query of the row
        for r in range(i1 // stride):
            a, b = max(r * stride, (r + 1) * stride - tail), (r + 1) * stride - 1
            if a <= b:
                fp16[m, a // gk:b // gk + 1] = True
    return _from_fp16_set(geo, fp16)


# ----------------------------------------------------------------------------------------- matching

def match_coverage(geo: Geometry, layout: str, target: float, seed: int = 0) -> tuple[np.ndarray, dict]:
    """Picks the layout's free parameter so that the realised coverage is as close as possible to
    `target` (the paper's 25 / 50 / 75 % settings are matched at tile-group granularity)."""
    cands: list[tuple[np.ndarray, dict]] = []
    T = geo.T_mask
    if layout == "one":
        cands = [(one(geo), {})]
    elif layout == "zero":
        cands = [(zero(geo), {})]
    elif layout == "band":
        cands = [(band(geo, w), {"w": w}) for w in range(0, T + 1)]
    elif layout == "global":
        cands = [(global_(geo, n), {"n_global": n}) for n in range(0, T + 1)]
    elif layout == "row_random":
        cands = [(row_random(geo, target, seed), {"rho": target})]
    elif layout == "aligned_sparse":
        for alpha in (1.0, 2.0, 4.0):
            for beta in np.linspace(0.0, 1.0, 65):
                cands.append((aligned_sparse(geo, alpha, float(beta)), {"alpha": alpha, "beta": float(beta)}))
    elif layout == "bigbird":
        for w in range(0, max(1, T // 4) + 1):
            for n in range(0, max(1, T // 8) + 1):
                for rho_r in (1.0, 0.95, 0.9, 0.8, 0.7, 0.6, 0.5, 0.4):
                    cands.append((bigbird(geo, w, n, rho_r, seed), {"w": w, "n_global": n, "rho_random": rho_r}))
    elif layout == "sptrans":
        for s_groups in range(1, T + 1):
            stride = s_groups * geo.block_mask
            for tail in (geo.block_mask, 2 * geo.block_mask, stride // 2):
                if 0 < tail <= stride:
                    cands.append((sptrans(geo, stride, tail), {"stride": stride, "tail": tail}))
    else:
        raise ValueError(layout)
    best = min(cands, key=lambda c: abs(coverage(geo, c[0]) - target))
    return best[0], dict(best[1], coverage=coverage(geo, best[0]))


@lru_cache(maxsize=64)
def _cached(seqlen, tile_m, tile_n, group, layout, target, seed):
    R, info = match_coverage(Geometry(seqlen, tile_m, tile_n, group), layout, target, seed)
    R.setflags(write=False)
    return R, tuple(sorted(info.items()))


def template(seqlen: int, tile_m: int, tile_n: int, layout: str, target: float, group: int | None = None,
             seed: int = 0):
    """Cached template for (sequence length, geometry, layout, coverage): regenerated only when one of
    them changes.  `group=None` applies the automatic grouping rule.  Returns (Geometry, R, info)."""
    g = grouping_rule(seqlen, tile_n) if group is None else group
    R, info = _cached(seqlen, tile_m, tile_n, g, layout, float(target), seed)
    return Geometry(seqlen, tile_m, tile_n, g), R, dict(info)


def broadcast(R: np.ndarray, heads_kv: int, mask_batch: int = 1) -> np.ndarray:
    """One template for every KV head (and batch entry): uint8 [nb, H_k, T_m, T_mask], contiguous."""
    return np.ascontiguousarray(np.broadcast_to(R[None, None], (mask_batch, heads_kv) + R.shape))
