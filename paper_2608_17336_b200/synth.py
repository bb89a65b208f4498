"""Seeded synthetic inputs for the TileMix hot path: Q/K/V tensors and routing maps R.

This module serves both the CPU oracle's tests and the CUDA path's tests/bench, so it holds
only input *generation*: random values, outlier injection and the routing-template draws
(the policy layer that sits above the hot path).  None of the method's arithmetic
(quantisation, packing, scores, softmax) lives here, and it imports neither the oracle nor
the CUDA binding.

Values come from ``torch.Generator(device="cpu")``; routing draws come from a counter-based
hash u(seed, head, m, g) so that a map does not depend on iteration order.

The five workloads are synthetic stand-ins with LLaMA/Qwen-like head geometry for the LLM
prefill activations the paper evaluates on (no dataset or trained weight is used).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace

import numpy as np
import torch

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def splitmix64(x: np.ndarray) -> np.ndarray:
    """Vectorised SplitMix64 finaliser on uint64 counters."""
    with np.errstate(over="ignore"):
        z = (x.astype(np.uint64) + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return z ^ (z >> np.uint64(31))


def hash_uniform(seed: int, h, m, g) -> np.ndarray:
    """u(seed, h, m, g) in [0, 1): counter = seed*2^60 ^ h*2^40 ^ m*2^20 ^ g, hashed twice."""
    h = np.asarray(h, np.uint64); m = np.asarray(m, np.uint64); g = np.asarray(g, np.uint64)
    with np.errstate(over="ignore"):
        ctr = (np.uint64(seed) << np.uint64(60)) ^ (h << np.uint64(40)) ^ (m << np.uint64(20)) ^ g
    z = splitmix64(splitmix64(ctr))
    return (z >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


@dataclass(frozen=True)
class Workload:
    """One synthetic workload (shape + value recipe + routing recipe)."""
    name: str
    batch: int
    heads: int
    seqlen: int
    head_dim: int
    tile: int               # square score tile: tile_m = tile_n = tile
    group: int              # G adjacent key tiles per routing bit
    seed: int
    values: str = "normal"  # "normal" | "outlier_channels" | "student_t_k"
    routing: str = "bernoulli"  # "bernoulli" | "row_exact" | "band_per_head" | "zero" | "one"
    int8_fraction: float = 0.5
    pin_diagonal: bool = False
    band_tokens: int = 1024
    mask_batch: int = 1
    extras: dict = field(default_factory=dict)

    @property
    def T_m(self): return -(-self.seqlen // self.tile)
    @property
    def T_mask(self): return -(-self.seqlen // (self.group * self.tile))
    @property
    def W(self): return -(-self.T_mask // 32)

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations the hot path is tested and measured on.
WORKLOADS = {
    "cfg1_tiny": Workload("cfg1_tiny", 1, 1, 1024, 64, 64, 1, seed=0, routing="bernoulli",
                          int8_fraction=0.5),
    "cfg2_llama8k": Workload("cfg2_llama8k", 1, 32, 8192, 128, 128, 1, seed=2,
                             values="outlier_channels", routing="row_exact", int8_fraction=0.5),
    "cfg3_long32k": Workload("cfg3_long32k", 1, 32, 32768, 128, 128, 4, seed=3,
                             routing="row_exact", int8_fraction=0.75, pin_diagonal=True),
    "cfg4_batched4k": Workload("cfg4_batched4k", 8, 32, 4096, 128, 128, 2, seed=4,
                               routing="band_per_head", band_tokens=1024),
    "cfg5_verylong128k": Workload("cfg5_verylong128k", 1, 8, 131072, 128, 128, 8, seed=5,
                                  values="student_t_k", routing="bernoulli", int8_fraction=0.9),
}


def make_qkv(w: Workload):
    """FP16 Q, K, V [B, H, L, d] on the CPU (contiguous), drawn as float32 then cast."""
    gen = torch.Generator(device="cpu").manual_seed(w.seed)
    shape = (w.batch, w.heads, w.seqlen, w.head_dim)
    q = torch.randn(shape, generator=gen, dtype=torch.float32)
    k = torch.randn(shape, generator=gen, dtype=torch.float32)
    v = torch.randn(shape, generator=gen, dtype=torch.float32)
    if w.values == "outlier_channels":
        # 4 hash-chosen channels per head, the same set for Q and K of that head, scaled x8.
        for h in range(w.heads):
            u = hash_uniform(w.seed + 101, h, 0, np.arange(w.head_dim))
            ch = torch.from_numpy(np.argsort(u, kind="stable")[:4].copy())
            q[:, h, :, ch] *= 8.0
            k[:, h, :, ch] *= 8.0
    elif w.values == "student_t_k":
        # K ~ Student-t(3) elementwise: z / sqrt(chi2_3 / 3), no rescale.
        chi = torch.zeros(shape, dtype=torch.float32)
        for _ in range(3):
            chi += torch.randn(shape, generator=gen, dtype=torch.float32) ** 2
        k = k / torch.sqrt(chi / 3.0)
        del chi
    elif w.values != "normal":
        raise ValueError(w.values)
    return q.half().contiguous(), k.half().contiguous(), v.half().contiguous()


def legal_group_count(w: Workload) -> np.ndarray:
    """Number of key-tile groups that reach below the causal diagonal, per query-tile row.
    (Geometry of the causal triangle only; used to draw coverage-matched templates.)"""
    m = np.arange(w.T_m)
    last_row = np.minimum((m + 1) * w.tile, w.seqlen) - 1
    return np.minimum(last_row // (w.group * w.tile) + 1, w.T_mask)


def make_route(w: Workload) -> np.ndarray:
    """Routing map R (1 = INT8, 0 = FP16) as uint8 [mask_batch, H, T_m, T_mask].

    Entries of groups above the diagonal are drawn like any other (they are don't-care for
    the method; the packer canonicalises them)."""
    nb, H, T_m, T_mask = w.mask_batch, w.heads, w.T_m, w.T_mask
    hh, mm, gg = np.meshgrid(np.arange(H), np.arange(T_m), np.arange(T_mask), indexing="ij")
    out = np.zeros((nb, H, T_m, T_mask), np.uint8)
    for b in range(nb):
        u = hash_uniform(w.seed * 8 + b, hh, mm, gg)
        if w.routing == "zero":
            r = np.zeros_like(u, dtype=bool)
        elif w.routing == "one":
            r = np.ones_like(u, dtype=bool)
        elif w.routing == "bernoulli":
            r = u < w.int8_fraction
        elif w.routing == "row_exact":
            # Row-random template: per row keep k_m = round((1-rho)*|G_m|) groups FP16,
            # the ones with the smallest u among that row's eligible groups.  With the
            # diagonal pinned the pinned group is FP16 already and counts toward k_m.
            n_legal = legal_group_count(w)                       # [T_m]
            eligible = gg < n_legal[None, :, None]
            if w.pin_diagonal:
                eligible &= gg < (n_legal[None, :, None] - 1)
            k_fp16 = np.rint((1.0 - w.int8_fraction) * n_legal).astype(np.int64)
            if w.pin_diagonal:
                k_fp16 = np.maximum(k_fp16 - 1, 0)
            uu = np.where(eligible, u, 2.0)
            rank = np.argsort(np.argsort(uu, axis=-1, kind="stable"), axis=-1, kind="stable")
            r = eligible & (rank >= k_fp16[None, :, None])
        elif w.routing == "band_per_head":
            # FP16 within `band_tokens` of the diagonal; beyond it INT8 with a per-head
            # probability p_h drawn uniformly from [0, 1].
            p_h = hash_uniform(w.seed * 8 + b + 1000, np.arange(H), 0, 0)
            first_q = mm * w.tile
            last_k = np.minimum((gg + 1) * w.group * w.tile, w.seqlen) - 1
            in_band = (first_q - last_k) < w.band_tokens
            r = (~in_band) & (u < p_h[:, None, None])
        else:
            raise ValueError(w.routing)
        out[b] = r.astype(np.uint8)
    return out


def sample_rows(w: Workload, n_random_tiles: int = 2, n_random_rows: int = 64, heads=None):
    """(b, h, i) rows checked against the oracle at sizes where it cannot do every row:
    per head the first and last query tile, `n_random_tiles` hash-chosen whole tiles and
    `n_random_rows` hash-chosen single rows.  Returns int64 [n, 3]."""
    rows = []
    heads = range(w.heads) if heads is None else heads
    for b in range(w.batch):
        for h in heads:
            tiles = {0, w.T_m - 1}
            u = hash_uniform(w.seed + 7, h, b, np.arange(n_random_tiles))
            tiles |= {int(x) for x in (u * w.T_m).astype(np.int64)}
            idx = set()
            for t in tiles:
                idx |= set(range(t * w.tile, min((t + 1) * w.tile, w.seqlen)))
            u = hash_uniform(w.seed + 9, h, b, np.arange(n_random_rows))
            idx |= {int(x) for x in (u * w.seqlen).astype(np.int64)}
            rows += [(b, h, i) for i in sorted(idx)]
    return np.asarray(rows, np.int64).reshape(-1, 3)
