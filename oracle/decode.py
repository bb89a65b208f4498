"""Decode step over an INT8 key/value cache -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

The definition written out in float64 numpy (App. C, "Additional Execution Interfaces": the cache
holds K8 and V8 with per-block scales; cached K8 takes part in the routed INT8 score path, cached V8
is used in the floating-point PV product with its block scale applied).  One new query token per
sequence attends to the first cache_len[b] cached keys:

  INT8-routed group:  s_j = delta_q * delta_K[blk(j)] * (q8 . k8_j) * scale      (exact integer dot)
  FP16-routed group:  s_j = (q . k16_j) * scale                                   (FP16 inputs, exact products)
  o = sum_j softmax(s)_j * delta_V[blk(j)] * v8_j

with q8, delta_q the blockwise quantiser of App. C applied to the single query row (block = the rows
that exist), h_k = h_q // (H_q / H_k), and bit g of the mask row of h_k routing the keys
[g*G*tile_n, (g+1)*G*tile_n).  Nothing here is shared with the CUDA path.
"""
from __future__ import annotations

import numpy as np

import oracle


def half_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bits.view(np.float16).astype(np.float64)


def quantize_query(q16: np.ndarray):
    """q16 uint16 [B, Hq, d] -> (q8 int8 [B, Hq, d], delta_q float32 [B, Hq]): one block per row."""
    B, H, d = q16.shape
    q8, s = oracle.quantize(np.ascontiguousarray(q16.reshape(B, H, 1, d)), 1)
    return q8.reshape(B, H, d), s.reshape(B, H)


def pack_row(route: np.ndarray) -> np.ndarray:
    """uint8 [..., T_mask] -> uint32 [..., W] with bit g of word g>>5 = route[g] != 0."""
    T = route.shape[-1]
    W = -(-T // 32)
    words = np.zeros(route.shape[:-1] + (W,), np.uint32)
    for g in range(T):
        words[..., g >> 5] |= (route[..., g] != 0).astype(np.uint32) << np.uint32(g & 31)
    return words


def decode(q16, k16, k8, k_scale, v8, v_scale, words, cache_len, tile_n, group, softmax_scale=0.0):
    """q16 uint16 [B,Hq,d]; k16 uint16 [B,Hk,Lmax,d]; k8, v8 int8 [B,Hk,Lmax,d];
    k_scale, v_scale float32 [B,Hk,ceil(Lmax/tile_n)]; words uint32 [nb,Hk,W]; cache_len int [B].
    Returns (out float64 [B,Hq,d], lse float64 [B,Hq])."""
    B, Hq, d = q16.shape
    Hk, Lmax = k8.shape[1], k8.shape[2]
    rep = Hq // Hk
    scale = softmax_scale if softmax_scale > 0 else 1.0 / np.sqrt(d)
    q = half_bits_to_f64(q16)
    q8, dq = quantize_query(q16)
    out = np.zeros((B, Hq, d))
    lse = np.full((B, Hq), -np.inf)
    for b in range(B):
        L = int(cache_len[b])
        if L == 0:
            continue
        j = np.arange(L)
        blk = j // tile_n
        grp = j // (tile_n * group)
        for hq in range(Hq):
            hk = hq // rep
            wrow = words[0 if words.shape[0] == 1 else b, hk]
            bit = ((wrow[grp >> 5] >> (grp & 31).astype(np.uint32)) & 1).astype(bool)
            dots8 = k8[b, hk, :L].astype(np.int64) @ q8[b, hq].astype(np.int64)
            s8 = float(dq[b, hq]) * k_scale[b, hk, blk].astype(np.float64) * dots8 * scale
            s16 = (half_bits_to_f64(k16[b, hk, :L]) @ q[b, hq]) * scale
            s = np.where(bit, s8, s16)
            m = s.max()
            p = np.exp(s - m)
            z = p.sum()
            v = v8[b, hk, :L].astype(np.float64) * v_scale[b, hk, blk].astype(np.float64)[:, None]
            out[b, hq] = (p[:, None] * v).sum(0) / z
            lse[b, hq] = m + np.log(z)
    return out, lse
