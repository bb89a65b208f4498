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
[g*G*tile_n, (g+1)*G*tile_n).  `chunk_v8` is the same cache read by the last L_q tokens of a context (chunked
prefill: causal alignment, blockwise Q8 as in the prefill oracle).  Both functions are pinned by
tests/test_oracle_decode_pins.py (a library attention routine, the prefill oracle, each other, plain loops).
Nothing here is shared with the CUDA path.
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


def chunk_v8(q16, q8, q_scale, k16, k8, k_scale, v8, v_scale, words, tile, group, blk_q=0, blk_k=0,
             softmax_scale=0.0):
    """Chunked prefill against an INT8 value cache (App. C, "Additional Execution Interfaces"; Sec. 3.1 softmax;
    App. C score formulas), the definition written out: the queries are the LAST L_q tokens of a context of L_k
    tokens, query i sits at context position c = L_k - L_q + i and attends to the keys j <= c;

      INT8-routed group:  s_ij = delta_q[blk_q(i)] * delta_K[blk_k(j)] * (q8_i . k8_j) * scale
      FP16-routed group:  s_ij = (q_i . k16_j) * scale
      o_i = sum_j softmax(s_i)_j * delta_V[j // tile] * v8_j

    where bit g of the mask row of (h_k, query tile c // tile) routes the keys [g*G*tile, (g+1)*G*tile).
    q16 uint16 / q8 int8 [B,Hq,Lq,d]; q_scale float32 [B,Hq,ceil(Lq/blk_q)]; k16 uint16 / k8, v8 int8 [B,Hk,Lk,d];
    k_scale float32 [B,Hk,ceil(Lk/blk_k)]; v_scale float32 [B,Hk,ceil(Lk/tile)]; words uint32 [nb,Hk,ceil(Lk/tile),W]
    (the words of the whole context).  Returns (out float64 [B,Hq,Lq,d], lse float64 [B,Hq,Lq])."""
    B, Hq, Lq, d = q16.shape
    Hk, Lk = k8.shape[1], k8.shape[2]
    rep = Hq // Hk
    blk_q = blk_q or tile
    blk_k = blk_k or tile
    off = Lk - Lq
    scale = softmax_scale if softmax_scale > 0 else 1.0 / np.sqrt(d)
    q = half_bits_to_f64(q16)
    j = np.arange(Lk)
    grp = j // (tile * group)
    out = np.zeros((B, Hq, Lq, d))
    lse = np.zeros((B, Hq, Lq))
    for b in range(B):
        for hq in range(Hq):
            hk = hq // rep
            k = half_bits_to_f64(k16[b, hk])
            v = v8[b, hk].astype(np.float64) * v_scale[b, hk, j // tile].astype(np.float64)[:, None]
            dots8 = q8[b, hq].astype(np.int64) @ k8[b, hk].astype(np.int64).T                      # [Lq, Lk], exact
            dq = q_scale[b, hq, np.arange(Lq) // blk_q].astype(np.float64)[:, None]
            dk = k_scale[b, hk, j // blk_k].astype(np.float64)[None, :]
            s8 = dq * dk * dots8 * scale
            s16 = (q[b, hq] @ k.T) * scale
            for i in range(Lq):
                c = off + i
                wrow = words[0 if words.shape[0] == 1 else b, hk, c // tile]
                bit = ((wrow[grp[:c + 1] >> 5] >> (grp[:c + 1] & 31).astype(np.uint32)) & 1).astype(bool)
                s = np.where(bit, s8[i, :c + 1], s16[i, :c + 1])
                m = s.max()
                p = np.exp(s - m)
                z = p.sum()
                out[b, hq, i] = (p[:, None] * v[:c + 1]).sum(0) / z
                lse[b, hq, i] = m + np.log(z)
    return out, lse
