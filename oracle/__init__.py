"""TileMix CPU oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes wrappers over ``tilemix_oracle.c`` (plain C, fp64 / exact int32 / FP32 where the
paper fixes it) plus two closed forms the paper prints.  Only the tests, the smoke check and
the bench's CPU-baseline leg may import this package; the CUDA product path never does, and
nothing here imports the product package.

Every array is a dense numpy array:
  q16/k16/v16  uint16 (binary16 bit patterns) [B, H, L, d];  q8/k8 int8 [B, H, L, d]
  q_scale float32 [B, Hq, ceil(L/blk_q)];  k_scale float32 [B, Hk, ceil(L/blk_k)]
  route uint8 [nb, Hk, T_m, T_mask];  words uint32 [nb, Hk, T_m, W]
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tilemix_oracle.c")
_LIB = os.path.join(_HERE, "libtilemix_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class _Problem(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "batch", "heads_q", "heads_kv", "seqlen", "head_dim", "tile_m", "tile_n", "group",
        "blk_q", "blk_k", "mask_batch")] + [("softmax_scale", ctypes.c_double)]


@dataclass
class Problem:
    """Shape of one attention call (paper notation: B, H_q, H_k, L, d, BLOCK_M x BLOCK_N, g)."""
    batch: int
    heads_q: int
    heads_kv: int
    seqlen: int
    head_dim: int
    tile_m: int
    tile_n: int
    group: int = 1
    blk_q: int = 0          # 0 -> tile_m
    blk_k: int = 0          # 0 -> tile_n
    mask_batch: int = 1
    softmax_scale: float = 0.0

    @property
    def T_m(self): return -(-self.seqlen // self.tile_m)
    @property
    def T_n(self): return -(-self.seqlen // self.tile_n)
    @property
    def T_mask(self): return -(-self.seqlen // (self.group * self.tile_n))
    @property
    def W(self): return -(-self.T_mask // 32)
    @property
    def bq(self): return self.blk_q or self.tile_m
    @property
    def bk(self): return self.blk_k or self.tile_n

    def _c(self) -> _Problem:
        return _Problem(self.batch, self.heads_q, self.heads_kv, self.seqlen, self.head_dim,
                        self.tile_m, self.tile_n, self.group, self.bq, self.bk, self.mask_batch,
                        float(self.softmax_scale))


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_init()
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _chk(a, dtype, shape=None):
    assert isinstance(a, np.ndarray) and a.dtype == np.dtype(dtype), (a.dtype, dtype)
    assert a.flags["C_CONTIGUOUS"]
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def quantize(x16: np.ndarray, blk: int):
    """Blockwise symmetric INT8 (App. C): returns (int8 like x16, float32 scales [..., ceil(L/blk)])."""
    _chk(x16, np.uint16)
    *lead, L, d = x16.shape
    n_heads = int(np.prod(lead)) if lead else 1
    out = np.empty(x16.shape, np.int8)
    scale = np.empty(tuple(lead) + (-(-L // blk),), np.float32)
    _load().oracle_quantize(_ptr(x16), ctypes.c_int64(n_heads), ctypes.c_int32(L),
                            ctypes.c_int32(d), ctypes.c_int32(blk), _ptr(out), _ptr(scale))
    return out, scale


def pack(p: Problem, route: np.ndarray, pin_diagonal: bool = False):
    """Packed routing words (Sec. 4.2) and the coverage counters (App. B)."""
    _chk(route, np.uint8, (p.mask_batch, p.heads_kv, p.T_m, p.T_mask))
    words = np.empty((p.mask_batch, p.heads_kv, p.T_m, p.W), np.uint32)
    counts = np.empty((p.mask_batch, p.heads_kv, 2), np.uint64)
    c = p._c()
    _load().oracle_pack(ctypes.byref(c), _ptr(route), ctypes.c_int32(int(pin_diagonal)),
                        _ptr(words), _ptr(counts))
    return words, counts


def attention_rows(p: Problem, q16, k16, v16, q8, k8, q_scale, k_scale, words, rows):
    """Outputs for the listed (b, h_q, i) rows: (out float64 [n, d], lse [n], row_sum [n])."""
    B, Hq, Hk, L, d = p.batch, p.heads_q, p.heads_kv, p.seqlen, p.head_dim
    _chk(q16, np.uint16, (B, Hq, L, d)); _chk(k16, np.uint16, (B, Hk, L, d))
    _chk(v16, np.uint16, (B, Hk, L, d))
    if q8 is not None:
        _chk(q8, np.int8, (B, Hq, L, d)); _chk(k8, np.int8, (B, Hk, L, d))
        _chk(q_scale, np.float32, (B, Hq, -(-L // p.bq)))
        _chk(k_scale, np.float32, (B, Hk, -(-L // p.bk)))
    else:
        assert not words.any(), "INT8-routed groups need the quantised operands"
    _chk(words, np.uint32, (p.mask_batch, Hk, p.T_m, p.W))
    rows = np.ascontiguousarray(np.asarray(rows, np.int64).reshape(-1, 3))
    assert (rows[:, 0] < B).all() and (rows[:, 1] < Hq).all() and (rows[:, 2] < L).all()
    assert (rows >= 0).all()
    n = rows.shape[0]
    out = np.empty((n, d), np.float64)
    lse = np.empty((n,), np.float64)
    rsum = np.empty((n,), np.float64)
    c = p._c()
    _load().oracle_attention_rows(ctypes.byref(c), _ptr(q16), _ptr(k16), _ptr(v16), _ptr(q8),
                                  _ptr(k8), _ptr(q_scale), _ptr(k_scale), _ptr(words),
                                  ctypes.c_int64(n), _ptr(rows), _ptr(out), _ptr(lse), _ptr(rsum))
    return out, lse, rsum


def attention_full(p: Problem, q16, k16, v16, q8, k8, q_scale, k_scale, words):
    """All rows: out float64 [B, Hq, L, d], lse [B, Hq, L]."""
    B, Hq, L = p.batch, p.heads_q, p.seqlen
    bb, hh, ii = np.meshgrid(np.arange(B), np.arange(Hq), np.arange(L), indexing="ij")
    rows = np.stack([bb.ravel(), hh.ravel(), ii.ravel()], axis=1)
    out, lse, rsum = attention_rows(p, q16, k16, v16, q8, k8, q_scale, k_scale, words, rows)
    return (out.reshape(B, Hq, L, p.head_dim), lse.reshape(B, Hq, L), rsum.reshape(B, Hq, L))


def int32_tile(p: Problem, q8, k8, b, hq, m, n):
    """Raw INT32 accumulator tile Q8_m K8_n^T (App. C), unmasked, zero beyond the sequence."""
    _chk(q8, np.int8); _chk(k8, np.int8)
    out = np.empty((p.tile_m, p.tile_n), np.int32)
    c = p._c()
    _load().oracle_int32_tile(ctypes.byref(c), _ptr(q8), _ptr(k8), ctypes.c_int64(b),
                              ctypes.c_int64(hq), ctypes.c_int64(m), ctypes.c_int64(n), _ptr(out))
    return out


def fp_tile(p: Problem, q16, k16, b, hq, m, n):
    """Raw FP16-route tile Q_m K_n^T in float64 (before 1/sqrt(d)), unmasked."""
    _chk(q16, np.uint16); _chk(k16, np.uint16)
    out = np.empty((p.tile_m, p.tile_n), np.float64)
    c = p._c()
    _load().oracle_fp_tile(ctypes.byref(c), _ptr(q16), _ptr(k16), ctypes.c_int64(b),
                           ctypes.c_int64(hq), ctypes.c_int64(m), ctypes.c_int64(n), _ptr(out))
    return out


# ---------------------------------------------------------------------------------------
# Closed forms the paper prints (used as pins and by tests of the host-side helpers).
# ---------------------------------------------------------------------------------------

def grouping_rule(L_k: int, block_n: int):
    """App. B "Policy Construction and Sharing": b64 = ceil(L_k/64),
    BLOCK_N^mask = BLOCK_N * ceil(max(b64, BLOCK_N) / BLOCK_N); returns (g, T_mask)."""
    b64 = -(-L_k // 64)
    block_mask = block_n * (-(-max(b64, block_n) // block_n))
    g = block_mask // block_n
    return g, -(-L_k // block_mask)


def resident_bytes_quantize_once(Hq, Hk, L, d, blk_q, blk_k, tile_m, scale_bytes=2, word_bytes=8):
    """App. D memory accounting, quantize-once row: FP16 Q/K/V + INT8 Q/K + one scale per
    (block, head) in the operand dtype + one packed 64-bit word per (h_k, m).  Bytes."""
    fp16 = 2 * d * L * (Hq + 2 * Hk)
    int8 = d * L * (Hq + Hk)
    scales = scale_bytes * (Hq * (-(-L // blk_q)) + Hk * (-(-L // blk_k)))
    words = word_bytes * Hk * (-(-L // tile_m))
    return fp16 + int8 + scales + words, fp16
