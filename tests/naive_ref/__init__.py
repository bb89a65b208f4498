"""Naive CUDA reference of the hot path -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

ctypes wrapper over ``naive_attention.cu`` (one warp per query row, FP32 CUDA-core arithmetic, __dp4a for the
INT8 dot products, no tensor cores).  It is the middle rung of the parity ladder: checked against the CPU oracle,
then used to check every row of the fused kernel at sizes the oracle cannot cover.  Nothing of the product
imports it and it imports nothing of the product.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "naive_attention.cu")
_LIB = os.path.join(_HERE, "libnaive_ref.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        nvcc = "/usr/local/cuda/bin/nvcc" if os.path.exists("/usr/local/cuda/bin/nvcc") else "nvcc"
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-std=c++17", "-O3", "-lineinfo", "-shared",
                        "-Xcompiler", "-fPIC", "-o", _LIB, _SRC], check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(t):
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def quantize(x: torch.Tensor, blk: int):
    """x: CUDA FP16 [..., L, d] contiguous -> (int8 like x, float32 scales [..., ceil(L/blk)])."""
    assert x.is_cuda and x.dtype == torch.float16 and x.is_contiguous()
    *lead, L, d = x.shape
    n_heads = int(math.prod(lead)) if lead else 1
    out = torch.empty(x.shape, dtype=torch.int8, device=x.device)
    scale = torch.empty(tuple(lead) + (-(-L // blk),), dtype=torch.float32, device=x.device)
    rc = _load().naive_quantize(_p(x), ctypes.c_int64(n_heads), L, d, blk, _p(out), _p(scale), _stream())
    assert rc == 0, rc
    return out, scale


def attention(q, k, v, route, tile: int, group: int, pin_diagonal: bool = False, blk_q: int = 0, blk_k: int = 0,
              softmax_scale: float = 0.0, want_lse: bool = False):
    """q [B,Hq,L,d], k/v [B,Hk,L,d] CUDA FP16 contiguous; route: CUDA uint8 [nb,Hk,T_m,T_mask] (non-zero = INT8).
    Quantises Q and K itself.  Returns dict(out FP32 [B,Hq,L,d], lse, q8, k8, qs, ks)."""
    B, Hq, L, d = q.shape
    Hk = k.shape[1]
    for t in (q, k, v, route):
        assert t.is_cuda and t.is_contiguous()
    blk_q, blk_k = blk_q or tile, blk_k or tile
    q8, qs = quantize(q, blk_q)
    k8, ks = quantize(k, blk_k)
    out = torch.empty((B, Hq, L, d), dtype=torch.float32, device=q.device)
    lse = torch.empty((B, Hq, L), dtype=torch.float32, device=q.device) if want_lse else None
    scale = softmax_scale if softmax_scale > 0 else 1.0 / math.sqrt(d)
    rc = _load().naive_attention(_p(q), _p(k), _p(v), _p(q8), _p(k8), _p(qs), _p(ks), _p(route), B, Hq, Hk, L, d, tile,
                                 group, blk_q, blk_k, route.shape[0], int(bool(pin_diagonal)), ctypes.c_float(scale),
                                 _p(out), _p(lse), _stream())
    assert rc == 0, rc
    return dict(out=out, lse=lse, q8=q8, k8=k8, qs=qs, ks=ks)
