"""ctypes binding over libtilemix.so: same names as the C ABI (include/tilemix.h), argument
marshalling only.  torch supplies device memory and the current stream; every step of the
path runs in the library's kernels.  There is no fallback: a missing library raises."""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtilemix.so")

OK = 0
ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGN, ERR_WORKSPACE, ERR_DEVICE_TIMEOUT = -1, -2, -3, -4, -5, -6
FORCE_FP16 = 1
QUANT_ON_THE_FLY = 2   # flags: INT8 tiles and scales are made inside the attention kernel
PIN_DIAGONAL_FP16 = 1

EXPORTS = (
    "tilemix_quantize_qk", "tilemix_pack_routing_mask", "tilemix_attention_fwd", "tilemix_attention_fwd_noalloc",
    "tilemix_prefill_host",
    "tilemix_mask_words_per_row", "tilemix_workspace_size", "tilemix_scratch_bytes", "tilemix_arena_size",
    "tilemix_read_status", "tilemix_status_string", "tilemix_launch_count",
    "tilemix_varlen_counts", "tilemix_varlen_workspace_size", "tilemix_quantize_qk_varlen",
    "tilemix_pack_routing_mask_varlen", "tilemix_attention_fwd_varlen",
    "tilemix_decode_workspace_size", "tilemix_decode_int8kv", "tilemix_attention_fwd_chunk",
    "tilemix_chunk_v8_workspace_size", "tilemix_attention_fwd_chunk_v8",
    "tilemix_test_drop_copy", "tilemix_tensor_peak_probe",
)


class TilemixError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().tilemix_status_string(code).decode()
        super().__init__(f"{where} failed with {code}: {msg}")


class ProblemStruct(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("heads_q", ctypes.c_int32), ("heads_kv", ctypes.c_int32),
        ("seqlen", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("tile_m", ctypes.c_int32), ("tile_n", ctypes.c_int32), ("group", ctypes.c_int32),
        ("quant_blk_q", ctypes.c_int32), ("quant_blk_k", ctypes.c_int32),
        ("mask_batch", ctypes.c_int32), ("flags", ctypes.c_uint32),
        ("softmax_scale", ctypes.c_float), ("reserved", ctypes.c_int32),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
        ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
    ]

    @property
    def T_m(self): return -(-self.seqlen // self.tile_m)
    @property
    def T_n(self): return -(-self.seqlen // self.tile_n)
    @property
    def T_mask(self): return -(-self.seqlen // (self.group * self.tile_n))
    @property
    def W(self): return -(-self.T_mask // 32)
    @property
    def blk_q(self): return self.quant_blk_q or self.tile_m
    @property
    def blk_k(self): return self.quant_blk_k or self.tile_n


class DebugStruct(ctypes.Structure):
    _fields_ = [("tiles", ctypes.c_void_p), ("n_tiles", ctypes.c_int32), ("raw", ctypes.c_void_p),
                ("kind", ctypes.c_void_p)]


class VarlenStruct(ctypes.Structure):
    _fields_ = [("n_seqs", ctypes.c_int32), ("max_seqlen", ctypes.c_int32),
                ("cu_seqlens", ctypes.POINTER(ctypes.c_int32))]


class DecodeStruct(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("batch", "heads_q", "heads_kv", "head_dim", "max_len", "tile_n",
                                               "group", "mask_batch", "n_splits")] + [("softmax_scale", ctypes.c_float)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libtilemix.so (built by paper_2608_17336_b200.build); raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2608_17336_b200.build` "
                               "(there is no CPU or library fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32
        pp = ctypes.POINTER(ProblemStruct)
        L.tilemix_quantize_qk.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
        L.tilemix_pack_routing_mask.argtypes = [pp, vp, u32, vp, vp, vp]
        L.tilemix_attention_fwd.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t,
                                            ctypes.POINTER(DebugStruct), vp]
        L.tilemix_attention_fwd_chunk.argtypes = [pp, ctypes.c_int32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                  ctypes.c_size_t, ctypes.POINTER(DebugStruct), vp]
        L.tilemix_chunk_v8_workspace_size.argtypes = [pp, ctypes.c_int32]
        L.tilemix_chunk_v8_workspace_size.restype = ctypes.c_size_t
        L.tilemix_attention_fwd_chunk_v8.argtypes = [pp, ctypes.c_int32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                     ctypes.c_size_t, vp]
        L.tilemix_attention_fwd_noalloc.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                    ctypes.POINTER(DebugStruct), ctypes.POINTER(vp), vp]
        L.tilemix_prefill_host.argtypes = [pp, vp, vp, vp, vp, u32, vp, vp, ctypes.c_size_t, vp]
        L.tilemix_mask_words_per_row.argtypes = [i32, i32, i32]
        for name in ("tilemix_workspace_size", "tilemix_scratch_bytes", "tilemix_arena_size"):
            getattr(L, name).argtypes = [pp]
            getattr(L, name).restype = ctypes.c_size_t
        L.tilemix_read_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32 * 4), vp]
        L.tilemix_status_string.argtypes = [i32]
        L.tilemix_status_string.restype = ctypes.c_char_p
        L.tilemix_launch_count.restype = ctypes.c_uint64
        L.tilemix_test_drop_copy.argtypes = [i32, ctypes.c_uint64]
        L.tilemix_tensor_peak_probe.argtypes = [i32, i32, ctypes.POINTER(ctypes.c_int), vp, vp]
        dp = ctypes.POINTER(DecodeStruct)
        L.tilemix_decode_workspace_size.argtypes = [dp]
        L.tilemix_decode_workspace_size.restype = ctypes.c_size_t
        L.tilemix_decode_int8kv.argtypes = [dp] + [vp] * 12 + [vp, ctypes.c_size_t, vp]
        vlp = ctypes.POINTER(VarlenStruct)
        L.tilemix_varlen_counts.argtypes = [pp, vlp, ctypes.POINTER(ctypes.c_int64 * 7)]
        L.tilemix_varlen_workspace_size.argtypes = [pp, vlp]
        L.tilemix_varlen_workspace_size.restype = ctypes.c_size_t
        L.tilemix_quantize_qk_varlen.argtypes = [pp, vlp, vp, vp, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.tilemix_pack_routing_mask_varlen.argtypes = [pp, vlp, vp, u32, vp, vp, vp, ctypes.c_size_t, vp]
        L.tilemix_attention_fwd_varlen.argtypes = [pp, vlp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                                   ctypes.c_size_t, ctypes.POINTER(DebugStruct), vp]
        _lib = L
    return _lib


def problem(batch, heads_q, heads_kv, seqlen, head_dim, tile_m, tile_n, group=1, quant_blk_q=0,
            quant_blk_k=0, mask_batch=1, flags=0, softmax_scale=0.0) -> ProblemStruct:
    p = ProblemStruct()
    p.batch, p.heads_q, p.heads_kv, p.seqlen, p.head_dim = batch, heads_q, heads_kv, seqlen, head_dim
    p.tile_m, p.tile_n, p.group = tile_m, tile_n, group
    p.quant_blk_q, p.quant_blk_k, p.mask_batch = quant_blk_q, quant_blk_k, mask_batch
    p.flags, p.softmax_scale = flags, softmax_scale
    return p


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc, where):
    if rc != OK:
        raise TilemixError(rc, where)


def _strides(p_field, t, d):
    assert t.stride(-1) == 1 and t.shape[-1] == d, "head_dim axis must be contiguous"
    p_field[0], p_field[1], p_field[2] = t.stride(0), t.stride(1), t.stride(2)


def _with_strides(p: ProblemStruct, q=None, k=None, v=None, o=None) -> ProblemStruct:
    pp = ProblemStruct.from_buffer_copy(p)
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
        if t is not None:
            _strides(getattr(pp, name), t, p.head_dim)
    return pp


def tilemix_quantize_qk(p: ProblemStruct, q: torch.Tensor, k: torch.Tensor):
    """-> (q_i8, k_i8, q_scale, k_scale); q [B,Hq,L,d], k [B,Hk,L,d] FP16 CUDA tensors."""
    assert q.dtype == torch.float16 and k.dtype == torch.float16 and q.is_cuda and k.is_cuda
    q8 = torch.empty(q.shape, dtype=torch.int8, device=q.device)
    k8 = torch.empty(k.shape, dtype=torch.int8, device=k.device)
    qs = torch.empty((p.batch, p.heads_q, -(-p.seqlen // p.blk_q)), dtype=torch.float32, device=q.device)
    ks = torch.empty((p.batch, p.heads_kv, -(-p.seqlen // p.blk_k)), dtype=torch.float32, device=q.device)
    pp = _with_strides(p, q=q, k=k)
    _check(lib().tilemix_quantize_qk(ctypes.byref(pp), _ptr(q), _ptr(k), _ptr(q8), _ptr(k8), _ptr(qs), _ptr(ks),
                                     _stream()), "tilemix_quantize_qk")
    return q8, k8, qs, ks


def tilemix_pack_routing_mask(p: ProblemStruct, route: torch.Tensor, pin_diagonal: bool = False):
    """route uint8 [nb,Hk,T_m,T_mask] -> (words int32-typed uint32 bits [nb,Hk,T_m,W], counts int64 [nb,Hk,2])."""
    assert route.dtype == torch.uint8 and route.is_cuda and route.is_contiguous()
    assert tuple(route.shape) == (p.mask_batch, p.heads_kv, p.T_m, p.T_mask), route.shape
    words = torch.empty((p.mask_batch, p.heads_kv, p.T_m, p.W), dtype=torch.int32, device=route.device)
    counts = torch.empty((p.mask_batch, p.heads_kv, 2), dtype=torch.int64, device=route.device)
    _check(lib().tilemix_pack_routing_mask(ctypes.byref(p), _ptr(route), PIN_DIAGONAL_FP16 if pin_diagonal else 0,
                                           _ptr(words), _ptr(counts), _stream()), "tilemix_pack_routing_mask")
    return words, counts


def tilemix_attention_fwd(p: ProblemStruct, q, k, v, q8=None, k8=None, q_scale=None, k_scale=None, words=None,
                          out=None, want_lse=False, debug_tiles=None, workspace=None):
    """Fused forward.  Returns a dict: out [B,Hq,L,d] FP16, lse (if asked), raw/kind (if debug_tiles),
    workspace.  debug_tiles: int32 tensor/list [n,4] of (b, h_q, m, n)."""
    dev = q.device
    if out is None:
        out = torch.empty((p.batch, p.heads_q, p.seqlen, p.head_dim), dtype=torch.float16, device=dev)
    lse = torch.empty((p.batch, p.heads_q, p.seqlen), dtype=torch.float32, device=dev) if want_lse else None
    if workspace is None:
        workspace = torch.empty(lib().tilemix_workspace_size(ctypes.byref(p)), dtype=torch.uint8, device=dev)
    dbg, raw, kind, tiles = None, None, None, None
    if debug_tiles is not None:
        tiles = torch.as_tensor(debug_tiles, dtype=torch.int32).reshape(-1, 4).contiguous().to(dev)
        n = tiles.shape[0]
        raw = torch.zeros((n, p.tile_m, p.tile_n), dtype=torch.int32, device=dev)
        kind = torch.full((n,), 255, dtype=torch.uint8, device=dev)
        dbg = DebugStruct(tiles.data_ptr(), n, raw.data_ptr(), kind.data_ptr())
    pp = _with_strides(p, q=q, k=k, v=v, o=out)
    rc = lib().tilemix_attention_fwd(ctypes.byref(pp), _ptr(q), _ptr(k), _ptr(v), _ptr(q8), _ptr(k8), _ptr(q_scale),
                                     _ptr(k_scale), _ptr(words), _ptr(out), _ptr(lse), _ptr(workspace),
                                     workspace.numel(), ctypes.byref(dbg) if dbg is not None else None, _stream())
    _check(rc, "tilemix_attention_fwd")
    return {"out": out, "lse": lse, "raw": raw, "kind": kind, "workspace": workspace}


def tilemix_attention_fwd_noalloc(p: ProblemStruct, q, k, v, q8, k8, q_scale, k_scale, words, out, lse=None):
    """The fused forward for callers that cannot allocate device memory: every tensor, `out` included,
    is passed in, and the library's built-in 4096-byte workspace replaces the caller's.  Nothing is
    allocated here or in the library.  Returns the device address (int) of that workspace; pass it to
    tilemix_read_status_at to read the status record.  Calls on one device share the workspace, so do
    not let two of them overlap on the GPU."""
    pp = _with_strides(p, q=q, k=k, v=v, o=out)
    ws = ctypes.c_void_p()
    rc = lib().tilemix_attention_fwd_noalloc(ctypes.byref(pp), _ptr(q), _ptr(k), _ptr(v), _ptr(q8), _ptr(k8),
                                             _ptr(q_scale), _ptr(k_scale), _ptr(words), _ptr(out), _ptr(lse), None,
                                             ctypes.byref(ws), _stream())
    _check(rc, "tilemix_attention_fwd_noalloc")
    return ws.value


def tilemix_read_status_at(workspace_addr: int):
    """tilemix_read_status on a raw device address (synchronises the current stream)."""
    rec = (ctypes.c_int32 * 4)()
    rc = lib().tilemix_read_status(ctypes.c_void_p(workspace_addr), ctypes.byref(rec), _stream())
    return rc, list(rec)


def tilemix_read_status(workspace: torch.Tensor):
    """Synchronises the current stream; returns (code, [code, role, tile, barrier])."""
    rec = (ctypes.c_int32 * 4)()
    rc = lib().tilemix_read_status(_ptr(workspace), ctypes.byref(rec), _stream())
    return rc, list(rec)


def tilemix_prefill_host(p: ProblemStruct, q_host, k_host, v_host, route_host, out_host, arena,
                         pin_diagonal=False):
    """Whole path on host (ideally pinned) tensors; `arena` is a CUDA uint8 tensor of
    tilemix_arena_size(p) bytes.  Asynchronous on the current stream."""
    for t in (q_host, k_host, v_host, route_host, out_host):
        assert not t.is_cuda and t.is_contiguous()
    rc = lib().tilemix_prefill_host(ctypes.byref(p), _ptr(q_host), _ptr(k_host), _ptr(v_host), _ptr(route_host),
                                    PIN_DIAGONAL_FP16 if pin_diagonal else 0, _ptr(out_host), _ptr(arena),
                                    arena.numel(), _stream())
    _check(rc, "tilemix_prefill_host")
    return out_host


def tilemix_arena_size(p): return int(lib().tilemix_arena_size(ctypes.byref(p)))
def tilemix_workspace_size(p): return int(lib().tilemix_workspace_size(ctypes.byref(p)))
def tilemix_scratch_bytes(p): return int(lib().tilemix_scratch_bytes(ctypes.byref(p)))
def tilemix_mask_words_per_row(seqlen, tile_n, group): return int(lib().tilemix_mask_words_per_row(seqlen, tile_n, group))
def tilemix_launch_count(): return int(lib().tilemix_launch_count())


def tilemix_tensor_peak_probe(int8: bool, n_mma: int, workspace) -> int:
    """Enqueues the tensor-pipe issue-rate probe on the current stream; returns the number of CTAs (time it with events)."""
    n = ctypes.c_int(0)
    _check(lib().tilemix_tensor_peak_probe(1 if int8 else 0, n_mma, ctypes.byref(n), _ptr(workspace), _stream()), "tilemix_tensor_peak_probe")
    return n.value


def tilemix_test_drop_copy(which: int, wait_limit_ns: int = 0):
    """Testing aid of the bounded waits (see tilemix.h); which = 0 switches it off."""
    _check(lib().tilemix_test_drop_copy(which, wait_limit_ns), "tilemix_test_drop_copy")


# ------------------------------------------------------------------ variable-length batches

class Varlen:
    """Host-side description of a packed batch: keeps the cu_seqlens array alive for the C struct."""

    def __init__(self, cu_seqlens, max_seqlen: int = 0):
        cu = [int(x) for x in cu_seqlens]
        self.cu = (ctypes.c_int32 * len(cu))(*cu)
        self.struct = VarlenStruct(len(cu) - 1, max_seqlen, ctypes.cast(self.cu, ctypes.POINTER(ctypes.c_int32)))
        self.cu_list = cu

    def ref(self):
        return ctypes.byref(self.struct)


def tilemix_varlen_counts(p: ProblemStruct, vl: Varlen) -> dict:
    out = (ctypes.c_int64 * 7)()
    _check(lib().tilemix_varlen_counts(ctypes.byref(p), vl.ref(), ctypes.byref(out)), "tilemix_varlen_counts")
    keys = ("total", "sum_T_m", "sum_blk_q", "sum_blk_k", "T_mask_max", "W", "max_seqlen")
    return dict(zip(keys, (int(x) for x in out)))


def tilemix_varlen_workspace_size(p: ProblemStruct, vl: Varlen) -> int:
    return int(lib().tilemix_varlen_workspace_size(ctypes.byref(p), vl.ref()))


def _varlen_strides(p: ProblemStruct, q=None, k=None, v=None, o=None) -> ProblemStruct:
    """Tensors are [total, H, d]; the C struct wants (batch, head, token) strides."""
    pp = ProblemStruct.from_buffer_copy(p)
    for name, t in (("q_stride", q), ("k_stride", k), ("v_stride", v), ("o_stride", o)):
        if t is not None:
            assert t.dim() == 3 and t.stride(-1) == 1 and t.shape[-1] == p.head_dim
            f = getattr(pp, name)
            f[0], f[1], f[2] = 0, t.stride(1), t.stride(0)
    return pp


def _varlen_ws(p, vl, dev, workspace):
    if workspace is None:
        workspace = torch.empty(tilemix_varlen_workspace_size(p, vl), dtype=torch.uint8, device=dev)
    return workspace


def tilemix_quantize_qk_varlen(p: ProblemStruct, vl: Varlen, q: torch.Tensor, k: torch.Tensor, workspace=None):
    """q [total,Hq,d], k [total,Hk,d] FP16 -> (q_i8 [Hq,total,d], k_i8 [Hk,total,d], q_scale [blocks_q,Hq],
    k_scale [blocks_k,Hk])."""
    c = tilemix_varlen_counts(p, vl)
    dev = q.device
    q8 = torch.empty((p.heads_q, p.seqlen, p.head_dim), dtype=torch.int8, device=dev)
    k8 = torch.empty((p.heads_kv, p.seqlen, p.head_dim), dtype=torch.int8, device=dev)
    qs = torch.empty((c["sum_blk_q"], p.heads_q), dtype=torch.float32, device=dev)
    ks = torch.empty((c["sum_blk_k"], p.heads_kv), dtype=torch.float32, device=dev)
    ws = _varlen_ws(p, vl, dev, workspace)
    pp = _varlen_strides(p, q=q, k=k)
    _check(lib().tilemix_quantize_qk_varlen(ctypes.byref(pp), vl.ref(), _ptr(q), _ptr(k), _ptr(q8), _ptr(k8),
                                            _ptr(qs), _ptr(ks), _ptr(ws), ws.numel(), _stream()),
           "tilemix_quantize_qk_varlen")
    return q8, k8, qs, ks


def tilemix_pack_routing_mask_varlen(p: ProblemStruct, vl: Varlen, route: torch.Tensor, pin_diagonal=False,
                                     workspace=None):
    """route uint8 [Hk, sum T_m, T_mask_max] -> (words [Hk, sum T_m, W] int32-typed bits, counts int64 [Hk,2])."""
    c = tilemix_varlen_counts(p, vl)
    assert route.dtype == torch.uint8 and route.is_cuda and route.is_contiguous()
    assert tuple(route.shape) == (p.heads_kv, c["sum_T_m"], c["T_mask_max"]), route.shape
    words = torch.empty((p.heads_kv, c["sum_T_m"], c["W"]), dtype=torch.int32, device=route.device)
    counts = torch.empty((p.heads_kv, 2), dtype=torch.int64, device=route.device)
    ws = _varlen_ws(p, vl, route.device, workspace)
    _check(lib().tilemix_pack_routing_mask_varlen(ctypes.byref(p), vl.ref(), _ptr(route),
                                                  PIN_DIAGONAL_FP16 if pin_diagonal else 0, _ptr(words),
                                                  _ptr(counts), _ptr(ws), ws.numel(), _stream()),
           "tilemix_pack_routing_mask_varlen")
    return words, counts


def tilemix_attention_fwd_varlen(p: ProblemStruct, vl: Varlen, q, k, v, q8=None, k8=None, q_scale=None,
                                 k_scale=None, words=None, out=None, want_lse=False, debug_tiles=None,
                                 workspace=None):
    """Fused forward over a packed batch; q [total,Hq,d], k/v [total,Hk,d].  Returns a dict like
    tilemix_attention_fwd with out [total,Hq,d] and lse [Hq,total]; debug_tiles are (sequence, h_q, m, n)."""
    dev = q.device
    if out is None:
        out = torch.empty((p.seqlen, p.heads_q, p.head_dim), dtype=torch.float16, device=dev)
    lse = torch.empty((p.heads_q, p.seqlen), dtype=torch.float32, device=dev) if want_lse else None
    ws = _varlen_ws(p, vl, dev, workspace)
    dbg, raw, kind = None, None, None
    if debug_tiles is not None:
        tiles = torch.as_tensor(debug_tiles, dtype=torch.int32).reshape(-1, 4).contiguous().to(dev)
        n = tiles.shape[0]
        raw = torch.zeros((n, p.tile_m, p.tile_n), dtype=torch.int32, device=dev)
        kind = torch.full((n,), 255, dtype=torch.uint8, device=dev)
        dbg = DebugStruct(tiles.data_ptr(), n, raw.data_ptr(), kind.data_ptr())
    pp = _varlen_strides(p, q=q, k=k, v=v, o=out)
    rc = lib().tilemix_attention_fwd_varlen(ctypes.byref(pp), vl.ref(), _ptr(q), _ptr(k), _ptr(v), _ptr(q8),
                                            _ptr(k8), _ptr(q_scale), _ptr(k_scale), _ptr(words), _ptr(out),
                                            _ptr(lse), _ptr(ws), ws.numel(),
                                            ctypes.byref(dbg) if dbg is not None else None, _stream())
    _check(rc, "tilemix_attention_fwd_varlen")
    return {"out": out, "lse": lse, "raw": raw, "kind": kind, "workspace": ws}


# ------------------------------------------------------------------ decode over an INT8 KV cache

def decode_problem(batch, heads_q, heads_kv, head_dim, max_len, tile_n, group=1, mask_batch=1, n_splits=0,
                   softmax_scale=0.0) -> DecodeStruct:
    return DecodeStruct(batch, heads_q, heads_kv, head_dim, max_len, tile_n, group, mask_batch, n_splits,
                        softmax_scale)


def tilemix_decode_workspace_size(p: DecodeStruct) -> int:
    return int(lib().tilemix_decode_workspace_size(ctypes.byref(p)))


def tilemix_decode_int8kv(p: DecodeStruct, q, k16, k8, k_scale, v8, v_scale, words, cache_len, out=None,
                          want_lse=False, want_q8=False, workspace=None):
    """One decode step: q [B,Hq,d] FP16; k16 [B,Hk,max_len,d] FP16 or None; k8/v8 INT8 like k16;
    scales FP32 [B,Hk,blocks]; words int32-typed bits [nb,Hk,W] or None; cache_len int32 [B] (CUDA).
    Returns a dict: out [B,Hq,d] FP16, lse, q8, q_scale (if asked)."""
    dev = q.device
    if out is None:
        out = torch.empty((p.batch, p.heads_q, p.head_dim), dtype=torch.float16, device=dev)
    lse = torch.empty((p.batch, p.heads_q), dtype=torch.float32, device=dev) if want_lse else None
    q8 = torch.empty((p.batch, p.heads_q, p.head_dim), dtype=torch.int8, device=dev) if want_q8 else None
    qs = torch.empty((p.batch, p.heads_q), dtype=torch.float32, device=dev) if want_q8 else None
    if workspace is None:
        workspace = torch.empty(tilemix_decode_workspace_size(p), dtype=torch.uint8, device=dev)
    assert cache_len.dtype == torch.int32 and cache_len.is_cuda
    rc = lib().tilemix_decode_int8kv(ctypes.byref(p), _ptr(q), _ptr(k16), _ptr(k8), _ptr(k_scale), _ptr(v8),
                                     _ptr(v_scale), _ptr(words), _ptr(cache_len), _ptr(out), _ptr(lse), _ptr(q8),
                                     _ptr(qs), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "tilemix_decode_int8kv")
    return {"out": out, "lse": lse, "q8": q8, "q_scale": qs, "workspace": workspace}


# ------------------------------------------------------------------ chunked prefill

def tilemix_attention_fwd_chunk(p: ProblemStruct, kv_len: int, q, k, v, q8, k8, q_scale, k_scale, words, out=None,
                                want_lse=False, workspace=None):
    """The last p.seqlen queries of a kv_len-token context: q [B,Hq,seqlen,d], k/v [B,Hk,kv_len,d], words
    those of the whole context.  Returns a dict like tilemix_attention_fwd."""
    dev = q.device
    if out is None:
        out = torch.empty((p.batch, p.heads_q, p.seqlen, p.head_dim), dtype=torch.float16, device=dev)
    lse = torch.empty((p.batch, p.heads_q, p.seqlen), dtype=torch.float32, device=dev) if want_lse else None
    if workspace is None:
        workspace = torch.empty(4096, dtype=torch.uint8, device=dev)
    pp = _with_strides(p, q=q, k=k, v=v, o=out)
    rc = lib().tilemix_attention_fwd_chunk(ctypes.byref(pp), kv_len, _ptr(q), _ptr(k), _ptr(v), _ptr(q8), _ptr(k8),
                                           _ptr(q_scale), _ptr(k_scale), _ptr(words), _ptr(out), _ptr(lse),
                                           _ptr(workspace), workspace.numel(), None, _stream())
    _check(rc, "tilemix_attention_fwd_chunk")
    return {"out": out, "lse": lse, "workspace": workspace}


def tilemix_chunk_v8_workspace_size(p: ProblemStruct, kv_len: int) -> int:
    return int(lib().tilemix_chunk_v8_workspace_size(ctypes.byref(p), kv_len))


def tilemix_attention_fwd_chunk_v8(p: ProblemStruct, kv_len: int, q, k, v8, v_scale, q8, k8, q_scale, k_scale, words,
                                   out=None, want_lse=False, workspace=None):
    """As tilemix_attention_fwd_chunk with the values taken from an INT8 cache: v8 int8 [B,Hk,kv_len,d] (dense),
    v_scale float32 [B,Hk,ceil(kv_len/tile)]."""
    dev = q.device
    if out is None:
        out = torch.empty((p.batch, p.heads_q, p.seqlen, p.head_dim), dtype=torch.float16, device=dev)
    lse = torch.empty((p.batch, p.heads_q, p.seqlen), dtype=torch.float32, device=dev) if want_lse else None
    pp = _with_strides(p, q=q, k=k, o=out)
    if workspace is None:
        workspace = torch.empty(max(tilemix_chunk_v8_workspace_size(pp, kv_len), 4096), dtype=torch.uint8, device=dev)
    rc = lib().tilemix_attention_fwd_chunk_v8(ctypes.byref(pp), kv_len, _ptr(q), _ptr(k), _ptr(v8), _ptr(v_scale),
                                              _ptr(q8), _ptr(k8), _ptr(q_scale), _ptr(k_scale), _ptr(words), _ptr(out),
                                              _ptr(lse), _ptr(workspace), workspace.numel(), _stream())
    _check(rc, "tilemix_attention_fwd_chunk_v8")
    return {"out": out, "lse": lse, "workspace": workspace}
