"""CPU-only checks of the C-ABI library: it loads, exports every symbol the public header
declares, rejects bad arguments on the host before any launch, and its size helpers agree
with the closed forms of the paper's accounting."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from paper_2608_17336_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_17336_b200 import build
    build.build()
    return b.lib()


def test_library_exports_every_declared_symbol(lib):
    declared = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        declared |= set(re.findall(r"\b(tilemix_[a-z0-9_]+)\s*\(", text))
    assert declared == set(b.EXPORTS), declared ^ set(b.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_problem_struct_matches_header_layout():
    assert ctypes.sizeof(b.ProblemStruct) == 14 * 4 + 12 * 8
    assert b.ProblemStruct.q_stride.offset == 56 and b.ProblemStruct.o_stride.offset == 56 + 72


def _args(n):
    return [ctypes.c_void_p(0x1000)] * n


def test_host_side_validation_without_gpu(lib):
    good = b.problem(1, 2, 2, 1024, 128, 128, 128)
    null = None
    # NULL problem / pointers
    assert lib.tilemix_quantize_qk(None, *_args(6), null) == b.ERR_NULL
    assert lib.tilemix_quantize_qk(ctypes.byref(good), null, null, null, null, null, null, null) == b.ERR_NULL
    assert lib.tilemix_quantize_qk(ctypes.byref(good), ctypes.c_void_p(0x1000), null, null, null, null, null, null) == b.ERR_NULL
    assert lib.tilemix_pack_routing_mask(ctypes.byref(good), null, 0, ctypes.c_void_p(0x1000), null, null) == b.ERR_NULL
    # shapes
    for field, val in (("batch", 0), ("seqlen", -1), ("group", 0), ("heads_kv", 3), ("head_dim", 12), ("mask_batch", 2)):
        bad = b.problem(1, 2, 2, 1024, 128, 128, 128)
        setattr(bad, field, val)
        assert lib.tilemix_quantize_qk(ctypes.byref(bad), *_args(6), null) == b.ERR_SHAPE, field
        assert lib.tilemix_workspace_size(ctypes.byref(bad)) == 0
    # alignment of bases and strides
    assert lib.tilemix_quantize_qk(ctypes.byref(good), ctypes.c_void_p(0x1008), *_args(5), null) == b.ERR_ALIGN
    odd = b.problem(1, 2, 2, 1024, 128, 128, 128)
    odd.q_stride[0], odd.q_stride[1], odd.q_stride[2] = 2 * 1024 * 132, 1024 * 132, 132
    assert lib.tilemix_quantize_qk(ctypes.byref(odd), *_args(6), null) == b.ERR_ALIGN
    # attention: unsupported tile / head_dim / quant block, missing INT8 operands, small workspace
    att = lambda p, ws=4096, q8=0x1000: lib.tilemix_attention_fwd(
        ctypes.byref(p), *_args(3), ctypes.c_void_p(q8) if q8 else None, *_args(5), None, ctypes.c_void_p(0x1000), ws, None, None)
    assert att(b.problem(1, 2, 2, 1024, 128, 64, 64)) == b.ERR_UNSUPPORTED
    assert att(b.problem(1, 2, 2, 1024, 96, 128, 128)) == b.ERR_UNSUPPORTED
    # quantisation blocks: K per key tile or per half key tile, Q per query tile; the on-the-fly mode per tile only
    assert att(b.problem(1, 2, 2, 1024, 128, 128, 128, quant_blk_k=32)) == b.ERR_UNSUPPORTED
    assert att(b.problem(1, 2, 2, 1024, 128, 128, 128, quant_blk_q=64)) == b.ERR_UNSUPPORTED
    assert att(b.problem(1, 2, 2, 1024, 128, 128, 128, quant_blk_k=64, flags=b.QUANT_ON_THE_FLY)) == b.ERR_UNSUPPORTED
    assert att(good, ws=8) == b.ERR_WORKSPACE
    assert att(good, q8=0) == b.ERR_NULL
    assert att(good, q8=0x1001) == b.ERR_ALIGN
    dbg = b.DebugStruct(None, 3, None, None)
    assert lib.tilemix_attention_fwd(ctypes.byref(good), *_args(9), None, ctypes.c_void_p(0x1000), 4096,
                                     ctypes.byref(dbg), None) == b.ERR_NULL
    # on-the-fly operand mode: the INT8 operands and scales may be NULL (the call gets as far as the workspace
    # check), the routing words may not; 128x128 tiles only
    one = ctypes.c_void_p(0x1000)
    otf = b.problem(1, 2, 2, 1024, 128, 128, 128, flags=b.QUANT_ON_THE_FLY)
    assert lib.tilemix_attention_fwd(ctypes.byref(otf), one, one, one, None, None, None, None, one, one, None,
                                     one, 8, None, None) == b.ERR_WORKSPACE
    assert lib.tilemix_attention_fwd(ctypes.byref(otf), one, one, one, None, None, None, None, None, one, None,
                                     one, 4096, None, None) == b.ERR_NULL
    otf64 = b.problem(1, 2, 2, 1024, 64, 64, 64, flags=b.QUANT_ON_THE_FLY)
    assert lib.tilemix_attention_fwd(ctypes.byref(otf64), one, one, one, None, None, None, None, one, one, None,
                                     one, 4096, None, None) == b.ERR_UNSUPPORTED
    chunk = b.problem(1, 2, 2, 256, 64, 64, 64, flags=b.QUANT_ON_THE_FLY)
    assert lib.tilemix_attention_fwd_chunk(ctypes.byref(chunk), 1024, *_args(9), None, one, 4096, None,
                                           None) == b.ERR_UNSUPPORTED
    assert lib.tilemix_launch_count() == 0


def test_status_strings(lib):
    for code in (0, -1, -2, -3, -4, -5, -6):
        assert lib.tilemix_status_string(code)
    assert b"wait" in lib.tilemix_status_string(b.ERR_DEVICE_TIMEOUT)


def test_mask_words_per_row(lib):
    assert b.tilemix_mask_words_per_row(1024, 64, 1) == 1
    assert b.tilemix_mask_words_per_row(8192, 128, 1) == 2
    assert b.tilemix_mask_words_per_row(32768, 128, 4) == 2
    assert b.tilemix_mask_words_per_row(4096, 128, 2) == 1
    assert b.tilemix_mask_words_per_row(131072, 128, 8) == 4
    assert b.tilemix_mask_words_per_row(0, 128, 8) < 0
    for L, t, g in ((1000, 128, 3), (77, 64, 1), (5000, 64, 2)):
        assert b.tilemix_mask_words_per_row(L, t, g) == oracle.Problem(1, 1, 1, L, 64, t, t, g).W


def test_scratch_bytes_matches_paper_accounting(lib):
    """App. D accounting shape (H_q=32, H_k=8, L=8192, d=128, BLK_Q=128, BLK_K=64): the
    quantize-once scratch is everything beyond the FP16 Q/K/V; with this library's FP32 scales
    and two uint32 words per row it is the closed form with 4-byte scales and 8-byte rows."""
    p = b.problem(1, 32, 8, 8192, 128, 128, 128, 1, quant_blk_q=128, quant_blk_k=64)
    total, fp16 = oracle.resident_bytes_quantize_once(32, 8, 8192, 128, 128, 64, 128, scale_bytes=4, word_bytes=8)
    assert b.tilemix_scratch_bytes(p) == total - fp16
    # and with the paper's FP16 scales the same sum is the printed 136.01 MiB
    total16, _ = oracle.resident_bytes_quantize_once(32, 8, 8192, 128, 128, 64, 128)
    assert round(total16 / 2 ** 20, 2) == 136.01
    assert b.tilemix_arena_size(p) >= total


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", "/nonexistent/libtilemix.so")
    with pytest.raises(RuntimeError, match="no CPU or library fallback"):
        b.lib()


# ------------------------------------------------------------------ variable-length batches

def test_varlen_counts_and_workspace(lib):
    lens = [1, 37, 64, 0, 200, 129, 513]
    cu = np.cumsum([0] + lens).tolist()
    p = b.problem(1, 4, 2, cu[-1], 64, 64, 64, group=2)
    vl = b.Varlen(cu)
    c = b.tilemix_varlen_counts(p, vl)
    tiles = sum(-(-L // 64) for L in lens)
    assert c == dict(total=cu[-1], sum_T_m=tiles, sum_blk_q=tiles, sum_blk_k=tiles,
                     T_mask_max=-(-513 // 128), W=1, max_seqlen=513)
    # the paper's scale shapes for variable-length batches: sum_b ceil(L_b / block) entries per head
    p2 = b.problem(1, 4, 2, cu[-1], 64, 64, 64, quant_blk_q=128, quant_blk_k=32)
    c2 = b.tilemix_varlen_counts(p2, vl)
    assert c2["sum_blk_q"] == sum(-(-L // 128) for L in lens)
    assert c2["sum_blk_k"] == sum(-(-L // 32) for L in lens)
    # status area + four int32 tables of n_seqs + 1 entries + two int32 per work item (pair of query
    # tiles: 12 here), rounded up to 256 bytes
    assert b.tilemix_varlen_workspace_size(p, vl) == 4096 + 256
    big = b.Varlen(list(range(0, 101)))
    assert b.tilemix_varlen_workspace_size(b.problem(1, 1, 1, 100, 64, 64, 64), big) == 4096 + 2560   # 4 * 101 * 4 + 2 * 100 * 4 = 2416 bytes


def test_varlen_host_side_validation(lib):
    cu = [0, 100, 300]
    ok = b.problem(1, 2, 2, 300, 64, 64, 64)
    out = (ctypes.c_int64 * 7)()

    def counts(p, vl):
        return lib.tilemix_varlen_counts(ctypes.byref(p), vl.ref() if vl else None, ctypes.byref(out))

    assert counts(ok, b.Varlen(cu)) == b.OK
    assert counts(ok, None) == b.ERR_NULL
    assert counts(ok, b.Varlen([0, 100, 299])) == b.ERR_SHAPE          # last entry != seqlen
    assert counts(ok, b.Varlen([1, 100, 300])) == b.ERR_SHAPE          # first entry != 0
    assert counts(ok, b.Varlen([0, 200, 100, 300])) == b.ERR_SHAPE     # decreasing
    assert counts(ok, b.Varlen(cu, max_seqlen=150)) == b.ERR_SHAPE     # bound below the longest sequence
    assert counts(ok, b.Varlen(cu, max_seqlen=4096)) == b.OK and out[4] == 64 and out[5] == 2
    assert counts(b.problem(2, 2, 2, 300, 64, 64, 64), b.Varlen(cu)) == b.ERR_SHAPE   # batch must be 1
    assert lib.tilemix_varlen_workspace_size(ctypes.byref(ok), b.Varlen([0, 1, 2]).ref()) == 0
    # the launching entry points reject bad arguments before touching the device
    vl = b.Varlen(cu)
    one = ctypes.c_void_p(4096)
    assert lib.tilemix_quantize_qk_varlen(ctypes.byref(ok), vl.ref(), None, None, None, None, None, None,
                                          one, 8192, None) == b.ERR_NULL
    assert lib.tilemix_quantize_qk_varlen(ctypes.byref(ok), vl.ref(), one, None, one, None, one, None,
                                          one, 100, None) == b.ERR_WORKSPACE
    assert lib.tilemix_pack_routing_mask_varlen(ctypes.byref(ok), vl.ref(), None, 0, one, None, one, 8192,
                                                None) == b.ERR_NULL
    assert lib.tilemix_attention_fwd_varlen(ctypes.byref(ok), vl.ref(), one, one, one, None, None, None, None,
                                            None, one, None, one, 8192, None, None) == b.ERR_NULL
    otf = b.problem(1, 2, 2, 300, 64, 64, 64, flags=b.QUANT_ON_THE_FLY)   # dense batches only
    assert lib.tilemix_attention_fwd_varlen(ctypes.byref(otf), vl.ref(), one, one, one, one, one, one, one,
                                            one, one, None, one, 8192, None, None) == b.ERR_UNSUPPORTED
    long = b.problem(1, 1, 1, 64 * 2049, 64, 64, 64, flags=b.FORCE_FP16)
    assert lib.tilemix_attention_fwd_varlen(ctypes.byref(long), b.Varlen([0, 64 * 2049]).ref(), one, one, one,
                                            None, None, None, None, None, one, None, one, 8192, None,
                                            None) == b.ERR_UNSUPPORTED


# ------------------------------------------------------------------ decode over an INT8 KV cache

def test_decode_host_side_validation(lib):
    ok = b.decode_problem(8, 32, 8, 128, 32768, 128, 4)
    size = lib.tilemix_decode_workspace_size(ctypes.byref(ok))
    # 256-byte status area + the clamped lengths (a 256-byte area for up to 64 sequences) + partial outputs and
    # two float arrays per (batch, query head, split)
    splits = (size - 512) // (8 * 32 * (128 * 4 + 8))
    assert splits >= 1 and size == 512 + 8 * 32 * splits * (128 * 4 + 8)
    assert b.tilemix_decode_workspace_size(b.decode_problem(1, 4, 1, 64, 64, 64, n_splits=7)) == 256 + 256 + 1024 + 2 * 256
    # head_dim 128 with 128-key tiles (the tcgen05 form): one wave of CTAs by default (148 SMs / 64 rows = 2 splits),
    # two partial results per split
    assert splits == 2 * 2
    # n_splits = -1: the kernel shares the wave's CTAs out by the rows' cost, up to max(16, 8 * 2) to a row
    shared = b.tilemix_decode_workspace_size(b.decode_problem(8, 32, 8, 128, 32768, 128, 4, n_splits=-1))
    assert shared == 512 + 8 * 32 * (2 * 16) * (128 * 4 + 8)
    assert lib.tilemix_decode_workspace_size(ctypes.byref(b.decode_problem(8, 32, 8, 128, 32768, 128, 4, n_splits=-2))) == 0
    # ... where it can: not with more rows than a wave has CTAs, and not in the warp-level form
    assert (b.tilemix_decode_workspace_size(b.decode_problem(32, 32, 8, 128, 32768, 128, 4, n_splits=-1))
            == b.tilemix_decode_workspace_size(b.decode_problem(32, 32, 8, 128, 32768, 128, 4)))
    assert (b.tilemix_decode_workspace_size(b.decode_problem(2, 8, 2, 64, 4096, 64, 1, n_splits=-1))
            == b.tilemix_decode_workspace_size(b.decode_problem(2, 8, 2, 64, 4096, 64, 1)))
    # more rows than a wave has CTAs: one split per row, nothing to share out
    many = b.tilemix_decode_workspace_size(b.decode_problem(32, 32, 8, 128, 32768, 128, 4))
    assert many == 256 + 256 + 32 * 32 * 2 * (128 * 4 + 8)
    # a short cache: at least four key tiles per split
    short = b.tilemix_decode_workspace_size(b.decode_problem(1, 8, 1, 128, 1024, 128, 1))
    assert short == 256 + 256 + 8 * (2 * 2) * 128 * 4 + 2 * 256      # (the two float arrays are rounded up to 256 bytes)
    three = b.tilemix_decode_workspace_size(b.decode_problem(8, 32, 8, 128, 32768, 128, 4, n_splits=3))
    assert three == 512 + 8 * 32 * (2 * 3) * (128 * 4 + 8)
    for bad in (b.decode_problem(0, 32, 8, 128, 1024, 128), b.decode_problem(1, 6, 4, 128, 1024, 128),
                b.decode_problem(1, 4, 4, 128, 0, 128), b.decode_problem(2, 4, 4, 128, 1024, 128, mask_batch=3)):
        assert lib.tilemix_decode_workspace_size(ctypes.byref(bad)) == 0
    one = ctypes.c_void_p(4096)

    def call(p, q=one, k16=one, k8=one, ks=one, v8=one, vs=one, words=one, lens=one, out=one, ws=one, nbytes=1 << 30):
        return lib.tilemix_decode_int8kv(ctypes.byref(p), q, k16, k8, ks, v8, vs, words, lens, out, None, None, None,
                                         ws, nbytes, None)

    assert call(b.decode_problem(1, 4, 4, 96, 1024, 128)) == b.ERR_UNSUPPORTED      # head_dim
    assert call(b.decode_problem(1, 12, 4, 128, 1024, 128)) == b.ERR_UNSUPPORTED    # 3 query heads per KV head
    assert call(b.decode_problem(1, 4, 4, 128, 1024, 32)) == b.ERR_UNSUPPORTED      # tile
    assert call(ok, q=None) == b.ERR_NULL and call(ok, lens=None) == b.ERR_NULL
    assert call(ok, k16=None, words=None) == b.ERR_NULL                               # all FP16 without an FP16 cache
    assert call(ok, k8=ctypes.c_void_p(4100)) == b.ERR_ALIGN
    assert call(ok, nbytes=size - 1) == b.ERR_WORKSPACE


def test_chunk_v8_host_side_validation(lib):
    """tilemix_attention_fwd_chunk_v8: what the host can refuse before any launch."""
    one = ctypes.c_void_p(0x1000)
    p = b.problem(1, 4, 2, 256, 128, 128, 128)
    need = lib.tilemix_chunk_v8_workspace_size(ctypes.byref(p), 1024)
    assert need == 4096 + 1 * 2 * 1024 * 128 * 2                       # status record + FP16 image of the value cache
    assert lib.tilemix_chunk_v8_workspace_size(ctypes.byref(p), 1000) == 0          # offset not a multiple of the tile
    args = [one] * 11                                                  # q, k, v8, v_scale, q8, k8, qs, ks, words, out, lse
    call = lambda prob, kv, a, ws=one, nbytes=need: lib.tilemix_attention_fwd_chunk_v8(
        ctypes.byref(prob), kv, *a, ws, nbytes, None)
    assert call(p, 1000, args) == b.ERR_SHAPE
    assert call(p, 128, args) == b.ERR_SHAPE                           # context shorter than the chunk
    no_scale = list(args); no_scale[3] = None
    assert call(p, 1024, no_scale) == b.ERR_NULL
    no_v = list(args); no_v[2] = None
    assert call(p, 1024, no_v) == b.ERR_NULL
    assert call(p, 1024, args, nbytes=need - 1) == b.ERR_WORKSPACE
    skew = list(args); skew[2] = ctypes.c_void_p(0x1008)
    assert call(p, 1024, skew) == b.ERR_ALIGN
    otf = b.problem(1, 4, 2, 256, 128, 128, 128, flags=b.QUANT_ON_THE_FLY)
    assert call(otf, 1024, args) == b.ERR_UNSUPPORTED
    assert lib.tilemix_attention_fwd_chunk_v8(None, 1024, *args, one, need, None) == b.ERR_NULL
