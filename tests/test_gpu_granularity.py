"""The paper's evaluated quantisation granularity (App. C "Quantization Granularity": BLK_Q = 128, BLK_K = 64 with
128 x 128 score tiles): one delta_K per half key tile.  Dense, variable-length and chunked calls against the oracle,
which takes the block sizes as they are; raw INT32 accumulator tiles bit for bit."""
import numpy as np
import pytest
import torch

import oracle
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _inputs(B, Hq, Hk, L, d, seed, k_scale_ramp=True):
    gen = torch.Generator().manual_seed(seed)
    q = torch.randn((B, Hq, L, d), generator=gen).half()
    k = torch.randn((B, Hk, L, d), generator=gen)
    if k_scale_ramp:     # neighbouring 64-row blocks get clearly different scales
        k = k * (1.0 + 3.0 * ((torch.arange(L) // (d // 2 if d == 64 else 64)) % 2).view(1, 1, L, 1))
    v = torch.randn((B, Hk, L, d), generator=gen).half()
    return q, k.half(), v


@pytest.mark.parametrize("B,Hq,Hk,L,d,tile,G,f8,pin", [
    (1, 2, 2, 1000, 128, 128, 1, 0.6, False),      # ragged: the last key tile has one full and one partial block
    (2, 4, 2, 640, 128, 128, 2, 1.0, True),
    (1, 2, 1, 520, 128, 128, 1, 1.0, False),       # the last tile's second block does not exist (520 = 4*128 + 8)
    (1, 2, 2, 333, 64, 64, 2, 0.7, False),         # 64 x 64 tiles with 32-row K blocks
])
def test_half_tile_k_blocks_dense(B, Hq, Hk, L, d, tile, G, f8, pin):
    from paper_2608_17336_b200 import binding as tm
    q, k, v = _inputs(B, Hq, Hk, L, d, seed=L + d)
    p = tm.problem(B, Hq, Hk, L, d, tile, tile, G, quant_blk_q=tile, quant_blk_k=tile // 2)
    po = oracle.Problem(B, Hq, Hk, L, d, tile, tile, G, blk_q=tile, blk_k=tile // 2)
    route = (np.random.default_rng(L).random((1, Hk, po.T_m, po.T_mask)) < f8).astype(np.uint8)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask(p, torch.from_numpy(route).to(DEV), pin)
    tiles = [(b, h, m, n) for b in range(B) for h in range(Hq) for m in range(po.T_m) for n in range(m + 1)]
    res = tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words, want_lse=True, debug_tiles=tiles)
    assert tm.tilemix_read_status(res["workspace"])[0] == 0
    qb, kb, vb = H.np_bits(q), H.np_bits(k), H.np_bits(v)
    q8o, qso = oracle.quantize(qb, tile)
    k8o, kso = oracle.quantize(kb, tile // 2)
    assert kso.shape[-1] == -(-L // (tile // 2)) and ks.shape == kso.shape
    assert np.array_equal(k8.cpu().numpy(), k8o) and np.array_equal(ks.cpu().numpy().view(np.uint32), kso.view(np.uint32))
    assert np.array_equal(q8.cpu().numpy(), q8o)
    wo, _ = oracle.pack(po, route, pin)
    ref, ref_lse, _ = oracle.attention_full(po, qb, kb, vb, q8o, k8o, qso, kso, wo)
    got = res["out"].float().cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref) <= H.ATOL * np.maximum(1.0, np.abs(ref))).all(), np.abs(got - ref).max()
    assert np.abs(res["lse"].cpu().numpy() - ref_lse).max() < 2e-3
    raw, kind = res["raw"].cpu().numpy(), res["kind"].cpu().numpy()
    n8 = 0
    for e, (b, h, m, n) in enumerate(tiles):
        if kind[e]:
            n8 += 1
            assert np.array_equal(raw[e], oracle.int32_tile(po, q8o, k8o, b, h, m, n))
    assert n8 > 0
    # the two granularities really differ here (the per-tile scale is the larger of the two block scales)
    _, ks_tile = oracle.quantize(kb, tile)
    assert not np.array_equal(np.repeat(ks_tile, 2, axis=-1)[..., :kso.shape[-1]], kso)
    # and the fast path (no debug request) gives the same within rounding
    fast = tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words)
    assert (np.abs(fast["out"].float().cpu().numpy() - ref) <= H.ATOL * np.maximum(1.0, np.abs(ref))).all()


def test_half_tile_k_blocks_scratch_size_is_the_papers_accounting():
    """App. D accounting shape (H_q = 32, H_k = 8, L = 8192, d = 128, BLK 128/64): the INT8 copies, the scales and the
    packed words of tilemix_scratch_bytes are what the paper's accounting adds to the 96 MB of FP16 operands."""
    from paper_2608_17336_b200 import binding as tm
    p = tm.problem(1, 32, 8, 8192, 128, 128, 128, 1, quant_blk_q=128, quant_blk_k=64)
    got = tm.tilemix_scratch_bytes(p)
    want = 32 * 8192 * 128 + 8 * 8192 * 128 + 4 * (32 * 64 + 8 * 128) + 4 * 8 * 64 * 2
    assert got == want
    # the closed form of App. D with this library's 4-byte scales (the paper's table, pinned in the oracle's tests
    # with 2-byte scales, prints 136.01 MiB in total)
    total, fp16 = oracle.resident_bytes_quantize_once(32, 8, 8192, 128, 128, 64, 128, scale_bytes=4, word_bytes=8)
    assert got == total - fp16

def test_half_tile_k_blocks_varlen_and_chunk():
    from paper_2608_17336_b200 import binding as tm
    tile, d, Hq, Hk, G = 128, 128, 2, 1, 1
    # ---- a packed batch: sequence lengths that leave partial blocks
    cu = [0, 300, 300, 940, 1010]
    total = cu[-1]
    gen = torch.Generator().manual_seed(7)
    q = torch.randn((total, Hq, d), generator=gen).half()
    k = (torch.randn((total, Hk, d), generator=gen) * (1.0 + 2.0 * ((torch.arange(total) // 64) % 2).view(total, 1, 1))).half()
    v = torch.randn((total, Hk, d), generator=gen).half()
    p = tm.problem(1, Hq, Hk, total, d, tile, tile, G, quant_blk_q=tile, quant_blk_k=64)
    vl = tm.Varlen(cu)
    lens = [cu[i + 1] - cu[i] for i in range(len(cu) - 1)]
    rows = sum(-(-x // tile) for x in lens)
    route = (np.random.default_rng(5).random((Hk, rows, -(-max(lens) // tile))) < 0.7).astype(np.uint8)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    q8, k8, qs, ks = tm.tilemix_quantize_qk_varlen(p, vl, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask_varlen(p, vl, torch.from_numpy(route).to(DEV), False)
    res = tm.tilemix_attention_fwd_varlen(p, vl, qd, kd, vd, q8, k8, qs, ks, words)
    assert tm.tilemix_read_status(res["workspace"])[0] == 0
    row0 = 0
    for s_, L in enumerate(lens):
        T_m = -(-L // tile)
        if L:
            po = oracle.Problem(1, Hq, Hk, L, d, tile, tile, G, blk_q=tile, blk_k=64)
            sl = slice(cu[s_], cu[s_ + 1])
            qb, kb, vb = (H.np_bits(t[sl].permute(1, 0, 2)[None]) for t in (q, k, v))
            q8o, qso = oracle.quantize(qb, tile)
            k8o, kso = oracle.quantize(kb, 64)
            wo, _ = oracle.pack(po, np.ascontiguousarray(route[None, :, row0:row0 + T_m, :po.T_mask]))
            ref, _, _ = oracle.attention_full(po, qb, kb, vb, q8o, k8o, qso, kso, wo)
            got = res["out"][sl].float().cpu().numpy().astype(np.float64).transpose(1, 0, 2)
            assert (np.abs(got - ref[0]) <= H.ATOL * np.maximum(1.0, np.abs(ref[0]))).all(), (s_, np.abs(got - ref[0]).max())
        row0 += T_m
    # ---- a chunk: the last 256 queries of a 700-token context equal those rows of the whole-context call
    L, Lq = 700, 256 + 60     # offset 384 = 3 tiles
    gen = torch.Generator().manual_seed(8)
    q = torch.randn((1, Hq, L, d), generator=gen).half()
    k = (torch.randn((1, Hk, L, d), generator=gen) * (1.0 + 2.0 * ((torch.arange(L) // 64) % 2).view(1, 1, L, 1))).half()
    v = torch.randn((1, Hk, L, d), generator=gen).half()
    pw = tm.problem(1, Hq, Hk, L, d, tile, tile, G, quant_blk_q=tile, quant_blk_k=64)
    route = (np.random.default_rng(6).random((1, Hk, pw.T_m, pw.T_mask)) < 0.7).astype(np.uint8)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(pw, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask(pw, torch.from_numpy(route).to(DEV), False)
    whole = tm.tilemix_attention_fwd(pw, qd, kd, vd, q8, k8, qs, ks, words)["out"]
    off = L - Lq
    assert off % tile == 0
    pc = tm.problem(1, Hq, Hk, Lq, d, tile, tile, G, quant_blk_q=tile, quant_blk_k=64)
    part = tm.tilemix_attention_fwd_chunk(pc, L, qd[:, :, off:].contiguous(), kd, vd, q8[:, :, off:].contiguous(), k8,
                                          qs[:, :, off // tile:].contiguous(), ks, words)["out"]
    assert torch.equal(part.view(torch.int16), whole[:, :, off:].contiguous().view(torch.int16))
