"""Chunked prefill: the last L_q queries of a context, against the whole-context prefill (bit for bit)
and against the CPU oracle's rows."""
import numpy as np
import pytest
import torch

from paper_2608_17336_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run(L, Lq, heads_q, heads_kv, d, tile, G, seed, f8=0.5, pin=False):
    from paper_2608_17336_b200 import binding as tm
    w = synth.Workload("ctx", 2, heads_q, L, d, tile, G, seed=seed, routing="bernoulli", int8_fraction=f8,
                       pin_diagonal=pin)
    q, k, v = synth.make_qkv(w)
    k, v = k[:, :heads_kv].contiguous(), v[:, :heads_kv].contiguous()
    route = np.ascontiguousarray(synth.make_route(w)[:, :heads_kv])
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    # the whole context in one call
    p_full = tm.problem(2, heads_q, heads_kv, L, d, tile, tile, G)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p_full, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask(p_full, torch.from_numpy(route).to(dev), pin)
    full = tm.tilemix_attention_fwd(p_full, qd, kd, vd, q8, k8, qs, ks, words, want_lse=True)
    # the last Lq queries as a chunk of their own: its Q is quantised on its own (blocks line up)
    off = L - Lq
    p_chunk = tm.problem(2, heads_q, heads_kv, Lq, d, tile, tile, G)
    qc = qd[:, :, off:].contiguous()
    q8c, _, qsc, _ = tm.tilemix_quantize_qk(p_chunk, qc, kd[:, :, off:].contiguous())
    assert torch.equal(q8c, q8[:, :, off:]) and torch.equal(qsc, qs[:, :, off // tile:])
    res = tm.tilemix_attention_fwd_chunk(p_chunk, L, qc, kd, vd, q8c, k8, qsc, ks, words, want_lse=True)
    code, rec = tm.tilemix_read_status(res["workspace"])
    assert code == 0, rec
    assert torch.equal(res["out"].view(torch.int16), full["out"][:, :, off:].contiguous().view(torch.int16))
    assert torch.equal(res["lse"], full["lse"][:, :, off:])
    return w, q, k, v, route, res, off


@pytest.mark.parametrize("L,Lq,tile,d", [(1000, 232, 128, 128), (640, 128, 128, 128), (700, 700, 128, 128),
                                         (333, 77, 64, 64), (512, 64, 64, 64)])
def test_chunk_equals_rows_of_the_whole_context(L, Lq, tile, d):
    _run(L, Lq, 2, 2, d, tile, 2, seed=51)


def test_chunk_gqa_against_the_oracle():
    L, Lq, tile = 900, 260, 128
    w, q, k, v, route, res, off = _run(L, Lq, 4, 2, 128, tile, 1, seed=52, f8=0.6, pin=True)
    import oracle
    p = oracle.Problem(2, 4, 2, L, 128, tile, tile, 1)
    qb, kb, vb = H.np_bits(q), H.np_bits(k), H.np_bits(v)
    q8, qs = oracle.quantize(qb, tile)
    k8, ks = oracle.quantize(kb, tile)
    words, _ = oracle.pack(p, route, True)
    rows = [(b, h, i) for b in range(2) for h in range(4) for i in range(off, L, 7)]
    ref, _, _ = oracle.attention_rows(p, qb, kb, vb, q8, k8, qs, ks, words, rows)
    got = np.stack([res["out"][b, h, i - off].float().cpu().numpy() for b, h, i in rows]).astype(np.float64)
    assert (np.abs(got - ref) <= H.ATOL * np.maximum(1.0, np.abs(ref))).all()


def test_chunk_rejects_unaligned_offsets():
    from paper_2608_17336_b200 import binding as tm
    p = tm.problem(1, 1, 1, 100, 64, 64, 64)
    dev = torch.device("cuda:0")
    x = torch.zeros((1, 1, 100, 64), dtype=torch.float16, device=dev)
    kv = torch.zeros((1, 1, 150, 64), dtype=torch.float16, device=dev)
    with pytest.raises(tm.TilemixError) as e:
        tm.tilemix_attention_fwd_chunk(p, 150, x, kv, kv, None, None, None, None, None)
    assert e.value.code == tm.ERR_SHAPE
