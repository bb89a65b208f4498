"""On-the-fly operand generation (App. D, the "fused on-the-fly" mode): the attention kernel makes the INT8
tiles and their scales on chip.  The quantiser's arithmetic is fixed (App. C), so the result has to equal the
quantise-once path bit for bit; it is also checked against the CPU oracle directly, including the raw INT32
accumulators of INT8-routed tiles."""
import numpy as np
import pytest
import torch

from paper_2608_17336_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _both(B, heads_q, heads_kv, L, G, seed, f8=0.5, pin=False, routing="bernoulli", transform=None, debug_tiles=None):
    from paper_2608_17336_b200 import binding as tm
    w = synth.Workload("otf", B, heads_q, L, 128, 128, G, seed=seed, routing=routing, int8_fraction=f8,
                       pin_diagonal=pin)
    q, k, v = synth.make_qkv(w)
    k, v = k[:, :heads_kv].contiguous(), v[:, :heads_kv].contiguous()
    if transform is not None:
        q, k, v = transform(q, k, v)
    route = np.ascontiguousarray(synth.make_route(w)[:, :heads_kv])
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    p = tm.problem(B, heads_q, heads_kv, L, 128, 128, 128, G)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask(p, torch.from_numpy(route).to(dev), pin)
    once = tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words, want_lse=True, debug_tiles=debug_tiles)
    p_otf = tm.problem(B, heads_q, heads_kv, L, 128, 128, 128, G, flags=tm.QUANT_ON_THE_FLY)
    otf = tm.tilemix_attention_fwd(p_otf, qd, kd, vd, None, None, None, None, words, want_lse=True,
                                   debug_tiles=debug_tiles)
    code, rec = tm.tilemix_read_status(otf["workspace"])
    assert code == 0, rec
    return w, (q, k, v), route, once, otf


@pytest.mark.parametrize("B,hq,hk,L,G,f8,pin", [
    (1, 2, 2, 1024, 1, 0.5, False),      # every key tile staged on both routes somewhere
    (2, 4, 2, 900, 2, 0.6, True),        # GQA, ragged tail, pinned diagonal
    (1, 2, 2, 2500, 4, 1.0, False),      # all INT8, more key tiles than ring slots and scale slots
    (1, 2, 1, 1300, 1, 0.0, False),      # mask routes nothing to INT8: the quantiser makes only Q
    (1, 1, 1, 100, 1, 1.0, False),       # one ragged tile
])
def test_on_the_fly_equals_quantise_once(B, hq, hk, L, G, f8, pin):
    _, _, _, once, otf = _both(B, hq, hk, L, G, seed=61, f8=f8, pin=pin)
    assert torch.equal(otf["out"].view(torch.int16), once["out"].view(torch.int16))
    assert torch.equal(otf["lse"], once["lse"])


def test_on_the_fly_against_the_oracle_with_raw_accumulators():
    import oracle
    B, hq, hk, L, G = 1, 2, 2, 700, 1
    tiles = [(0, h, m, n) for h in range(2) for m in range(6) for n in range(m + 1)]
    w, (q, k, v), route, once, otf = _both(B, hq, hk, L, G, seed=62, f8=0.5, debug_tiles=tiles)
    p = oracle.Problem(B, hq, hk, L, 128, 128, 128, G)
    qb, kb, vb = H.np_bits(q), H.np_bits(k), H.np_bits(v)
    q8, qs = oracle.quantize(qb, 128)
    k8, ks = oracle.quantize(kb, 128)
    words, _ = oracle.pack(p, route, False)
    rows = [(0, h, i) for h in range(2) for i in range(0, L, 3)]
    ref, _, _ = oracle.attention_rows(p, qb, kb, vb, q8, k8, qs, ks, words, rows)
    got = np.stack([otf["out"][b, h, i].float().cpu().numpy() for b, h, i in rows]).astype(np.float64)
    assert (np.abs(got - ref) <= H.ATOL * np.maximum(1.0, np.abs(ref))).all()
    # INT8-routed tiles: the INT32 accumulators are exactly Q8 K8^T of the oracle's quantiser output
    kind, raw = otf["kind"].cpu().numpy(), otf["raw"].cpu().numpy()
    assert np.array_equal(kind, once["kind"].cpu().numpy())
    n_int8 = 0
    for e, (b, h, m, n) in enumerate(tiles):
        if kind[e] != 1:
            continue
        n_int8 += 1
        r0, r1 = m * 128, min(L, (m + 1) * 128)
        c0, c1 = n * 128, min(L, (n + 1) * 128)
        want = q8[b, h, r0:r1].astype(np.int32) @ k8[b, h, c0:c1].astype(np.int32).T
        assert np.array_equal(raw[e, : r1 - r0, : c1 - c0], want), (m, n)
    assert n_int8 > 5


def test_on_the_fly_zero_blocks_and_large_magnitudes():
    def transform(q, k, v):
        q, k = q.clone(), k.clone()
        k[:, :, 128:256] = 0          # a zero key block: delta_K = 0
        q[:, 0, 256:384] = 0          # a zero query block
        k[:, :, 300:310] *= 200.0     # large magnitudes in one block
        q[:, :, 5] *= 64.0
        return q, k, v
    _, _, _, once, otf = _both(1, 2, 2, 640, 1, seed=63, f8=1.0, transform=transform)
    assert torch.isfinite(otf["out"].float()).all()
    assert torch.equal(otf["out"].view(torch.int16), once["out"].view(torch.int16))


def test_on_the_fly_rejects_what_it_does_not_cover():
    from paper_2608_17336_b200 import binding as tm
    dev = torch.device("cuda:0")
    p = tm.problem(1, 1, 1, 256, 64, 64, 64, 1, flags=tm.QUANT_ON_THE_FLY)
    x = torch.zeros((1, 1, 256, 64), dtype=torch.float16, device=dev)
    words = torch.zeros((1, 1, 4, 1), dtype=torch.int32, device=dev)
    with pytest.raises(tm.TilemixError) as ei:
        tm.tilemix_attention_fwd(p, x, x, x, None, None, None, None, words)
    assert ei.value.code == tm.ERR_UNSUPPORTED
    p = tm.problem(1, 1, 1, 256, 128, 128, 128, 1, flags=tm.QUANT_ON_THE_FLY)
    x = torch.zeros((1, 1, 256, 128), dtype=torch.float16, device=dev)
    with pytest.raises(tm.TilemixError) as ei:      # the routing words are still required
        tm.tilemix_attention_fwd(p, x, x, x, None, None, None, None, None)
    assert ei.value.code == tm.ERR_NULL


@pytest.mark.parametrize("B,hq,hk", [(3, 2, 2), (1, 4, 2)])
def test_on_the_fly_through_the_host_entry_point(B, hq, hk):
    """tilemix_prefill_host with the flag set skips the quantiser pass and returns the same bytes."""
    from paper_2608_17336_b200 import binding as tm
    L, d, tile, G = 400, 128, 128, 1
    gen = torch.Generator(device="cpu").manual_seed(64 + B)
    q = torch.randn((B, hq, L, d), generator=gen).half()
    k = torch.randn((B, hk, L, d), generator=gen).half()
    v = torch.randn((B, hk, L, d), generator=gen).half()
    dev = torch.device("cuda:0")
    outs = []
    for flags in (0, tm.QUANT_ON_THE_FLY):
        p = tm.problem(B, hq, hk, L, d, tile, tile, G, flags=flags)
        route = (np.random.default_rng(6).random((1, hk, p.T_m, p.T_mask)) < 0.6).astype(np.uint8)
        arena = torch.empty(tm.tilemix_arena_size(p), dtype=torch.uint8, device=dev)
        out = torch.zeros((B, hq, L, d), dtype=torch.float16).pin_memory()
        before = tm.lib().tilemix_launch_count()
        tm.tilemix_prefill_host(p, q.pin_memory(), k.pin_memory(), v.pin_memory(), torch.from_numpy(route).pin_memory(),
                                out, arena, pin_diagonal=False)
        torch.cuda.current_stream().synchronize()
        outs.append((out.clone(), tm.lib().tilemix_launch_count() - before))
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert outs[1][1] < outs[0][1]          # no quantiser launches


def test_on_the_fly_chunked_prefill():
    """The last L_q queries of a context: the chunk's Q tiles and the context's K tiles are quantised on chip."""
    from paper_2608_17336_b200 import binding as tm
    L, Lq, hq, hk, G = 1100, 332, 4, 2, 2
    w = synth.Workload("otfc", 1, hq, L, 128, 128, G, seed=65, routing="bernoulli", int8_fraction=0.7)
    q, k, v = synth.make_qkv(w)
    k, v = k[:, :hk].contiguous(), v[:, :hk].contiguous()
    route = np.ascontiguousarray(synth.make_route(w)[:, :hk])
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    p_full = tm.problem(1, hq, hk, L, 128, 128, 128, G)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p_full, qd, kd)
    words, _ = tm.tilemix_pack_routing_mask(p_full, torch.from_numpy(route).to(dev), False)
    full = tm.tilemix_attention_fwd(p_full, qd, kd, vd, q8, k8, qs, ks, words, want_lse=True)
    off = L - Lq
    pc = tm.problem(1, hq, hk, Lq, 128, 128, 128, G, flags=tm.QUANT_ON_THE_FLY)
    res = tm.tilemix_attention_fwd_chunk(pc, L, qd[:, :, off:].contiguous(), kd, vd, None, None, None, None, words,
                                         want_lse=True)
    code, rec = tm.tilemix_read_status(res["workspace"])
    assert code == 0, rec
    assert torch.equal(res["out"].view(torch.int16), full["out"][:, :, off:].contiguous().view(torch.int16))
    assert torch.equal(res["lse"], full["lse"][:, :, off:])


def test_on_the_fly_quantiser_on_ties_and_awkward_scales():
    """The on-chip quantiser forms the IEEE quotient by refinement instead of a division; the quantise-once kernel
    falls back to a true division near ties.  Inputs that sit exactly on ties (x / delta = k + 1/2), one binary16
    step next to them, and blocks whose maximum gives awkward reciprocals must come out the same, code for code:
    checked through the raw INT32 accumulators of every tile and the outputs."""
    from paper_2608_17336_b200 import binding as tm
    L, d, H = 512, 128, 2
    rng = np.random.default_rng(66)
    def block(amax, kind):
        x = np.zeros((128, d), np.float16)
        ks = rng.integers(0, 127, size=(128, d)).astype(np.float32)
        sign = rng.choice([-1.0, 1.0], size=(128, d)).astype(np.float32)
        delta = np.float32(amax) / np.float32(127)
        if kind == "tie":            # exact ties when delta is a power of two times something exact in binary16
            v = (ks + 0.5) * delta
        elif kind == "near":         # one binary16 step above / below a tie
            v = np.nextafter(((ks + 0.5) * delta).astype(np.float16), np.float16(np.inf) * rng.choice([-1, 1], size=(128, d)).astype(np.float16)).astype(np.float32)
        else:
            v = rng.standard_normal((128, d)).astype(np.float32) * amax / 4
        x[:] = np.clip(sign * v, -amax, amax).astype(np.float16)
        x[0, 0] = np.float16(amax)   # pins the block maximum
        return x
    recipe = [(127.0, "tie"), (63.5, "tie"), (127.0, "near"), (1.0, "near"), (3.0, "rand"), (0.3337, "near"),
              (1000.0, "tie"), (6.1e-5, "rand")]
    def tensor():
        t = np.zeros((1, H, L, d), np.float16)
        for h in range(H):
            for blk in range(L // 128):
                amax, kind = recipe[(h * 4 + blk) % len(recipe)]
                t[0, h, blk * 128:(blk + 1) * 128] = block(amax, kind)
        return torch.from_numpy(t)
    q, k = tensor(), tensor()
    v = torch.from_numpy(rng.standard_normal((1, H, L, d)).astype(np.float16))
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    p = tm.problem(1, H, H, L, d, 128, 128, 1, softmax_scale=1e-4)
    q8, k8, qs, ks_ = tm.tilemix_quantize_qk(p, qd, kd)
    route = np.ones((1, H, p.T_m, p.T_mask), np.uint8)
    words, _ = tm.tilemix_pack_routing_mask(p, torch.from_numpy(route).to(dev), False)
    tiles = [(0, h, m, n) for h in range(H) for m in range(4) for n in range(m + 1)]
    once = tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks_, words, debug_tiles=tiles)
    po = tm.problem(1, H, H, L, d, 128, 128, 1, softmax_scale=1e-4, flags=tm.QUANT_ON_THE_FLY)
    otf = tm.tilemix_attention_fwd(po, qd, kd, vd, None, None, None, None, words, debug_tiles=tiles)
    assert tm.tilemix_read_status(otf["workspace"])[0] == 0
    assert torch.equal(otf["raw"], once["raw"])
    assert torch.equal(otf["out"].view(torch.int16), once["out"].view(torch.int16))
    # and the codes are the definition's: raw accumulators against the oracle quantiser
    import oracle
    q8o, _ = oracle.quantize(H_np(q), 128)
    k8o, _ = oracle.quantize(H_np(k), 128)
    raw = otf["raw"].cpu().numpy()
    for e, (b, h, m, n) in enumerate(tiles):
        want = q8o[b, h, m * 128:(m + 1) * 128].astype(np.int32) @ k8o[b, h, n * 128:(n + 1) * 128].astype(np.int32).T
        assert np.array_equal(raw[e], want), (h, m, n)


def H_np(t):
    return H.np_bits(t)


def test_on_the_fly_with_the_mask_ignored():
    """TILEMIX_FORCE_FP16 on top of the on-the-fly flag: nothing is quantised, the result is the all-FP16 one."""
    from paper_2608_17336_b200 import binding as tm
    w = synth.Workload("otf16", 1, 2, 700, 128, 128, 1, seed=67)
    q, k, v = synth.make_qkv(w)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    outs = []
    for flags in (tm.FORCE_FP16, tm.FORCE_FP16 | tm.QUANT_ON_THE_FLY):
        p = tm.problem(1, 2, 2, 700, 128, 128, 128, 1, flags=flags)
        res = tm.tilemix_attention_fwd(p, qd, kd, vd, None, None, None, None, None)
        assert tm.tilemix_read_status(res["workspace"])[0] == 0
        outs.append(res["out"])
    assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))
