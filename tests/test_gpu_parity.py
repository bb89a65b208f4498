"""Parity of the CUDA path (through the C ABI) with the CPU oracle on the same seeded inputs:
bit-exact for INT8 operands, scales, packed words, counters and INT32 score accumulators;
FP16 outputs within 2e-3 * max(1, |O|)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_17336_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2608_17336_b200 import binding
    return binding


def _small(name, **kw):
    base = dict(name=name, batch=1, heads=2, seqlen=640, head_dim=128, tile=128, group=1, seed=11,
                routing="bernoulli", int8_fraction=0.5)
    base.update(kw)
    return synth.Workload(**base)


# ------------------------------------------------------------------------------ quantiser

@pytest.mark.parametrize("B,Hh,L,d,blk", [(1, 2, 640, 128, 128), (2, 3, 1000, 128, 128), (1, 1, 1024, 64, 64),
                                         (1, 2, 100, 64, 64), (1, 1, 777, 128, 64), (1, 2, 300, 32, 16)])
def test_quantize_bit_exact(B, Hh, L, d, blk):
    b = _binding()
    gen = torch.Generator().manual_seed(L + d)
    q = (torch.randn((B, Hh, L, d), generator=gen) * 3).half()
    k = torch.randn((B, Hh, L, d), generator=gen).half()
    k[0, 0, : min(L, 2 * blk)] = 0          # zero blocks
    p = b.problem(B, Hh, Hh, L, d, blk, blk)
    q8, k8, qs, ks = b.tilemix_quantize_qk(p, q.cuda(), k.cuda())
    for x, x8, xs in ((q, q8, qs), (k, k8, ks)):
        r8, rs = oracle.quantize(H.np_bits(x), blk)
        assert (x8.cpu().numpy() == r8).all()
        assert (xs.cpu().numpy().view(np.uint32) == rs.view(np.uint32)).all()


@pytest.mark.parametrize("B,Hq,Hk,L,d,blk_q,blk_k", [(2, 8, 2, 3000, 128, 128, 64), (1, 4, 1, 20000, 128, 128, 128),
                                                     (3, 2, 1, 130, 64, 64, 64)])
def test_quantize_pair_of_different_shapes_in_one_launch(B, Hq, Hk, L, d, blk_q, blk_k):
    """Q and K with different head counts and block sizes (grouped-query attention, the paper's BLK_K = BLOCK_N / 2)
    go through one launch of the streaming quantiser; more blocks than the persistent CTAs take in one round; a
    ragged last block; values on rounding ties (multiples of 1/2 scaled so that x / delta hits .5)."""
    b = _binding()
    gen = torch.Generator().manual_seed(L + Hq)
    q = (torch.randint(-254, 255, (B, Hq, L, d), generator=gen).float() * 0.5).half()      # max |x| = 127 -> delta = 1: ties
    q[:, :, 0, 0] = 127.0
    k = (torch.randn((B, Hk, L, d), generator=gen) * 2).half()
    p = b.problem(B, Hq, Hk, L, d, max(blk_q, blk_k), max(blk_q, blk_k), quant_blk_q=blk_q, quant_blk_k=blk_k)
    q8, k8, qs, ks = b.tilemix_quantize_qk(p, q.cuda(), k.cuda())
    for x, x8, xs, blk in ((q, q8, qs, blk_q), (k, k8, ks, blk_k)):
        r8, rs = oracle.quantize(H.np_bits(x), blk)
        assert (x8.cpu().numpy() == r8).all()
        assert (xs.cpu().numpy().view(np.uint32) == rs.view(np.uint32)).all()


def test_quantize_strided_input():
    b = _binding()
    B, Hh, L, d = 2, 3, 384, 128
    gen = torch.Generator().manual_seed(5)
    packed = torch.randn((B, L, 3, Hh, d), generator=gen).half().cuda()    # a fused QKV projection output
    q = packed[:, :, 0].permute(0, 2, 1, 3)                                # [B, H, L, d] view, d contiguous
    k = packed[:, :, 1].permute(0, 2, 1, 3)
    p = b.problem(B, Hh, Hh, L, d, 128, 128)
    q8, k8, qs, ks = b.tilemix_quantize_qk(p, q, k)
    r8, rs = oracle.quantize(H.np_bits(q.contiguous().cpu()), 128)
    assert (q8.cpu().numpy() == r8).all() and (qs.cpu().numpy() == rs).all()
    r8, rs = oracle.quantize(H.np_bits(k.contiguous().cpu()), 128)
    assert (k8.cpu().numpy() == r8).all() and (ks.cpu().numpy() == rs).all()


# ------------------------------------------------------------------------------ packer

@pytest.mark.parametrize("L,tile,G,nb,pin", [(1024, 64, 1, 1, False), (8192, 128, 1, 1, False), (32768, 128, 4, 1, True),
                                             (4096, 128, 2, 2, False), (131072, 128, 8, 1, False), (1000, 128, 3, 1, True),
                                             (100, 64, 1, 1, True)])
def test_pack_bit_exact(L, tile, G, nb, pin):
    b = _binding()
    Hk = 3
    p = b.problem(nb, Hk, Hk, L, tile, tile, tile, G, mask_batch=nb)
    rng = np.random.default_rng(L + G)
    route = (rng.random((nb, Hk, p.T_m, p.T_mask)) < 0.7).astype(np.uint8) * rng.integers(1, 255, 1, dtype=np.uint8)
    words, counts = b.tilemix_pack_routing_mask(p, torch.from_numpy(route).cuda(), pin)
    po = oracle.Problem(nb, Hk, Hk, L, tile, tile, tile, G, mask_batch=nb)
    rw, rc = oracle.pack(po, route, pin)
    assert (words.cpu().numpy().view(np.uint32) == rw).all()
    assert (counts.cpu().numpy().astype(np.uint64) == rc).all()


# ------------------------------------------------------------------------------ attention

def _full_check(w, debug=True, atol=H.ATOL):
    q, k, v = synth.make_qkv(w)
    route = synth.make_route(w)
    heads = list(range(w.heads))
    rows = H.all_rows(w)
    ref = H.run_oracle(w, q, k, v, route, heads, rows)
    tiles = None
    if debug:
        tiles = [(b, h, m, n) for b in range(w.batch) for h in heads for m in range(w.T_m) for n in range(m + 1)]
    res = H.run_gpu(w, q, k, v, route, debug_tiles=tiles)
    # bit-exact parts
    assert (res["q8"].cpu().numpy() == ref["q8"]).all() and (res["k8"].cpu().numpy() == ref["k8"]).all()
    assert (res["qs"].cpu().numpy() == ref["qs"]).all() and (res["ks"].cpu().numpy() == ref["ks"]).all()
    assert (res["words"].cpu().numpy().view(np.uint32) == ref["words"]).all()
    assert (res["counts"].cpu().numpy().astype(np.uint64) == ref["counts"]).all()
    if debug:
        raw = res["raw"].cpu().numpy()
        kind = res["kind"].cpu().numpy()
        po = ref["p"]
        n_int8 = 0
        for e, (b, h, m, n) in enumerate(tiles):
            g = n // w.group
            nbi = 0 if w.mask_batch == 1 else b
            bit = (int(ref["words"][nbi, h, m, g >> 5]) >> (g & 31)) & 1
            assert kind[e] == bit, (b, h, m, n, kind[e], bit)
            if bit:
                n_int8 += 1
                exp = oracle.int32_tile(po, ref["q8"], ref["k8"], b, h, m, n)
                assert (raw[e] == exp).all(), f"INT32 accumulator tile {(b, h, m, n)} differs"
            else:
                exp = oracle.fp_tile(po, ref["qb"], ref["kb"], b, h, m, n)
                got = raw[e].view(np.float32).astype(np.float64)
                assert np.abs(got - exp).max() <= 1e-3 * max(1.0, np.abs(exp).max()), (b, h, m, n)
        assert w.routing in ("zero",) or n_int8 > 0
    err = H.check_rows(res["out"], ref["out"], rows, atol)
    lse = res["lse"].cpu().numpy().astype(np.float64).reshape(-1)
    assert np.abs(lse - ref["lse"]).max() < 2e-3
    return err


def test_attention_cfg1_tiny_all_rows_all_int32_tiles():
    """Config 1 in full: every row against the oracle, all 136 raw accumulator tiles bit-exact."""
    _full_check(synth.WORKLOADS["cfg1_tiny"])


@pytest.mark.parametrize("routing,frac", [("zero", 0.0), ("one", 1.0), ("bernoulli", 0.5)])
def test_attention_small_d128(routing, frac):
    _full_check(_small("s128", routing=routing, int8_fraction=frac))


def test_attention_odd_tile_count_grouped_mask():
    _full_check(_small("odd", seqlen=896, group=2, heads=1, seed=12))          # 7 tiles: last pair has no B


def test_attention_ragged_tail():
    _full_check(_small("ragged", seqlen=1000, group=3, seed=13, pin_diagonal=True))
    _full_check(_small("ragged64", seqlen=333, head_dim=64, tile=64, group=2, seed=14))


def test_attention_single_partial_tile():
    _full_check(_small("one_tile", seqlen=100, heads=1, seed=15, routing="one"))
    _full_check(_small("one_tile16", seqlen=100, heads=1, seed=15, routing="zero"))
    _full_check(_small("one_row", seqlen=1, heads=1, seed=16, routing="one"))


def test_attention_batched_mask_per_batch_and_outliers():
    _full_check(_small("batched", batch=2, heads=2, seqlen=512, mask_batch=2, values="outlier_channels", seed=17))


@pytest.mark.parametrize("seed,heads,L,G,frac", [(101, 4, 1536, 1, 0.5), (102, 3, 2048, 2, 0.8), (103, 2, 2304, 3, 0.2),
                                                  (104, 4, 1280, 1, 0.65), (105, 1, 4096, 4, 0.75)])
def test_attention_fast_path_many_routing_patterns(seed, heads, L, G, frac):
    """No debug request, so interior tiles take the one-pass path; every row against the oracle.  The mixes
    make the two query tiles of a CTA disagree on many key tiles (both copies of K staged)."""
    _full_check(_small(f"mix{seed}", seed=seed, heads=heads, seqlen=L, group=G, int8_fraction=frac), debug=False)
    _full_check(_small(f"mix64_{seed}", seed=seed, heads=heads, seqlen=L // 2, head_dim=64, tile=64, group=G,
                       int8_fraction=frac), debug=False)


@pytest.mark.parametrize("layout", ["band", "global", "aligned_sparse", "bigbird", "sptrans"])
def test_attention_structured_layouts(layout):
    """The paper's structured precision layouts at 50 % coverage, packed and run; all rows vs the oracle."""
    from paper_2608_17336_b200 import policy
    b = _binding()
    w = _small(f"layout_{layout}", seqlen=2048, heads=2, group=2, seed=71)
    geo, R, info = policy.template(w.seqlen, w.tile, w.tile, layout, 0.5, group=w.group)
    route = policy.broadcast(R, w.heads)
    q, k, v = synth.make_qkv(w)
    rows = H.all_rows(w)
    ref = H.run_oracle(w, q, k, v, route, range(w.heads), rows)
    res = H.run_gpu(w, q, k, v, route)
    assert (res["words"].cpu().numpy().view(np.uint32) == ref["words"]).all()
    cov = ref["counts"][..., 1].sum() / ref["counts"][..., 0].sum()
    assert abs(cov - info["coverage"]) < 1e-12
    H.check_rows(res["out"], ref["out"], rows)


def test_attention_growing_scores_move_the_running_maximum():
    """Keys whose magnitude grows along the sequence: later tiles keep exceeding the running maximum, so
    interior tiles are redone with a new maximum and the output accumulator is rescaled many times."""
    b = _binding()
    w = _small("ramp", seqlen=2048, heads=2, seed=61, int8_fraction=0.5)
    q, k, v = synth.make_qkv(w)
    ramp = torch.linspace(0.25, 6.0, w.seqlen).view(1, 1, -1, 1)
    k = (k.float() * ramp).half()
    q = (q.float() * 1.5).half()
    route = synth.make_route(w)
    rows = H.all_rows(w)
    ref = H.run_oracle(w, q, k, v, route, range(w.heads), rows)
    res = H.run_gpu(w, q, k, v, route)
    H.check_rows(res["out"], ref["out"], rows)
    lse = res["lse"].cpu().numpy().astype(np.float64).reshape(-1)
    assert np.abs(lse - ref["lse"]).max() < 2e-3 * max(1.0, np.abs(ref["lse"]).max())


def test_attention_force_fp16_without_int8_operands():
    b = _binding()
    w = _small("force16", routing="zero", seqlen=512)
    q, k, v = synth.make_qkv(w)
    p = H.gpu_problem(w, flags=b.FORCE_FP16)
    res = b.tilemix_attention_fwd(p, q.cuda(), k.cuda(), v.cuda())
    assert b.tilemix_read_status(res["workspace"])[0] == 0
    rows = H.all_rows(w)
    ref = H.run_oracle(w, q, k, v, synth.make_route(w), range(w.heads), rows)
    H.check_rows(res["out"], ref["out"], rows)


def test_attention_gqa_heads_share_kv_and_mask():
    """H_q = 4, H_k = 2: h_k = floor(h_q / 2) indexes K, V, K8, scales and the routing words."""
    b = _binding()
    B, Hq, Hk, L, d, tile = 1, 4, 2, 512, 128, 128
    gen = torch.Generator().manual_seed(21)
    q = torch.randn((B, Hq, L, d), generator=gen).half()
    k = torch.randn((B, Hk, L, d), generator=gen).half()
    v = torch.randn((B, Hk, L, d), generator=gen).half()
    p = b.problem(B, Hq, Hk, L, d, tile, tile, 1)
    po = oracle.Problem(B, Hq, Hk, L, d, tile, tile, 1)
    route = (np.random.default_rng(3).random((1, Hk, po.T_m, po.T_mask)) < 0.5).astype(np.uint8)
    q8, k8, qs, ks = b.tilemix_quantize_qk(p, q.cuda(), k.cuda())
    words, _ = b.tilemix_pack_routing_mask(p, torch.from_numpy(route).cuda())
    res = b.tilemix_attention_fwd(p, q.cuda(), k.cuda(), v.cuda(), q8, k8, qs, ks, words)
    assert b.tilemix_read_status(res["workspace"])[0] == 0
    oq8, oqs = oracle.quantize(H.np_bits(q), tile)
    ok8, oks = oracle.quantize(H.np_bits(k), tile)
    ow, _ = oracle.pack(po, route)
    ref, _, _ = oracle.attention_full(po, H.np_bits(q), H.np_bits(k), H.np_bits(v), oq8, ok8, oqs, oks, ow)
    err = np.abs(res["out"].float().cpu().numpy() - ref)
    assert (err <= H.ATOL * np.maximum(1, np.abs(ref))).all(), err.max()


def test_attention_strided_qkv_views():
    b = _binding()
    B, Hh, L, d = 1, 2, 512, 128
    gen = torch.Generator().manual_seed(23)
    packed = torch.randn((B, L, 3, Hh, d), generator=gen).half()
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    w = _small("strided", seqlen=L, heads=Hh)
    route = synth.make_route(w)
    p = H.gpu_problem(w)
    pd = packed.cuda()
    qd, kd, vd = (pd[:, :, i].permute(0, 2, 1, 3) for i in range(3))
    q8, k8, qs, ks = b.tilemix_quantize_qk(p, qd, kd)
    words, _ = b.tilemix_pack_routing_mask(p, torch.from_numpy(route).cuda())
    res = b.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words)
    assert b.tilemix_read_status(res["workspace"])[0] == 0
    rows = H.all_rows(w)
    ref = H.run_oracle(w, q.contiguous(), k.contiguous(), v.contiguous(), route, range(Hh), rows)
    H.check_rows(res["out"], ref["out"], rows)


def test_lossless_inputs_every_mask_equals_fp16():
    """Q, K on the grid {-127..127}/64 with +-127/64 in every block quantise exactly, so every
    routing map must reproduce the all-FP16 result (up to summation order)."""
    b = _binding()
    w = _small("lossless", seqlen=768, heads=1, group=2)
    gen = torch.Generator().manual_seed(31)
    shape = (1, 1, w.seqlen, 128)
    q = torch.randint(-127, 128, shape, generator=gen).float()
    k = torch.randint(-127, 128, shape, generator=gen).float()
    q[..., ::128, 0] = 127; k[..., ::128, 0] = -127
    q, k = (q / 64).half(), (k / 64).half()
    v = torch.randn(shape, generator=gen).half()
    outs = []
    for routing in ("zero", "one", "bernoulli"):
        res = H.run_gpu(w.scaled(routing=routing), q, k, v, synth.make_route(w.scaled(routing=routing)))
        assert (res["qs"] == 1 / 64).all() and (res["ks"] == 1 / 64).all()
        outs.append(res["out"].float())
    assert (outs[0] - outs[1]).abs().max() < 1e-3 and (outs[0] - outs[2]).abs().max() < 1e-3


def test_two_runs_are_bit_identical():
    w = _small("repeat", seqlen=1024, heads=2)
    q, k, v = synth.make_qkv(w)
    route = synth.make_route(w)
    a = H.run_gpu(w, q, k, v, route)["out"]
    c = H.run_gpu(w, q, k, v, route)["out"]
    assert torch.equal(a, c)


# ------------------------------------------------------------------------------ full-size configs

FULL = [
    ("cfg2_llama8k", dict(routing="zero"), 2, 1, 8),
    ("cfg2_llama8k", dict(), 2, 1, 8),
    ("cfg2_llama8k", dict(routing="one"), 2, 1, 8),
    ("cfg3_long32k", dict(), 2, 0, 8),
    ("cfg4_batched4k", dict(), 3, 1, 8),
    ("cfg5_verylong128k", dict(), 2, 0, 6),
]


@pytest.mark.parametrize("name,override,n_heads,n_tiles,n_rows", FULL)
def test_full_size_config_sampled_rows(name, override, n_heads, n_tiles, n_rows):
    """The five configurations at full size, in the launch configuration the bench times; the oracle
    evaluates sampled rows of a few heads (first and last query tile, random tiles, random rows)."""
    w = synth.WORKLOADS[name].scaled(**override)
    q, k, v = synth.make_qkv(w)
    route = synth.make_route(w)
    # The kernel's grid interleaves the (batch, head) rows in groups of up to eight: take heads at every position
    # of such a group (0, 1, ..., the last of a group of 4 and of 8, the first of the next group, the last head).
    heads = sorted({h for h in (0, 1, 2, 3, 5, 7, 8, w.heads // 2 + 1, w.heads - 1) if h < w.heads})
    heads = heads[:max(n_heads, 1)] if w.seqlen > 40000 else heads
    rows = synth.sample_rows(w, n_random_tiles=n_tiles, n_random_rows=n_rows, heads=heads)
    if w.seqlen > 40000:
        # the longest configuration: a few rows of the last tile, and rows spread over the whole sequence (the
        # oracle costs O(i d) per row)
        keep = (rows[:, 2] < w.seqlen - w.tile) | (rows[:, 2] % 16 == 15)
        spread = np.asarray([(0, h, int(i)) for h in heads for i in np.linspace(w.tile, w.seqlen - 1, 160).astype(np.int64)], np.int64)
        rows = np.concatenate([rows[keep], spread])
    if w.batch > 1:
        rows = rows[(rows[:, 0] == 0) | (rows[:, 0] == w.batch - 1)]
    res = H.run_gpu(w, q, k, v, route, want_lse=False)
    ref = H.run_oracle(w, q, k, v, route, heads, [tuple(r) for r in rows])
    sub = torch.as_tensor(heads)
    assert (res["q8"][:, sub].cpu().numpy() == ref["q8"]).all() and (res["k8"][:, sub].cpu().numpy() == ref["k8"]).all()
    assert (res["qs"][:, sub].cpu().numpy() == ref["qs"]).all() and (res["ks"][:, sub].cpu().numpy() == ref["ks"]).all()
    assert (res["words"][:, sub].cpu().numpy().view(np.uint32) == ref["words"]).all()
    H.check_rows(res["out"], ref["out"], rows)
    # properties that hold at any size: finite outputs, |O| bounded by max |V| of the head
    out = res["out"]
    assert torch.isfinite(out).all()
    vmax = v.abs().amax(dim=(2, 3)).cuda()
    assert (out.abs().amax(dim=(2, 3)) <= vmax * (1 + 1e-2)).all()


@pytest.mark.parametrize("B,Hq,Hk,nb", [(1, 12, 6, 1), (1, 20, 10, 1), (3, 4, 2, 1), (11, 2, 2, 11)])
def test_prefill_host_equals_device_path(B, Hq, Hk, nb):
    """The host-buffer entry point (chunks pipelined over helper streams) returns, bit for bit, what
    the three device calls return; more than eight chunk units, GQA, shared and per-batch masks."""
    from paper_2608_17336_b200 import binding
    L, d, tile, G = 300, 64, 64, 2
    gen = torch.Generator(device="cpu").manual_seed(77 + B)
    q = torch.randn((B, Hq, L, d), generator=gen).half()
    k = torch.randn((B, Hk, L, d), generator=gen).half()
    v = torch.randn((B, Hk, L, d), generator=gen).half()
    p = binding.problem(B, Hq, Hk, L, d, tile, tile, G, mask_batch=nb)
    rng = np.random.default_rng(5)
    route = (rng.random((nb, Hk, p.T_m, p.T_mask)) < 0.5).astype(np.uint8)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    q8, k8, qs, ks = binding.tilemix_quantize_qk(p, qd, kd)
    words, _ = binding.tilemix_pack_routing_mask(p, torch.from_numpy(route).to(dev), True)
    ref = binding.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words)["out"].cpu()
    arena = torch.empty(binding.tilemix_arena_size(p), dtype=torch.uint8, device=dev)
    out = torch.empty((B, Hq, L, d), dtype=torch.float16).pin_memory()
    for _ in range(2):     # a second call right behind the first reuses the helper streams and the arena
        out.zero_()
        binding.tilemix_prefill_host(p, q.pin_memory(), k.pin_memory(), v.pin_memory(),
                                     torch.from_numpy(route).pin_memory(), out, arena, pin_diagonal=True)
        torch.cuda.current_stream().synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_prefill_host_from_two_threads_on_two_streams():
    """Two host threads, each with its own stream, arena and output buffer, call the host-buffer entry point
    at the same time, several times over: a call holds the library's per-device lock while it enqueues, so the
    calls never interleave on the shared helper streams and every output equals the single-threaded result."""
    import threading
    from paper_2608_17336_b200 import binding
    dev = torch.device("cuda:0")
    L, d, tile, G = 700, 128, 128, 1
    jobs = []
    for i, (B, Hq, Hk) in enumerate([(1, 12, 6), (3, 4, 2)]):
        gen = torch.Generator(device="cpu").manual_seed(300 + i)
        q = torch.randn((B, Hq, L, d), generator=gen).half().pin_memory()
        k = torch.randn((B, Hk, L, d), generator=gen).half().pin_memory()
        v = torch.randn((B, Hk, L, d), generator=gen).half().pin_memory()
        p = binding.problem(B, Hq, Hk, L, d, tile, tile, G)
        route = torch.from_numpy((np.random.default_rng(9 + i).random((1, Hk, p.T_m, p.T_mask)) < 0.5).astype(np.uint8)).pin_memory()
        arena = torch.empty(binding.tilemix_arena_size(p), dtype=torch.uint8, device=dev)
        out = torch.empty((B, Hq, L, d), dtype=torch.float16).pin_memory()
        binding.tilemix_prefill_host(p, q, k, v, route, out, arena)
        torch.cuda.synchronize()
        jobs.append(dict(p=p, q=q, k=k, v=v, route=route, arena=arena, out=out, ref=out.clone(), stream=torch.cuda.Stream()))
    errors = []

    def work(job):
        try:
            with torch.cuda.stream(job["stream"]):
                for _ in range(6):
                    job["out"].zero_()
                    binding.tilemix_prefill_host(job["p"], job["q"], job["k"], job["v"], job["route"], job["out"], job["arena"])
                    job["stream"].synchronize()
                    if not torch.equal(job["out"].view(torch.int16), job["ref"].view(torch.int16)):
                        errors.append("output differs")
        except Exception as exc:       # noqa: BLE001
            errors.append(repr(exc))

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for th in threads: th.start()
    for th in threads: th.join()
    assert not errors, errors


@pytest.mark.parametrize("seed", [101, 102, 103])
def test_attention_random_shapes(seed):
    """Random dense cases -- batch, GQA ratio, length (ragged), tile, group, INT8 share, pin, value recipe, shared or
    per-batch mask -- through the whole path: quantiser and packer bit-exact, sampled rows against the oracle."""
    from paper_2608_17336_b200 import binding as tm
    rng = np.random.default_rng(seed)
    dev = torch.device("cuda:0")
    for it in range(8):
        tile = int(rng.choice([64, 128]))
        hk = int(rng.choice([1, 2]))
        hq = hk * int(rng.choice([1, 2, 4]))
        B = int(rng.choice([1, 2, 3]))
        L = int(rng.integers(1, 9 * tile))
        G = int(rng.choice([1, 2, 3, 5]))
        f8 = float(rng.choice([0.0, 0.3, 0.5, 0.8, 1.0]))
        pin = bool(rng.integers(0, 2))
        mb = int(rng.choice([1, B]))
        w = synth.Workload("rnd", B, hq, L, tile, tile, G, seed=seed * 100 + it,
                           values=str(rng.choice(["normal", "outlier_channels", "student_t_k"])),
                           routing=str(rng.choice(["bernoulli", "row_exact"])), int8_fraction=f8, pin_diagonal=pin,
                           mask_batch=mb)
        q, k, v = synth.make_qkv(w)
        k, v = k[:, :hk].contiguous(), v[:, :hk].contiguous()
        route = np.ascontiguousarray(synth.make_route(w)[:, :hk])
        qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
        p = tm.problem(B, hq, hk, L, tile, tile, tile, G, mask_batch=mb)
        q8, k8, qs, ks = tm.tilemix_quantize_qk(p, qd, kd)
        words, _ = tm.tilemix_pack_routing_mask(p, torch.from_numpy(route).to(dev), pin)
        res = tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words)
        code, rec = tm.tilemix_read_status(res["workspace"])
        assert code == 0, rec
        po = oracle.Problem(B, hq, hk, L, tile, tile, tile, G, mask_batch=mb)
        qb, kb, vb = H.np_bits(q), H.np_bits(k), H.np_bits(v)
        q8o, qso = oracle.quantize(qb, tile)
        k8o, kso = oracle.quantize(kb, tile)
        assert np.array_equal(q8.cpu().numpy(), q8o) and np.array_equal(k8.cpu().numpy(), k8o)
        wo, _ = oracle.pack(po, route, pin)
        assert np.array_equal(words.cpu().numpy().view(np.uint32), wo)
        rows = [(b, h, int(i)) for b in range(B) for h in range(hq)
                for i in rng.choice(L, size=min(L, 8), replace=False)]
        ref, _, _ = oracle.attention_rows(po, qb, kb, vb, q8o, k8o, qso, kso, wo, rows)
        got = np.stack([res["out"][b, h, i].float().cpu().numpy() for b, h, i in rows]).astype(np.float64)
        assert (np.abs(got - ref) <= H.ATOL * np.maximum(1.0, np.abs(ref))).all(), (it, B, hq, hk, L, tile, G, f8, pin)
