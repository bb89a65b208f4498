"""Decode step over an INT8 key/value cache on the GPU against the float64 oracle: the quantised
query bit-exact, outputs and LSE within tolerance."""
import numpy as np
import pytest
import torch

import oracle
from oracle import decode as od
from tests.helpers import ATOL

pytestmark = pytest.mark.gpu


def _case(B, Hq, Hk, L, d, tile, G, seed, lens, f8=0.5, mask_batch=1):
    gen = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, Hq, d), generator=gen).half()
    k = torch.randn((B, Hk, L, d), generator=gen).half()
    v = torch.randn((B, Hk, L, d), generator=gen).half()
    rng = np.random.default_rng(seed + 1)
    T_mask = -(-L // (tile * G))
    route = (rng.random((mask_batch, Hk, T_mask)) < f8).astype(np.uint8)
    return q, k, v, route, np.asarray(lens, np.int32)


def _gpu(q, k, v, route, lens, tile, G, n_splits=0, k16_none=False):
    from paper_2608_17336_b200 import binding as tm
    dev = torch.device("cuda:0")
    B, Hq, d = q.shape
    Hk, L = k.shape[1], k.shape[2]
    # the cache is quantised with the library's own blockwise quantiser (K and V as its two operands)
    pq = tm.problem(B, Hk, Hk, L, d, tile, tile)
    kd, vd = k.to(dev), v.to(dev)
    k8, v8, ks, vs = tm.tilemix_quantize_qk(pq, kd, vd)
    p = tm.decode_problem(B, Hq, Hk, d, L, tile, G, mask_batch=route.shape[0], n_splits=n_splits)
    words = torch.from_numpy(od.pack_row(route).view(np.int32)).to(dev)
    res = tm.tilemix_decode_int8kv(p, q.to(dev), None if k16_none else kd, k8, ks, v8, vs, words,
                                   torch.from_numpy(lens).to(dev), want_lse=True, want_q8=True)
    torch.cuda.synchronize()
    return res, dict(k8=k8.cpu().numpy(), ks=ks.cpu().numpy(), v8=v8.cpu().numpy(), vs=vs.cpu().numpy())


def _check(q, k, v, route, lens, tile, G, **kw):
    res, cache = _gpu(q, k, v, route, lens, tile, G, **kw)
    q16 = np.ascontiguousarray(q.view(torch.int16).numpy()).view(np.uint16)
    k16 = np.ascontiguousarray(k.view(torch.int16).numpy()).view(np.uint16)
    # the cache itself: the library quantiser against the oracle's (bit-exact)
    k8_ref, ks_ref = oracle.quantize(k16, tile)
    assert np.array_equal(cache["k8"], k8_ref) and np.array_equal(cache["ks"].view(np.uint32), ks_ref.view(np.uint32))
    v16 = np.ascontiguousarray(v.view(torch.int16).numpy()).view(np.uint16)
    v8_ref, vs_ref = oracle.quantize(v16, tile)      # the V cache too, before the oracle is given it
    assert np.array_equal(cache["v8"], v8_ref) and np.array_equal(cache["vs"].view(np.uint32), vs_ref.view(np.uint32))
    q8_ref, dq_ref = od.quantize_query(q16)
    assert np.array_equal(res["q8"].cpu().numpy(), q8_ref)
    assert np.array_equal(res["q_scale"].cpu().numpy().view(np.uint32), dq_ref.view(np.uint32))
    ref, ref_lse = od.decode(q16, k16, cache["k8"], cache["ks"], cache["v8"], cache["vs"], od.pack_row(route), lens,
                             tile, G)
    out = res["out"].float().cpu().numpy().astype(np.float64)
    err = np.abs(out - ref)
    assert (err <= ATOL * np.maximum(1.0, np.abs(ref))).all(), f"max err {err.max():.3e}"
    lse = res["lse"].cpu().numpy().astype(np.float64)
    live = lens > 0
    assert np.abs(lse[live] - ref_lse[live]).max() < 2e-3
    assert np.isneginf(lse[~live]).all() and not out[~live].any()
    return float(err.max())


def test_decode_gqa4_d128():
    q, k, v, route, lens = _case(3, 8, 2, 1500, 128, 128, 2, seed=21, lens=[1500, 777, 129])
    _check(q, k, v, route, lens, 128, 2)


def test_decode_small_tiles_mha_edge_lengths():
    q, k, v, route, lens = _case(5, 2, 2, 300, 64, 64, 1, seed=22, lens=[300, 1, 0, 64, 65])
    _check(q, k, v, route, lens, 64, 1)


@pytest.mark.parametrize("rep", [1, 2, 8])
def test_decode_group_sizes(rep):
    q, k, v, route, lens = _case(2, 2 * rep, 2, 900, 128, 64, 3, seed=23 + rep, lens=[900, 450])
    _check(q, k, v, route, lens, 64, 3)


@pytest.mark.parametrize("n_splits", [1, 3, 1000])
def test_decode_split_counts(n_splits):
    q, k, v, route, lens = _case(1, 4, 1, 2000, 64, 128, 1, seed=24, lens=[1999])
    _check(q, k, v, route, lens, 128, 1, n_splits=n_splits)


def test_decode_per_batch_mask_and_pure_routes():
    q, k, v, route, lens = _case(2, 4, 2, 700, 128, 128, 1, seed=25, lens=[700, 300], mask_batch=2)
    _check(q, k, v, route, lens, 128, 1)
    _check(q, k, v, np.zeros_like(route), lens, 128, 1)
    _check(q, k, v, np.ones_like(route), lens, 128, 1, k16_none=True)    # all INT8: no FP16 cache needed


def test_decode_keys_beyond_cache_len_are_not_read():
    q, k, v, route, lens = _case(1, 4, 1, 512, 128, 128, 1, seed=26, lens=[200])
    a, _ = _gpu(q, k, v, route, lens, 128, 1)
    k2, v2 = k.clone(), v.clone()
    k2[:, :, 256:] = 5.0       # later blocks only: the scales of the blocks in use are unchanged
    v2[:, :, 256:] = -7.0
    b_, _ = _gpu(q, k2, v2, route, lens, 128, 1)
    assert torch.equal(a["out"].view(torch.int16), b_["out"].view(torch.int16))


def test_decode_zero_query_and_zero_blocks():
    """A zero query row (delta_q = 0) and an all-zero key block (delta_K = 0): every INT8 score is 0, the
    probabilities are uniform over the cached keys, no division by zero anywhere."""
    q, k, v, route, lens = _case(2, 4, 2, 384, 128, 128, 1, seed=27, lens=[384, 200], f8=1.0)
    q[0, 1] = 0
    k[1, :, 128:256] = 0
    _check(q, k, v, route, lens, 128, 1)
    mixed = route.copy(); mixed[..., 1] = 0
    _check(q, k, v, mixed, lens, 128, 1)


def test_decode_large_magnitudes():
    """Keys and values near the top of the FP16 range in a few channels, large score spread."""
    q, k, v, route, lens = _case(1, 8, 2, 640, 128, 128, 1, seed=28, lens=[601])
    k[:, :, :, 5] *= 40.0
    q[:, :, 5] *= 6.0
    v[:, :, 100:130, 7] = 30000.0
    _check(q, k, v, route, lens, 128, 1)


@pytest.mark.parametrize("seed", [31, 32, 33])
def test_decode_random_shapes(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.choice([64, 128])); tile = int(rng.choice([64, 128])); rep = int(rng.choice([1, 2, 4, 8]))
    Hk = int(rng.integers(1, 4)); B = int(rng.integers(1, 5)); L = int(rng.integers(1, 1200)); G = int(rng.integers(1, 4))
    lens = rng.integers(0, L + 1, B).tolist()
    q, k, v, route, lens = _case(B, Hk * rep, Hk, L, d, tile, G, seed=seed, lens=lens, f8=float(rng.random()))
    _check(q, k, v, route, lens, tile, G, n_splits=int(rng.integers(0, 6)))


def test_decode_out_of_range_lengths_are_clamped():
    """cache_len lives on the device; a value above max_len acts as max_len, a negative one as 0."""
    q, k, v, route, _ = _case(3, 4, 2, 300, 128, 128, 1, seed=41, lens=[0, 0, 0])
    good, _ = _gpu(q, k, v, route, np.asarray([300, 0, 123], np.int32), 128, 1)
    bad, _ = _gpu(q, k, v, route, np.asarray([100000, -5, 123], np.int32), 128, 1)
    assert torch.equal(good["out"].view(torch.int16), bad["out"].view(torch.int16))
    assert torch.equal(good["lse"], bad["lse"])


def test_decode_without_fp16_cache_reports_an_fp16_routed_group():
    """No FP16 key cache is passed but one group inside the cache length is routed to FP16: the kernel must find
    that before it reads anything and say so in the status record (no fault); the same workspace then serves a
    correct call."""
    from paper_2608_17336_b200 import binding as tm
    dev = torch.device("cuda:0")
    q, k, v, route, lens = _case(2, 4, 2, 700, 128, 128, 1, seed=51, lens=[700, 300], f8=1.0)
    route[:] = 1
    B, Hq, d = q.shape
    Hk, L = k.shape[1], k.shape[2]
    kd, vd = k.to(dev), v.to(dev)
    k8, v8, ks, vs = tm.tilemix_quantize_qk(tm.problem(B, Hk, Hk, L, d, 128, 128), kd, vd)
    p = tm.decode_problem(B, Hq, Hk, d, L, 128, 1)
    bad = route.copy()
    bad[0, 1, 3] = 0                                     # keys 384..511 of KV head 1: inside both cache lengths? (300 < 384: batch 0 only)
    for r, want in ((bad, tm.ERR_NULL), (route, 0)):
        words = torch.from_numpy(od.pack_row(r).view(np.int32)).to(dev)
        res = tm.tilemix_decode_int8kv(p, q.to(dev), None, k8, ks, v8, vs, words, torch.from_numpy(lens).to(dev))
        code, rec = tm.tilemix_read_status(res["workspace"])
        assert code == want, rec
    # a 0 bit beyond every cache length is never looked at
    far = route.copy()
    far[0, :, 5] = 0                                     # keys 640..767 >= both... batch 0 has 700 keys: use a shorter cache
    words = torch.from_numpy(od.pack_row(far).view(np.int32)).to(dev)
    res = tm.tilemix_decode_int8kv(p, q.to(dev), None, k8, ks, v8, vs, words,
                                   torch.from_numpy(np.asarray([640, 300], np.int32)).to(dev))
    assert tm.tilemix_read_status(res["workspace"])[0] == 0


@pytest.mark.parametrize("n_splits", [1, 2])
def test_decode_running_maximum_moves_many_times(n_splits):
    """Scores that climb along the cache (about 2 log2 units per 128-key tile, far more than the 2^8 by which the
    lazy running maximum may lag): the maximum moves every few steps, in every split and stream, so the rescale of
    the row sums and of the accumulated output (in tensor memory in the tcgen05 form of the step) is exercised many
    times.  The same cache read backwards (maximum first) must work too."""
    B, Hq, Hk, L, d, tile, G = 2, 8, 2, 3000, 128, 128, 1
    q, k, v, route, lens = _case(B, Hq, Hk, L, d, tile, G, seed=51, lens=[3000, 2500], f8=0.5)
    rep = Hq // Hk
    qm = q.float().view(B, Hk, rep, d).mean(2)                       # a direction every head of the group likes
    qm = qm / qm.norm(dim=-1, keepdim=True)
    ramp = torch.linspace(0.0, 1.0, L).view(1, 1, L, 1)
    for sign in (1.0, -1.0):
        kk = (0.3 * k.float() + sign * 60.0 * ramp * qm.unsqueeze(2)).half()
        # the ramp is what the test is about: the scores of every head span far more than 2^8
        s = torch.einsum("bhrd,bhld->bhrl", q.float().view(B, Hk, rep, d), kk.float()) * (1.4427 / d ** 0.5)
        assert (s.max(-1).values - s.min(-1).values).min() > 30.0
        _check(q, kk, v, route, lens, tile, G, n_splits=n_splits)


def test_decode_more_tiles_per_split_than_the_staged_metadata():
    """A split of 266 key tiles: the step stages route bit and block scales of its first 256 tiles in shared memory and
    takes the rest from global memory; more than 32 routing groups per row, so more than one mask word."""
    q, k, v, route, lens = _case(1, 4, 1, 34000, 128, 128, 3, seed=52, lens=[33990], f8=0.5)
    _check(q, k, v, route, lens, 128, 3, n_splits=1)


def test_decode_zero_length_and_one_key_rows_on_the_tcgen05_form():
    """head_dim 128 with 128-key tiles: a sequence without keys (zero output, lse = -inf, its quantised query still
    reported), one with a single key, and splits that get no group at all (more splits than groups)."""
    q, k, v, route, lens = _case(4, 4, 2, 300, 128, 128, 1, seed=53, lens=[300, 0, 1, 128])
    _check(q, k, v, route, lens, 128, 1)
    _check(q, k, v, route, lens, 128, 1, n_splits=5)


@pytest.mark.parametrize("rep", [1, 2, 4, 8])
def test_decode_gqa_group_sizes_on_the_tcgen05_form(rep):
    """head_dim 128 with 128-key tiles, H_q / H_k = 1, 2, 4, 8, a ragged cache of nine tiles and a mixed mask, with
    one split per row (both softmax streams of a CTA get several steps) and with the library's choice."""
    q, k, v, route, lens = _case(2, 2 * rep, 2, 1152, 128, 128, 1, seed=70 + rep, lens=[1100, 1152])
    _check(q, k, v, route, lens, 128, 1, n_splits=1)
    _check(q, k, v, route, lens, 128, 1)


@pytest.mark.parametrize("mask_batch", [1, 5])
def test_decode_splits_shared_out_by_the_kernel(mask_batch):
    """n_splits = -1 on the tcgen05 form: the CTAs of one wave are shared out over the rows by their cost.  Unequal
    cache lengths (one long sequence, short ones, an empty one, a single key), mixed masks, per batch entry or shared:
    the long rows get many splits (up to the cap of 16), the others one each -- every output against the oracle."""
    lens = [16384, 300, 0, 1, 4100]
    q, k, v, route, lens = _case(5, 8, 2, 16384, 128, 128, 2, seed=90 + mask_batch, lens=lens, f8=0.6, mask_batch=mask_batch)
    _check(q, k, v, route, lens, 128, 2, n_splits=-1)


def test_decode_splits_shared_out_pure_routes_and_equal_rows():
    """n_splits = -1 with rows of equal cost (nothing to gain: every row gets the same share, CTAs are left over) and
    with the two pure masks; all INT8 without an FP16 cache."""
    q, k, v, route, lens = _case(3, 4, 4, 2048, 128, 128, 1, seed=95, lens=[2048, 2048, 2048])
    _check(q, k, v, np.ones_like(route), lens, 128, 1, n_splits=-1, k16_none=True)
    _check(q, k, v, np.zeros_like(route), lens, 128, 1, n_splits=-1)
    _check(q, k, v, route, lens, 128, 1, n_splits=-1)


def test_decode_splits_shared_out_falls_back_where_it_cannot():
    """n_splits = -1 means 0 in the warp-level form and with more rows than one wave has CTAs."""
    q, k, v, route, lens = _case(2, 4, 2, 700, 64, 64, 2, seed=96, lens=[700, 33])
    _check(q, k, v, route, lens, 64, 2, n_splits=-1)
    q, k, v, route, lens = _case(80, 2, 2, 256, 128, 128, 1, seed=97, lens=[256 - (i % 7) * 30 for i in range(80)])
    _check(q, k, v, route, lens, 128, 1, n_splits=-1)


def test_decode_at_the_bench_workload_size():
    """8 sequences x 32768 cached tokens, H_q 32 / H_k 8, d 128, G = 4, 75 % INT8 groups, ragged lengths in the last
    two sequences -- the shapes and the launch configuration (library-chosen splits) that bench.py times.  Every output
    of three of the eight sequences against the oracle, after the cache the oracle is given was checked."""
    from paper_2608_17336_b200 import binding as tm
    B, Hq, Hk, L, d, tile, G = 8, 32, 8, 32768, 128, 128, 4
    gen = torch.Generator(device="cpu").manual_seed(81)
    q = torch.randn((B, Hq, d), generator=gen).half()
    k = torch.randn((B, Hk, L, d), generator=gen).half()
    v = torch.randn((B, Hk, L, d), generator=gen).half()
    rng = np.random.default_rng(82)
    route = (rng.random((1, Hk, -(-L // (tile * G)))) < 0.75).astype(np.uint8)
    lens = np.asarray([L, L, L, L, L, L, 30001, 17], np.int32)
    dev = torch.device("cuda:0")
    kd, vd = k.to(dev), v.to(dev)
    k8, v8, ks, vs = tm.tilemix_quantize_qk(tm.problem(B, Hk, Hk, L, d, tile, tile), kd, vd)
    p = tm.decode_problem(B, Hq, Hk, d, L, tile, G)
    words = torch.from_numpy(od.pack_row(route).view(np.int32)).to(dev)
    res = tm.tilemix_decode_int8kv(p, q.to(dev), kd, k8, ks, v8, vs, words, torch.from_numpy(lens).to(dev), want_lse=True)
    torch.cuda.synchronize()
    assert tm.tilemix_read_status(res["workspace"])[0] == 0
    out = res["out"].float().cpu().numpy().astype(np.float64)
    lse = res["lse"].cpu().numpy().astype(np.float64)
    bits = lambda t: np.ascontiguousarray(t.view(torch.int16).numpy()).view(np.uint16)
    for b in (0, 6, 7):
        sl = slice(b, b + 1)
        k16, v16 = bits(k[sl]), bits(v[sl])
        k8_ref, ks_ref = oracle.quantize(k16, tile)
        v8_ref, vs_ref = oracle.quantize(v16, tile)
        assert np.array_equal(k8[sl].cpu().numpy(), k8_ref) and np.array_equal(v8[sl].cpu().numpy(), v8_ref)
        assert np.array_equal(ks[sl].cpu().numpy().view(np.uint32), ks_ref.view(np.uint32))
        assert np.array_equal(vs[sl].cpu().numpy().view(np.uint32), vs_ref.view(np.uint32))
        ref, ref_lse = od.decode(bits(q[sl]), k16, k8_ref, ks_ref, v8_ref, vs_ref, od.pack_row(route), lens[sl], tile, G)
        err = np.abs(out[sl] - ref)
        assert (err <= ATOL * np.maximum(1.0, np.abs(ref))).all(), f"sequence {b}: max err {err.max():.3e}"
        assert np.abs(lse[sl] - ref_lse).max() < 2e-3
