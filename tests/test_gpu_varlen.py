"""Variable-length batches (Sec. 4.1; App. C scale shapes) on the GPU against the oracle applied to
every sequence on its own: quantiser and packer bit-exact, attention outputs within tolerance."""
import numpy as np
import pytest
import torch

import oracle
from tests.helpers import ATOL, run_gpu_varlen, varlen_inputs, varlen_oracle

pytestmark = pytest.mark.gpu


def _check_batch(cu, Hq, Hk, d, tile, group, seed, f8=0.5, pin=False):
    q, k, v, route = varlen_inputs(cu, Hq, Hk, d, tile, group, seed, f8)
    g = run_gpu_varlen(cu, q, k, v, route, tile, group, pin)
    ref = varlen_oracle(cu, q, k, v, route, tile, group, pin)
    q8, k8 = g["q8"].cpu().numpy(), g["k8"].cpu().numpy()
    qs, ks = g["qs"].cpu().numpy(), g["ks"].cpu().numpy()
    words = g["words"].cpu().numpy().view(np.uint32)
    out = g["out"].float().cpu().numpy().astype(np.float64)
    lse = g["lse"].cpu().numpy().astype(np.float64)
    legal = int8 = 0
    worst = 0.0
    for s, r in enumerate(ref):
        if r is None:
            continue
        t0, L, row0, p = r["tok0"], r["p"].seqlen, r["row0"], r["p"]
        # quantiser: INT8 codes [H, total, d] and block-major scales [blocks, H], bit-exact
        assert np.array_equal(q8[:, t0:t0 + L], r["q8"][0]), f"q8 of sequence {s}"
        assert np.array_equal(k8[:, t0:t0 + L], r["k8"][0]), f"k8 of sequence {s}"
        nb = p.T_m                                       # blocks == tiles here
        assert np.array_equal(qs[row0:row0 + nb].T.view(np.uint32), r["qs"][0].view(np.uint32))
        assert np.array_equal(ks[row0:row0 + nb].T.view(np.uint32), r["ks"][0].view(np.uint32))
        # packer: the sequence's own words, zero beyond its own W
        w_s = words[:, row0:row0 + p.T_m]
        assert np.array_equal(w_s[:, :, :p.W], r["words"][0]), f"mask words of sequence {s}"
        assert not w_s[:, :, p.W:].any()
        legal += int(r["counts"][0, :, 0].sum()); int8 += int(r["counts"][0, :, 1].sum())
        # attention: out [total, Hq, d], lse [Hq, total]
        o_ref = r["out"][0].transpose(1, 0, 2)
        err = np.abs(out[t0:t0 + L] - o_ref)
        bound = ATOL * np.maximum(1.0, np.abs(o_ref))
        assert (err <= bound).all(), f"sequence {s}: max err {err.max():.3e}"
        worst = max(worst, float(err.max()))
        assert np.abs(lse[:, t0:t0 + L] - r["lse"][0]).max() < 2e-3
    counts = g["counts"].cpu().numpy()
    assert int(counts[:, 0].sum()) == legal and int(counts[:, 1].sum()) == int8
    return worst


def test_varlen_small_tiles_ragged():
    # 64x64 tiles, d = 64: single token, sub-tile, exact tile, ragged multi-tile, an empty sequence
    cu = np.cumsum([0, 1, 37, 64, 0, 200, 129, 513]).tolist()
    _check_batch(cu, 2, 2, 64, 64, 1, seed=11)


def test_varlen_large_tiles_grouped():
    # 128x128 tiles, d = 128, G = 2, odd and even numbers of tile rows per sequence
    cu = np.cumsum([0, 300, 128, 1000, 5, 640]).tolist()
    _check_batch(cu, 2, 2, 128, 128, 2, seed=12, f8=0.6)


def test_varlen_gqa_pinned_diagonal():
    cu = np.cumsum([0, 257, 900, 64]).tolist()
    _check_batch(cu, 4, 2, 128, 128, 1, seed=13, f8=0.7, pin=True)


@pytest.mark.parametrize("f8", [0.0, 1.0])
def test_varlen_pure_routes(f8):
    cu = np.cumsum([0, 130, 70, 333]).tolist()
    _check_batch(cu, 2, 1, 64, 64, 2, seed=14, f8=f8)


def test_varlen_single_sequence_equals_dense():
    """One sequence in the packed layout gives the dense call's output bit for bit."""
    from tests.helpers import run_gpu
    from paper_2608_17336_b200 import synth
    L, H, d, tile, G = 700, 2, 128, 128, 1
    cu = [0, L]
    q, k, v, route = varlen_inputs(cu, H, H, d, tile, G, seed=15)
    g = run_gpu_varlen(cu, q, k, v, route, tile, G)
    w = synth.Workload("dense", 1, H, L, d, tile, G, seed=15)
    qd, kd, vd = (t.permute(1, 0, 2)[None].contiguous() for t in (q, k, v))
    dense = run_gpu(w, qd, kd, vd, np.ascontiguousarray(route[None]))
    assert torch.equal(g["out"].permute(1, 0, 2)[None].view(torch.int16), dense["out"].view(torch.int16))


def test_varlen_no_leak_across_sequences():
    """Changing one sequence's K and V leaves every other sequence's output bit-identical."""
    cu = np.cumsum([0, 190, 260, 150]).tolist()
    q, k, v, route = varlen_inputs(cu, 2, 2, 64, 64, 1, seed=16)
    a = run_gpu_varlen(cu, q, k, v, route, 64, 1)["out"].cpu()
    k2, v2 = k.clone(), v.clone()
    k2[cu[1]:cu[2]] = 7.0
    v2[cu[1]:cu[2]] = -3.0
    b = run_gpu_varlen(cu, q, k2, v2, route, 64, 1)["out"].cpu()
    for s in (0, 2):
        assert torch.equal(a[cu[s]:cu[s + 1]].view(torch.int16), b[cu[s]:cu[s + 1]].view(torch.int16))
    assert not torch.equal(a[cu[1]:cu[2]], b[cu[1]:cu[2]])


def test_varlen_int32_accumulators():
    """Raw INT32 score accumulators of INT8-routed tiles inside a later sequence, bit-exact on the
    rows and columns that belong to the sequence."""
    cu = np.cumsum([0, 100, 300]).tolist()
    tile = 64
    q, k, v, route = varlen_inputs(cu, 1, 1, 64, tile, 1, seed=17, int8_fraction=1.0)
    tiles = [(1, 0, m, n) for m in range(5) for n in range(m + 1)]
    g = run_gpu_varlen(cu, q, k, v, route, tile, 1, debug_tiles=tiles)
    r = varlen_oracle(cu, q, k, v, route, tile, 1, seqs={1})[1]
    raw, kind = g["raw"].cpu().numpy(), g["kind"].cpu().numpy()
    L = 300
    for e, (_, h, m, n) in enumerate(tiles):
        assert kind[e] == 1
        want = oracle.int32_tile(r["p"], r["q8"], r["k8"], 0, h, m, n)
        rows, cols = min(tile, L - m * tile), min(tile, L - n * tile)
        assert np.array_equal(raw[e, :rows, :cols], want[:rows, :cols]), (m, n)


def test_varlen_max_seqlen_fixes_mask_width():
    """A caller-chosen max_seqlen widens T_mask_max / W without changing the result."""
    cu = np.cumsum([0, 150, 90]).tolist()
    tile, G = 64, 1
    q, k, v, route = varlen_inputs(cu, 2, 2, 64, tile, G, seed=18)
    a = run_gpu_varlen(cu, q, k, v, route, tile, G)
    wide = np.zeros((2, route.shape[1], 40), np.uint8)     # max_seqlen 2560 -> T_mask_max 40, W 2
    wide[:, :, :route.shape[2]] = route
    wide[:, :, route.shape[2]:] = 1                        # beyond every sequence: ignored
    b = run_gpu_varlen(cu, q, k, v, wide, tile, G, max_seqlen=2560)
    assert b["words"].shape[-1] == 2
    assert torch.equal(a["out"].view(torch.int16), b["out"].view(torch.int16))
    assert torch.equal(a["counts"], b["counts"])


@pytest.mark.parametrize("seed", [41, 42, 43])
def test_varlen_random_batches(seed):
    rng = np.random.default_rng(seed)
    big = bool(rng.integers(0, 2))
    d = tile = 128 if big else 64
    n = int(rng.integers(1, 7))
    lens = rng.integers(0, 700, n).tolist()
    if sum(lens) == 0:
        lens[0] = 5
    Hk = int(rng.integers(1, 3)); rep = int(rng.choice([1, 2]))
    cu = np.cumsum([0] + lens).tolist()
    _check_batch(cu, Hk * rep, Hk, d, tile, int(rng.integers(1, 4)), seed=seed, f8=float(rng.random()),
                 pin=bool(rng.integers(0, 2)))
