"""Routing templates (the paper's precision layouts): set definitions checked by brute force on small
geometries, coverage matching, the automatic grouping factor and the cache.  CPU only."""
import numpy as np
import pytest

import oracle
from paper_2608_17336_b200 import policy as P

GEO = [P.Geometry(1000, 16, 16, 2), P.Geometry(512, 32, 16, 1), P.Geometry(777, 16, 32, 3)]


def brute_legal(geo):
    out = np.zeros((geo.T_m, geo.T_mask), bool)
    for m in range(geo.T_m):
        for g in range(geo.T_mask):
            rows = range(m * geo.tile_m, min((m + 1) * geo.tile_m, geo.seqlen))
            cols = range(g * geo.block_mask, min((g + 1) * geo.block_mask, geo.seqlen))
            out[m, g] = any(j <= i for i in rows for j in cols[:1])      # first key of the group suffices
    return out


@pytest.mark.parametrize("geo", GEO)
def test_legal_groups_and_trivial_layouts(geo):
    legal = brute_legal(geo)
    assert (P.legal_groups(geo) == legal).all()
    assert (P.one(geo) == legal).all() and not P.zero(geo).any()
    assert P.coverage(geo, P.one(geo)) == 1.0 and P.coverage(geo, P.zero(geo)) == 0.0
    # the same legality as the packer's (oracle): packing `One` sets exactly the legal bits
    po = oracle.Problem(1, 1, 1, geo.seqlen, 8, geo.tile_m, geo.tile_n, geo.group)
    words, counts = oracle.pack(po, P.broadcast(np.ones_like(P.one(geo)), 1))
    assert int(counts[0, 0, 0]) == int(legal.sum()) == int(counts[0, 0, 1])


@pytest.mark.parametrize("geo", GEO)
def test_band_global_aligned_definitions(geo):
    legal = brute_legal(geo)
    for w in (0, 1, 3):
        R = P.band(geo, w)
        for m in range(geo.T_m):
            gamma = (m * geo.tile_m) // geo.block_mask
            for g in range(geo.T_mask):
                assert R[m, g] == (legal[m, g] and abs(g - gamma) > w)
    R = P.global_(geo, 2)
    assert not R[:, :2].any() and (R[:, 2:] == legal[:, 2:]).all()
    alpha, beta = 1.0, 0.25
    R = P.aligned_sparse(geo, alpha, beta)
    for m in range(geo.T_m):
        gs = np.nonzero(legal[m])[0]
        a = min(len(gs), int(np.ceil(alpha + beta * m)))
        fp16 = set(gs[len(gs) - a:])
        assert {g for g in gs if R[m, g] == 0} == fp16
    # the FP16 count never shrinks with the query index while the row is not saturated
    n_fp16 = (legal & (R == 0)).sum(1)
    assert (np.diff(n_fp16) >= 0).all()


@pytest.mark.parametrize("geo", GEO[:2])
def test_row_random_counts_and_bigbird_union(geo):
    legal = brute_legal(geo)
    rho = 0.7
    R = P.row_random(geo, rho, seed=3)
    k = np.rint((1 - rho) * legal.sum(1)).astype(int)
    assert ((legal & (R == 0)).sum(1) == k).all()
    assert (R == P.row_random(geo, rho, seed=3)).all() and (R != P.row_random(geo, rho, seed=4)).any()
    B = P.bigbird(geo, 1, 1, 0.8, seed=3)
    fp16 = legal & (B == 0)
    union = legal & ((P.band(geo, 1) == 0) | (P.global_(geo, 1) == 0) | (P.row_random(geo, 0.8, seed=3) == 0))
    assert (fp16 == union).all()


def test_sptrans_against_element_level_definition():
    geo = P.Geometry(300, 16, 16, 1)
    s, c = 64, 20
    R = P.sptrans(geo, s, c)
    legal = brute_legal(geo)
    for m in range(geo.T_m):
        sel = np.zeros(geo.T_mask, bool)
        for i in range(m * geo.tile_m, min((m + 1) * geo.tile_m, geo.seqlen)):
            u = i // s
            keys = set(range(u * s, i + 1))
            for r in range(u):
                keys |= set(range(max(r * s, (r + 1) * s - c), (r + 1) * s))
            for j in keys:
                sel[j // geo.block_mask] = True
        assert ((R[m] == 0) & legal[m] == sel & legal[m]).all(), m


@pytest.mark.parametrize("layout", ["band", "global", "row_random", "aligned_sparse", "bigbird", "sptrans"])
@pytest.mark.parametrize("target", [0.25, 0.5, 0.75])
def test_coverage_matching(layout, target):
    geo = P.Geometry(8192, 128, 128, 1)
    R, info = P.match_coverage(geo, layout, target)
    assert abs(info["coverage"] - target) < 0.06, info
    assert abs(P.coverage(geo, R) - info["coverage"]) < 1e-12
    assert not R[~P.legal_groups(geo)].any()


def test_grouping_rule_and_cache():
    for L, bn in ((32768, 128), (8192, 128), (4096, 128), (131072, 128), (5000, 64), (100, 64)):
        assert (P.grouping_rule(L, bn), -(-L // (P.grouping_rule(L, bn) * bn))) == oracle.grouping_rule(L, bn)
    geo, R, info = P.template(32768, 128, 128, "band", 0.75)
    assert geo.group == 4 and geo.T_mask == 64 and R.shape == (256, 64)
    geo2, R2, _ = P.template(32768, 128, 128, "band", 0.75)
    assert R2 is R                                  # cached until length or geometry changes
    _, R3, _ = P.template(16384, 128, 128, "band", 0.75)
    assert R3 is not R
    full = P.broadcast(R, 8)
    assert full.shape == (1, 8, 256, 64) and full.flags["C_CONTIGUOUS"] and (full[0, 5] == R).all()
