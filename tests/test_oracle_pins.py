"""Pins for the CPU oracle: what the paper and the mathematics fix, checked against
something other than the oracle itself (library routines, brute force on tiny inputs,
closed forms, invariants, the values the paper prints).  CPU only."""
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import Problem

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def f16(x):
    """float array -> binary16 bit patterns (uint16)."""
    return np.ascontiguousarray(np.asarray(x, np.float32).astype(np.float16)).view(np.uint16)


def as_f64(bits):
    return bits.view(np.float16).astype(np.float64)


def rand_qkv(rng, B, Hq, Hk, L, d, scale=1.0):
    q = f16(rng.standard_normal((B, Hq, L, d)) * scale)
    k = f16(rng.standard_normal((B, Hk, L, d)) * scale)
    v = f16(rng.standard_normal((B, Hk, L, d)))
    return q, k, v


def quantized(p, q, k):
    q8, qs = oracle.quantize(q, p.bq)
    k8, ks = oracle.quantize(k, p.bk)
    return q8, k8, qs, ks


def zero_words(p):
    return np.zeros((p.mask_batch, p.heads_kv, p.T_m, p.W), np.uint32)


def random_words(p, rng, frac=0.5, pin=False):
    route = (rng.random((p.mask_batch, p.heads_kv, p.T_m, p.T_mask)) < frac).astype(np.uint8)
    words, counts = oracle.pack(p, route, pin)
    return route, words, counts


# --------------------------------------------------------------------------- FP16 route

@pytest.mark.parametrize("L,d,tile", [(96, 16, 32), (77, 32, 16), (1, 8, 16)])
def test_zero_mask_is_standard_causal_attention(L, d, tile):
    """`Zero` layout (App. B): all groups FP16 == full-precision causal attention.
    Checked against torch's scaled_dot_product_attention in float64."""
    rng = np.random.default_rng(1)
    p = Problem(2, 2, 2, L, d, tile, tile)
    q, k, v = rand_qkv(rng, 2, 2, 2, L, d)
    out, lse, rsum = oracle.attention_full(p, q, k, v, None, None, None, None, zero_words(p))
    tq, tk, tv = (torch.from_numpy(as_f64(x)) for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).numpy()
    assert np.abs(out - ref).max() < 1e-12
    # and against a plain numpy softmax, which also pins lse
    S = np.einsum("bhid,bhjd->bhij", as_f64(q), as_f64(k)) / np.sqrt(d)
    S = np.where(np.tril(np.ones((L, L), bool)), S, -np.inf)
    lse_ref = np.log(np.exp(S - S.max(-1, keepdims=True)).sum(-1)) + S.max(-1)
    assert np.abs(lse - lse_ref).max() < 1e-12
    assert np.abs(rsum - 1.0).max() < 1e-12


def test_first_row_is_first_value_row():
    rng = np.random.default_rng(2)
    p = Problem(1, 1, 1, 40, 8, 16, 16)
    q, k, v = rand_qkv(rng, 1, 1, 1, 40, 8)
    q8, k8, qs, ks = quantized(p, q, k)
    _, words, _ = random_words(p, rng, 0.5)
    out, _, _ = oracle.attention_rows(p, q, k, v, q8, k8, qs, ks, words, [(0, 0, 0)])
    assert np.abs(out[0] - as_f64(v)[0, 0, 0]).max() < 1e-15


def test_shift_invariance_and_custom_scale():
    """Adding one vector w to every key shifts all scores of row i by q_i.w, which softmax
    ignores.  Values sit on a coarse grid so K + w is exact in binary16."""
    rng = np.random.default_rng(3)
    L, d = 48, 8
    p = Problem(1, 1, 1, L, d, 16, 16, softmax_scale=0.37)
    q = f16(rng.integers(-8, 9, (1, 1, L, d)) / 4.0)
    kk = rng.integers(-8, 9, (1, 1, L, d)) / 4.0
    w = rng.integers(-8, 9, (d,)) / 4.0
    v = f16(rng.standard_normal((1, 1, L, d)))
    a, _, _ = oracle.attention_full(p, q, f16(kk), v, None, None, None, None, zero_words(p))
    b, _, _ = oracle.attention_full(p, q, f16(kk + w), v, None, None, None, None, zero_words(p))
    assert np.abs(a - b).max() < 1e-12
    # the explicit scale is used (not 1/sqrt(d)): compare with numpy
    S = np.einsum("id,jd->ij", as_f64(q)[0, 0], kk[0, 0]) * 0.37
    S = np.where(np.tril(np.ones((L, L), bool)), S, -np.inf)
    P = np.exp(S - S.max(-1, keepdims=True)); P /= P.sum(-1, keepdims=True)
    assert np.abs(a[0, 0] - P @ as_f64(v)[0, 0]).max() < 1e-12


# --------------------------------------------------------------------------- quantiser

def test_quantiser_properties():
    rng = np.random.default_rng(4)
    L, d, blk = 70, 24, 16                       # ragged tail block of 6 rows
    x = rng.standard_normal((3, L, d)) * rng.choice([0.01, 1.0, 50.0], (3, 1, 1))
    x[1, 16:32] = 0.0                            # an all-zero block
    xb = f16(x)
    q8, sc = oracle.quantize(xb, blk)
    xf = xb.view(np.float16).astype(np.float32)
    assert q8.dtype == np.int8 and q8.min() >= -127 and q8.max() <= 127
    for h in range(3):
        for r in range(-(-L // blk)):
            blkv = xf[h, r * blk:(r + 1) * blk]
            amax = np.abs(blkv).max()
            # scale definition: absmax/127 as an FP32 division (App. C)
            assert sc[h, r].view(np.uint32) == (np.float32(amax) / np.float32(127)).view(np.uint32)
            qq = q8[h, r * blk:(r + 1) * blk].astype(np.float64)
            if amax == 0:
                assert sc[h, r] == 0 and not qq.any()
                continue
            delta = np.float64(sc[h, r])
            # nearest-integer conversion: error at most half a step (plus FP32 division slack)
            assert np.abs(blkv.astype(np.float64) - delta * qq).max() <= delta / 2 * (1 + 2.0 ** -20)
            # the block maximum maps to +-127
            i = np.unravel_index(np.abs(blkv).argmax(), blkv.shape)
            assert qq[i] == np.sign(blkv[i]) * 127


def test_quantiser_ties_to_even_and_exact_grid():
    """delta = 2^-6 exactly when absmax = 127*2^-6; then x/delta is exact, halves round to even."""
    vals = np.array([127, -127, 0.5, 1.5, 2.5, -0.5, -1.5, 3.49, 100.5, -100.5, 64, 1], np.float64)
    x = (vals * 2.0 ** -6).reshape(1, 1, -1)
    q8, sc = oracle.quantize(f16(x), 1)
    assert sc[0, 0] == np.float32(2.0 ** -6)
    expect = np.array([127, -127, 0, 2, 2, 0, -2, 3, 100, -100, 64, 1])
    # 3.49*2^-6 is not a binary16 value; use what binary16 holds
    held = f16(x).view(np.float16).astype(np.float64)[0, 0] * 64
    expect[7] = int(np.rint(held[7]))
    assert (q8[0, 0] == expect).all()


def test_quantiser_idempotent():
    rng = np.random.default_rng(5)
    x = np.round(rng.standard_normal((2, 64, 16)) * 20) * 2.0 ** -4
    x[:, ::16, 0] = 127 * 2.0 ** -4                      # every 16-row block holds +absmax
    x = np.clip(x, -127 * 2.0 ** -4, 127 * 2.0 ** -4)
    q8, sc = oracle.quantize(f16(x), 16)
    deq = q8.astype(np.float64) * sc.astype(np.float64).repeat(16, axis=1)[..., None]
    q8b, scb = oracle.quantize(f16(deq), 16)
    assert (q8 == q8b).all() and (sc == scb).all()


# --------------------------------------------------------------------------- INT8 route

@pytest.mark.parametrize("L,d,tile", [(40, 16, 16), (64, 8, 32), (33, 4, 8)])
def test_int32_tiles_match_brute_force(L, d, tile):
    rng = np.random.default_rng(6)
    p = Problem(1, 2, 1, L, d, tile, tile)
    q8 = rng.integers(-127, 128, (1, 2, L, d)).astype(np.int8)
    k8 = rng.integers(-127, 128, (1, 1, L, d)).astype(np.int8)
    q8[0, 0, 0] = 127; k8[0, 0, 0] = -127                     # reach the bound
    full = np.einsum("hid,jd->hij", q8[0].astype(np.int64), k8[0, 0].astype(np.int64))
    assert np.abs(full).max() <= 127 * 127 * d
    pad = p.T_m * tile
    fullp = np.zeros((2, pad, pad), np.int64); fullp[:, :L, :L] = full
    for hq in range(2):
        for m in range(p.T_m):
            for n in range(p.T_n):
                t = oracle.int32_tile(p, q8, k8, 0, hq, m, n)
                ref = fullp[hq, m * tile:(m + 1) * tile, n * tile:(n + 1) * tile]
                assert (t.astype(np.int64) == ref).all(), (hq, m, n)


def test_fp_tiles_match_brute_force():
    rng = np.random.default_rng(7)
    L, d, tile = 40, 16, 16
    p = Problem(1, 1, 1, L, d, tile, tile)
    q, k, _ = rand_qkv(rng, 1, 1, 1, L, d)
    full = as_f64(q)[0, 0] @ as_f64(k)[0, 0].T
    pad = np.zeros((48, 48)); pad[:L, :L] = full
    for m in range(3):
        for n in range(3):
            t = oracle.fp_tile(p, q, k, 0, 0, m, n)
            assert np.abs(t - pad[m * 16:(m + 1) * 16, n * 16:(n + 1) * 16]).max() < 1e-12


def brute_force_mixed(p, q, k, v, q8, k8, qs, ks, route_elem, scale):
    """Independent numpy statement for tiny inputs: element-level route map [Hk, L, L]."""
    B, Hq, Hk, L, d = p.batch, p.heads_q, p.heads_kv, p.seqlen, p.head_dim
    out = np.zeros((B, Hq, L, d))
    for b in range(B):
        for hq in range(Hq):
            hk = hq // (Hq // Hk)
            S16 = as_f64(q)[b, hq] @ as_f64(k)[b, hk].T
            C = q8[b, hq].astype(np.int64) @ k8[b, hk].astype(np.int64).T
            dq = qs[b, hq].astype(np.float64).repeat(p.bq)[:L, None]
            dk = ks[b, hk].astype(np.float64).repeat(p.bk)[None, :L]
            S = np.where(route_elem[hk] == 1, dq * dk * C, S16) * scale
            S = np.where(np.tril(np.ones((L, L), bool)), S, -np.inf)
            P = np.exp(S - S.max(-1, keepdims=True)); P /= P.sum(-1, keepdims=True)
            out[b, hq] = P @ as_f64(v)[b, hk]
    return out


@pytest.mark.parametrize("L,tile,G,Hq,Hk", [(64, 16, 1, 2, 1), (100, 16, 2, 4, 2), (60, 8, 4, 1, 1)])
def test_mixed_route_matches_brute_force(L, tile, G, Hq, Hk):
    """Quantise -> integer dots -> dequantise -> softmax -> PV against a numpy brute force with
    an element-level route map built from the *unpacked* decisions (also pins the GQA head
    map h_k = floor(h_q / (H_q/H_k)) and the grouping index g_j = floor(n/G))."""
    rng = np.random.default_rng(8)
    d = 16
    p = Problem(2, Hq, Hk, L, d, tile, tile, G)
    q, k, v = rand_qkv(rng, 2, Hq, Hk, L, d, scale=1.5)
    q8, k8, qs, ks = quantized(p, q, k)
    route, words, _ = random_words(p, rng, 0.5)
    # element map from the routing map: pair (i, j) -> R[hk, i//tile, (j//tile)//G]
    ii, jj = np.meshgrid(np.arange(L), np.arange(L), indexing="ij")
    route_elem = route[0][:, ii // tile, (jj // tile) // G]
    ref = brute_force_mixed(p, q, k, v, q8, k8, qs, ks, route_elem, 1 / np.sqrt(d))
    out, _, rsum = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, words)
    assert np.abs(out - ref).max() < 1e-12
    assert np.abs(rsum - 1).max() < 1e-12
    # the INT8 route really differs from FP16 here (the test would be vacuous otherwise)
    z, _, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, zero_words(p))
    assert np.abs(out - z).max() > 1e-4


@pytest.mark.parametrize("G", [2, 4, 8])
def test_group_mask_equals_expanded_tile_mask(G):
    """One bit per G adjacent key tiles == the same decisions written per tile (G = 1)."""
    rng = np.random.default_rng(9)
    L, d, tile = 200, 8, 8
    pg = Problem(1, 2, 2, L, d, tile, tile, G)
    p1 = Problem(1, 2, 2, L, d, tile, tile, 1)
    q, k, v = rand_qkv(rng, 1, 2, 2, L, d)
    q8, k8, qs, ks = quantized(pg, q, k)
    route, words, _ = random_words(pg, rng, 0.5)
    expanded = np.repeat(route, G, axis=-1)[..., :p1.T_mask]
    words1, _ = oracle.pack(p1, np.ascontiguousarray(expanded))
    a, la, _ = oracle.attention_full(pg, q, k, v, q8, k8, qs, ks, words)
    b, lb, _ = oracle.attention_full(p1, q, k, v, q8, k8, qs, ks, words1)
    assert (a == b).all() and (la == lb).all()


def test_lossless_quantisation_makes_every_mask_equal_fp16():
    """Q, K on the grid {-127..127}*2^-6 with +-127*2^-6 in every block: delta = 2^-6, the
    quantisation is exact, so INT8 and FP16 scores coincide and any routing map gives the
    all-FP16 result."""
    rng = np.random.default_rng(10)
    L, d, tile = 96, 16, 16
    p = Problem(1, 2, 1, L, d, tile, tile, 2)
    def grid(shape):
        x = rng.integers(-127, 128, shape).astype(np.float64)
        x[..., ::tile, 0] = 127
        return f16(x * 2.0 ** -6)
    q, k = grid((1, 2, L, d)), grid((1, 1, L, d))
    v = f16(rng.standard_normal((1, 1, L, d)))
    q8, k8, qs, ks = quantized(p, q, k)
    assert (qs == np.float32(2.0 ** -6)).all() and (ks == np.float32(2.0 ** -6)).all()
    ref, _, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, zero_words(p))
    for frac in (0.3, 1.0):
        _, words, _ = random_words(p, rng, frac)
        out, _, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, words)
        assert np.abs(out - ref).max() < 1e-13


def test_zero_queries_give_prefix_means():
    """Q == 0: every score is 0 (also through the zero-block guard of the quantiser), so
    O[i] = mean(V[0..i]) for any routing map."""
    rng = np.random.default_rng(11)
    L, d, tile = 50, 8, 16
    p = Problem(1, 1, 1, L, d, tile, tile)
    q = f16(np.zeros((1, 1, L, d)))
    k = f16(rng.standard_normal((1, 1, L, d)))
    v = f16(rng.standard_normal((1, 1, L, d)))
    q8, k8, qs, ks = quantized(p, q, k)
    assert not qs.any() and not q8.any()
    _, words, _ = random_words(p, rng, 0.5)
    out, lse, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, words)
    ref = np.cumsum(as_f64(v)[0, 0], 0) / np.arange(1, L + 1)[:, None]
    assert np.abs(out[0, 0] - ref).max() < 1e-13
    assert np.abs(lse[0, 0] - np.log(np.arange(1, L + 1))).max() < 1e-13


def test_int8_score_error_bound():
    """|S8 - S16| <= (dQ/2*|k^|_1 + dK/2*|q^|_1 + d*dQ*dK/4)/sqrt(d), from |x - delta*x^| <= delta/2."""
    rng = np.random.default_rng(12)
    L, d, tile = 64, 32, 16
    p = Problem(1, 1, 1, L, d, tile, tile)
    q, k, _ = rand_qkv(rng, 1, 1, 1, L, d)
    q8, k8, qs, ks = quantized(p, q, k)
    for m in range(p.T_m):
        for n in range(p.T_n):
            C = oracle.int32_tile(p, q8, k8, 0, 0, m, n).astype(np.float64)
            S16 = oracle.fp_tile(p, q, k, 0, 0, m, n)
            dq, dk = float(qs[0, 0, m]), float(ks[0, 0, n])
            qh = np.abs(q8[0, 0, m * tile:(m + 1) * tile].astype(np.float64) * dq).sum(-1)
            kh = np.abs(k8[0, 0, n * tile:(n + 1) * tile].astype(np.float64) * dk).sum(-1)
            bound = dq / 2 * kh[None, :] + dk / 2 * qh[:, None] + d * dq * dk / 4
            assert (np.abs(dq * dk * C - S16) <= bound * (1 + 1e-6)).all()
            assert np.abs(dq * dk * C - S16).max() > 0          # and it is not the FP16 value


# --------------------------------------------------------------------------- packer

def brute_legal_and_diag(p, m, g):
    """Element-level statement: a group is legal iff it holds a pair j <= i; diagonal iff one
    of its key tiles holds both a pair j <= i and a pair j >= i."""
    rows = range(m * p.tile_m, min((m + 1) * p.tile_m, p.seqlen))
    legal = diag = False
    for n in range(g * p.group, min((g + 1) * p.group, p.T_n)):
        cols = range(n * p.tile_n, min((n + 1) * p.tile_n, p.seqlen))
        below = any(j <= i for i in rows for j in cols)
        above = any(j >= i for i in rows for j in cols)
        legal |= below
        diag |= below and above
    return legal, diag


@pytest.mark.parametrize("L,tm,tn,G", [(100, 16, 16, 1), (100, 16, 16, 3), (130, 32, 16, 2),
                                       (64, 16, 32, 1), (17, 16, 16, 4), (1, 16, 16, 1)])
def test_packer_against_brute_force(L, tm, tn, G):
    rng = np.random.default_rng(13)
    p = Problem(1, 2, 2, L, 8, tm, tn, G, mask_batch=1)
    route = (rng.random((1, 2, p.T_m, p.T_mask)) < 0.6).astype(np.uint8)
    for pin in (False, True):
        words, counts = oracle.pack(p, route, pin)
        for h in range(2):
            n_legal = n_int8 = 0
            for m in range(p.T_m):
                val = 0
                for g in range(p.T_mask):
                    legal, diag = brute_legal_and_diag(p, m, g)
                    n_legal += legal
                    bit = int(route[0, h, m, g]) if legal and not (pin and diag) else 0
                    n_int8 += bit
                    val += bit << g                     # b = sum R * 2^g  (Sec. 4.2)
                got = sum(int(words[0, h, m, w]) << (32 * w) for w in range(p.W))
                assert got == val, (h, m, hex(got), hex(val))
            assert int(counts[0, h, 0]) == n_legal and int(counts[0, h, 1]) == n_int8
            pop = sum(bin(int(x)).count("1") for x in words[0, h].ravel())
            assert pop == n_int8


def test_packed_row_is_the_papers_uint64_for_T_mask_le_64():
    rng = np.random.default_rng(14)
    p = Problem(1, 1, 1, 64 * 8, 8, 8, 8, 1)             # T_mask = 64 -> W = 2
    assert p.T_mask == 64 and p.W == 2
    route = (rng.random((1, 1, p.T_m, 64)) < 0.5).astype(np.uint8)
    words, _ = oracle.pack(p, route)
    as64 = words.view("<u8")[0, 0, :, 0]
    for m in range(p.T_m):
        legal = m + 1
        ref = sum(int(route[0, 0, m, g]) << g for g in range(legal))
        assert int(as64[m]) == ref
        # constant-time lookup (Sec. 4.2): R = (b >> g) & 1
        for g in range(legal):
            assert (int(as64[m]) >> g) & 1 == route[0, 0, m, g]


def test_grouping_rule_matches_configs():
    """App. B: g = 4, T_mask = 64 at L = 32768 and g = 1, T_mask = 64 at L = 8192 (BLOCK_N = 128)."""
    assert oracle.grouping_rule(32768, 128) == (4, 64)
    assert oracle.grouping_rule(8192, 128) == (1, 64)
    assert oracle.grouping_rule(4096, 128) == (1, 32)
    assert oracle.grouping_rule(131072, 128) == (16, 64)
    for L in (1000, 5000, 70000, 200000):
        g, t = oracle.grouping_rule(L, 64)
        assert t <= 64 and (g == 1 or -(-L // ((g - 1) * 64)) > 64)


def test_memory_accounting_matches_printed_table():
    golden = {}
    for line in open(os.path.join(GOLDEN, "memory_accounting.txt")):
        if line.strip() and not line.startswith("#"):
            key, val = line.split("=")
            golden[key.strip()] = float(val)
    total, fp16 = oracle.resident_bytes_quantize_once(32, 8, 8192, 128, 128, 64, 128)
    assert fp16 / 2 ** 20 == golden["flashattention_resident_hbm_mb"]
    assert round(total / 2 ** 20, 2) == golden["quantize_once_resident_hbm_mib"]
    assert fp16 / 2 ** 20 == golden["on_the_fly_resident_hbm_mb"]
    # an INT8 K tile of 128 x 128 is half the FP16 tile the on-the-fly mode reads
    assert 128 * 128 * 2 / 1024 == golden["on_the_fly_int8_qk_tile_read_kb"]
    assert 128 * 128 / 1024 == int(golden["quantize_once_int8_qk_tile_read_kb"])


# --------------------------------------------------------------------------- per-batch routing maps

def test_per_batch_masks_equal_single_batch_runs():
    """App. B "Policy Construction and Sharing": a template may be shared over the batch (mask_batch = 1)
    or not (mask_batch = B).  With one routing map per batch entry, entry b must be exactly the
    single-batch problem on entry b's tensors with entry b's map -- packed words, counters and outputs --
    and must differ from what entry b gives under the other entry's map (so a wrong batch index fails)."""
    rng = np.random.default_rng(15)
    B, Hq, Hk, L, d, tile, G = 2, 2, 1, 90, 16, 16, 2
    p = Problem(B, Hq, Hk, L, d, tile, tile, G, mask_batch=B)
    q, k, v = rand_qkv(rng, B, Hq, Hk, L, d, scale=1.5)
    q8, k8, qs, ks = quantized(p, q, k)
    route = (rng.random((B, Hk, p.T_m, p.T_mask)) < 0.5).astype(np.uint8)
    route[1] = 1 - route[0]                               # the two maps disagree on every group
    for pin in (False, True):
        words, counts = oracle.pack(p, route, pin)
        out, lse, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, words)
        p1 = Problem(1, Hq, Hk, L, d, tile, tile, G, mask_batch=1)
        for b in range(B):
            sl = slice(b, b + 1)
            w1, c1 = oracle.pack(p1, np.ascontiguousarray(route[sl]), pin)
            assert (w1[0] == words[b]).all() and (c1[0] == counts[b]).all()
            o1, l1, _ = oracle.attention_full(p1, *(np.ascontiguousarray(x[sl]) for x in (q, k, v, q8, k8, qs, ks)), w1)
            assert (o1[0] == out[b]).all() and (l1[0] == lse[b]).all()
            wrong, _ = oracle.pack(p1, np.ascontiguousarray(route[1 - b:2 - b]), pin)
            o2, _, _ = oracle.attention_full(p1, *(np.ascontiguousarray(x[sl]) for x in (q, k, v, q8, k8, qs, ks)), wrong)
            assert np.abs(o2[0] - out[b]).max() > 1e-4
        # sampled rows take the same branch as the full evaluation
        rows = [(b, h, i) for b in range(B) for h in range(Hq) for i in (0, 17, L - 1)]
        o3, _, _ = oracle.attention_rows(p, q, k, v, q8, k8, qs, ks, words, rows)
        for r, (b, h, i) in enumerate(rows):
            assert (o3[r] == out[b, h, i]).all()


def test_per_batch_masks_match_brute_force():
    """The numpy brute force of the mixed route, with the element-level route map taken from route[b]."""
    rng = np.random.default_rng(16)
    B, Hq, Hk, L, d, tile, G = 3, 2, 2, 70, 16, 16, 1
    p = Problem(B, Hq, Hk, L, d, tile, tile, G, mask_batch=B)
    q, k, v = rand_qkv(rng, B, Hq, Hk, L, d, scale=1.5)
    q8, k8, qs, ks = quantized(p, q, k)
    route = (rng.random((B, Hk, p.T_m, p.T_mask)) < 0.5).astype(np.uint8)
    words, _ = oracle.pack(p, route)
    out, _, _ = oracle.attention_full(p, q, k, v, q8, k8, qs, ks, words)
    ii, jj = np.meshgrid(np.arange(L), np.arange(L), indexing="ij")
    p1 = Problem(1, Hq, Hk, L, d, tile, tile, G)
    for b in range(B):
        route_elem = route[b][:, ii // tile, (jj // tile) // G]
        sl = slice(b, b + 1)
        ref = brute_force_mixed(p1, q[sl], k[sl], v[sl], q8[sl], k8[sl], qs[sl], ks[sl], route_elem, 1 / np.sqrt(d))
        assert np.abs(out[b] - ref[0]).max() < 1e-12
    assert np.abs(out[0] - out[1]).max() > 1e-4
