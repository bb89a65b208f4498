"""Pins of the decode-step oracle (INT8 key/value cache interface) against things other than itself:
a library attention routine, the already pinned prefill oracle, brute-force loops and invariants."""
import math

import numpy as np
import torch

import oracle
from oracle import decode as od


def _case(B, Hq, Hk, L, d, tile, G, seed, lens=None, f8=0.5, pow2_v=False):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B, Hq, d)).astype(np.float16)
    k = rng.standard_normal((B, Hk, L, d)).astype(np.float16)
    v = rng.standard_normal((B, Hk, L, d)).astype(np.float16)
    k16 = k.view(np.uint16)
    k8, ks = oracle.quantize(np.ascontiguousarray(k16), tile)
    if pow2_v:
        v8 = rng.integers(-127, 128, (B, Hk, L, d)).astype(np.int8)
        vs = np.full((B, Hk, -(-L // tile)), 2.0 ** -5, np.float32)
    else:
        v8, vs = oracle.quantize(np.ascontiguousarray(v.view(np.uint16)), tile)
    T_mask = -(-L // (tile * G))
    route = (rng.random((1, Hk, T_mask)) < f8).astype(np.uint8)
    lens = np.full(B, L) if lens is None else np.asarray(lens)
    return dict(q16=q.view(np.uint16), k16=k16, k8=k8, ks=ks, v8=v8, vs=vs, route=route,
                words=od.pack_row(route), lens=lens, tile=tile, G=G)


def _run(c, **kw):
    return od.decode(c["q16"], c["k16"], c["k8"], c["ks"], c["v8"], c["vs"], kw.get("words", c["words"]),
                     c["lens"], c["tile"], c["G"], kw.get("scale", 0.0))


def test_all_fp16_route_is_library_attention_over_dequantised_v():
    c = _case(2, 4, 2, 300, 64, 64, 2, seed=1, lens=[300, 117])
    out, lse = _run(c, words=np.zeros_like(c["words"]))
    for b in range(2):
        L = int(c["lens"][b])
        q = torch.from_numpy(od.half_bits_to_f64(c["q16"][b]))[:, None, :]                  # [Hq,1,d]
        k = torch.from_numpy(od.half_bits_to_f64(c["k16"][b, :, :L])).repeat_interleave(2, 0)
        blk = np.arange(L) // 64
        v = torch.from_numpy(c["v8"][b, :, :L].astype(np.float64) * c["vs"][b][:, blk, None].astype(np.float64))
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v.repeat_interleave(2, 0))
        assert np.abs(out[b] - ref[:, 0].numpy()).max() < 1e-12
        s = (q @ k.transpose(1, 2))[:, 0] / math.sqrt(64)
        assert np.abs(lse[b] - torch.logsumexp(s, -1).numpy()).max() < 1e-12


def test_mixed_route_equals_last_row_of_the_prefill_oracle():
    """A decode step is the last query row of a causal prefill whose query blocks are single rows and
    whose FP16 V equals delta_V * V8 exactly (power-of-two scale)."""
    B, Hq, Hk, L, d, tile, G = 1, 2, 1, 200, 64, 64, 2
    c = _case(B, Hq, Hk, L, d, tile, G, seed=2, pow2_v=True)
    rng = np.random.default_rng(3)
    Q = rng.standard_normal((B, Hq, L, d)).astype(np.float16)
    Q[:, :, L - 1] = c["q16"].view(np.float16)
    qb = np.ascontiguousarray(Q.view(np.uint16))
    v16 = (c["v8"].astype(np.float32) * 2.0 ** -5).astype(np.float16)
    assert np.array_equal(v16.astype(np.float64), c["v8"].astype(np.float64) * 2.0 ** -5)
    p = oracle.Problem(B, Hq, Hk, L, d, tile, tile, G, blk_q=1)
    q8, qs = oracle.quantize(qb, 1)
    route = np.zeros((1, Hk, p.T_m, p.T_mask), np.uint8)
    route[:, :, p.T_m - 1] = c["route"]
    words, _ = oracle.pack(p, route)
    rows = [(0, h, L - 1) for h in range(Hq)]
    ref, ref_lse, _ = oracle.attention_rows(p, qb, c["k16"], np.ascontiguousarray(v16.view(np.uint16)), q8, c["k8"],
                                            qs, c["ks"], words, rows)
    out, lse = _run(c)
    assert np.abs(out[0] - ref).max() < 1e-12
    assert np.abs(lse[0] - ref_lse).max() < 1e-12
    assert c["route"].any() and not c["route"].all()


def test_brute_force_loops():
    c = _case(1, 2, 1, 70, 16, 32, 1, seed=4, lens=[53])
    out, lse = _run(c)
    half = lambda bits: float(np.array(bits, np.uint16).view(np.float16))
    for hq in range(2):
        q = [half(x) for x in c["q16"][0, hq]]
        amax = max(abs(x) for x in q)
        dq = np.float32(amax) / np.float32(127.0)
        q8 = [int(np.rint(np.float32(x) / dq)) for x in q]
        assert q8 == od.quantize_query(c["q16"])[0][0, hq].tolist()
        s = []
        for j in range(53):
            g = j // 32
            if (int(c["words"][0, 0, g >> 5]) >> (g & 31)) & 1:
                dot = sum(a * int(b) for a, b in zip(q8, c["k8"][0, 0, j]))
                s.append(float(dq) * float(c["ks"][0, 0, j // 32]) * dot / 4.0)
            else:
                s.append(sum(a * half(b) for a, b in zip(q, c["k16"][0, 0, j])) / 4.0)
        m = max(s)
        w = [math.exp(x - m) for x in s]
        for e in range(16):
            o = sum(w[j] * float(c["vs"][0, 0, j // 32]) * int(c["v8"][0, 0, j, e]) for j in range(53)) / sum(w)
            assert abs(o - out[0, hq, e]) < 1e-12
        assert abs(m + math.log(sum(w)) - lse[0, hq]) < 1e-12


def test_invariants():
    c = _case(2, 4, 4, 256, 32, 64, 1, seed=5, lens=[256, 1])
    out, lse = _run(c)
    # a cache of one key returns that key's dequantised value, whatever the route
    v0 = c["v8"][1, :, 0].astype(np.float64) * c["vs"][1, :, 0:1].astype(np.float64)
    assert np.abs(out[1] - v0).max() < 1e-12
    # the V scales are linear in the output; the scores do not see them
    c2 = dict(c, vs=c["vs"] * np.float32(4.0))
    out2, lse2 = _run(c2)
    assert np.allclose(out2, 4.0 * out, rtol=0, atol=1e-12) and np.array_equal(lse, lse2)
    # keys beyond cache_len are never read
    c3 = dict(c, k8=c["k8"].copy(), v8=c["v8"].copy(), k16=c["k16"].copy())
    c3["k8"][1, :, 1:] = 99; c3["v8"][1, :, 1:] = -99; c3["k16"][1, :, 1:] = 0x7bff
    out3, _ = _run(c3)
    assert np.array_equal(out3, out)
    # a custom softmax scale equals pre-scaled queries on the FP16 route (power of two: exact)
    z = np.zeros_like(c["words"])
    a, _ = _run(c, words=z, scale=0.5 / math.sqrt(32))
    c4 = dict(c, q16=(c["q16"].view(np.float16) * np.float16(0.5)).view(np.uint16))
    b_, _ = _run(c4, words=z)
    assert np.abs(a - b_).max() < 1e-12


def test_int8_route_equals_fp16_route_when_quantisation_is_lossless():
    rng = np.random.default_rng(6)
    B, Hq, Hk, L, d, tile = 1, 2, 2, 128, 32, 64
    q = rng.integers(-127, 128, (B, Hq, d)).astype(np.float16)
    k = rng.integers(-127, 128, (B, Hk, L, d)).astype(np.float16)
    q[:, :, 0] = 127; k[:, :, ::tile, 0] = 127      # every block's maximum is 127: delta = 1
    q *= np.float16(1 / 64); k *= np.float16(1 / 64)
    k16 = np.ascontiguousarray(k.view(np.uint16))
    k8, ks = oracle.quantize(k16, tile)
    v8 = rng.integers(-127, 128, (B, Hk, L, d)).astype(np.int8)
    vs = np.full((B, Hk, L // tile), 0.25, np.float32)
    args = (q.view(np.uint16), k16, k8, ks, v8, vs)
    one = od.pack_row(np.ones((1, Hk, 2), np.uint8))
    a, la = od.decode(*args, np.zeros_like(one), [L], tile, 1)
    b_, lb = od.decode(*args, one, [L], tile, 1)
    assert np.abs(a - b_).max() < 1e-12 and np.abs(la - lb).max() < 1e-12


def test_per_batch_mask_rows_select_their_own_batch_entry():
    """One mask row per batch entry (words [B, Hk, W]): entry b must equal the single-sequence step on
    entry b's cache with entry b's row, and differ from what the other entry's row gives."""
    B, Hq, Hk, L, d, tile, G = 2, 4, 2, 260, 32, 64, 1
    c = _case(B, Hq, Hk, L, d, tile, G, seed=7, lens=[260, 131])
    rng = np.random.default_rng(8)
    route = (rng.random((B, Hk, -(-L // (tile * G)))) < 0.5).astype(np.uint8)
    route[1] = 1 - route[0]
    words = od.pack_row(route)
    assert words.shape[0] == B
    out, lse = _run(c, words=words)
    for b in range(B):
        sl = slice(b, b + 1)
        one = od.decode(c["q16"][sl], c["k16"][sl], c["k8"][sl], c["ks"][sl], c["v8"][sl], c["vs"][sl],
                        words[sl], c["lens"][sl], tile, G)
        assert np.array_equal(one[0][0], out[b]) and np.array_equal(one[1][0], lse[b])
        other = od.decode(c["q16"][sl], c["k16"][sl], c["k8"][sl], c["ks"][sl], c["v8"][sl], c["vs"][sl],
                          words[1 - b:2 - b], c["lens"][sl], tile, G)
        assert np.abs(other[0][0] - out[b]).max() > 1e-5
    # and against explicit loops for one head of entry 1 (its own row, not entry 0's)
    half = lambda bits: float(np.array(bits, np.uint16).view(np.float16))
    b, hq, hk = 1, 3, 1
    qv = [half(x) for x in c["q16"][b, hq]]
    q8, dq = od.quantize_query(c["q16"])
    s = []
    for j in range(131):
        g = j // (tile * G)
        if route[b, hk, g]:
            dot = sum(int(a) * int(x) for a, x in zip(q8[b, hq], c["k8"][b, hk, j]))
            s.append(float(dq[b, hq]) * float(c["ks"][b, hk, j // tile]) * dot / math.sqrt(d))
        else:
            s.append(sum(a * half(x) for a, x in zip(qv, c["k16"][b, hk, j])) / math.sqrt(d))
    m = max(s)
    w = [math.exp(x - m) for x in s]
    for e in range(0, d, 7):
        o = sum(w[j] * float(c["vs"][b, hk, j // tile]) * int(c["v8"][b, hk, j, e]) for j in range(131)) / sum(w)
        assert abs(o - out[b, hq, e]) < 1e-12


# ---- chunked prefill against an INT8 value cache (chunk_v8) -------------------------------------------------------

def _chunk_case(B, Hq, Hk, Lk, Lq, d, tile, G, seed, f8=0.5, pow2_v=False, blk_q=0):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, Hq, Lk, d)).astype(np.float16)          # the whole context's queries; the chunk = last Lq
    k = rng.standard_normal((B, Hk, Lk, d)).astype(np.float16)
    v = rng.standard_normal((B, Hk, Lk, d)).astype(np.float16)
    q16 = np.ascontiguousarray(Q.view(np.uint16)); k16 = np.ascontiguousarray(k.view(np.uint16))
    q8, qs = oracle.quantize(q16, blk_q or tile)
    k8, ks = oracle.quantize(k16, tile)
    if pow2_v:
        v8 = rng.integers(-127, 128, (B, Hk, Lk, d)).astype(np.int8)
        vs = (2.0 ** rng.integers(-6, -2, (B, Hk, -(-Lk // tile)))).astype(np.float32)
    else:
        v8, vs = oracle.quantize(np.ascontiguousarray(v.view(np.uint16)), tile)
    p = oracle.Problem(B, Hq, Hk, Lk, d, tile, tile, G, blk_q=blk_q)
    route = (rng.random((1, Hk, p.T_m, p.T_mask)) < f8).astype(np.uint8)
    words, _ = oracle.pack(p, route)
    off = Lk - Lq
    bq = blk_q or tile
    chunk = dict(q16=np.ascontiguousarray(q16[:, :, off:]), q8=np.ascontiguousarray(q8[:, :, off:]),
                 qs=np.ascontiguousarray(qs[:, :, off // bq:]))
    return dict(p=p, q16=q16, q8=q8, qs=qs, k16=k16, k8=k8, ks=ks, v8=v8, vs=vs, route=route, words=words, off=off,
                chunk=chunk, tile=tile, G=G, blk_q=blk_q)


def _chunk_run(c):
    ch = c["chunk"]
    return od.chunk_v8(ch["q16"], ch["q8"], ch["qs"], c["k16"], c["k8"], c["ks"], c["v8"], c["vs"], c["words"],
                       c["tile"], c["G"], blk_q=c["blk_q"])


def test_chunk_v8_with_a_lossless_value_cache_equals_the_prefill_oracle_rows():
    """Power-of-two block scales make delta_V * V8 exactly representable in FP16: the chunk against the INT8 value
    cache must then equal the already pinned prefill oracle on the same rows of the whole context (GQA, grouping
    factor 2, mixed routes, a ragged last tile)."""
    B, Hq, Hk, Lk, Lq, d, tile, G = 2, 4, 2, 300, 172, 32, 64, 2
    c = _chunk_case(B, Hq, Hk, Lk, Lq, d, tile, G, seed=11, pow2_v=True)
    blk = np.arange(Lk) // tile
    v16 = (c["v8"].astype(np.float64) * c["vs"][:, :, blk, None].astype(np.float64)).astype(np.float16)
    assert np.array_equal(v16.astype(np.float64), c["v8"].astype(np.float64) * c["vs"][:, :, blk, None].astype(np.float64))
    rows = [(b, h, c["off"] + i) for b in range(B) for h in range(Hq) for i in range(0, Lq, 7)] + \
           [(b, h, Lk - 1) for b in range(B) for h in range(Hq)]
    ref, ref_lse, _ = oracle.attention_rows(c["p"], c["q16"], c["k16"], np.ascontiguousarray(v16.view(np.uint16)),
                                            c["q8"], c["k8"], c["qs"], c["ks"], c["words"], rows)
    out, lse = _chunk_run(c)
    for n, (b, h, i) in enumerate(rows):
        assert np.abs(out[b, h, i - c["off"]] - ref[n]).max() < 1e-12
        assert abs(lse[b, h, i - c["off"]] - ref_lse[n]) < 1e-12
    assert c["route"].any() and not c["route"].all()


def test_chunk_v8_of_one_query_is_the_decode_step():
    """L_q = 1 with single-row query blocks: the chunk is the decode step over the same cache (the decode oracle
    quantises the query row itself and takes one mask row per KV head)."""
    B, Hq, Hk, Lk, d, tile, G = 2, 4, 2, 257, 32, 64, 1
    c = _chunk_case(B, Hq, Hk, Lk, 1, d, tile, G, seed=12, blk_q=1)
    out, lse = _chunk_run(c)
    last = c["route"][:, :, c["p"].T_m - 1]                               # the mask row of the last query tile
    ref, ref_lse = od.decode(np.ascontiguousarray(c["chunk"]["q16"][:, :, 0]), c["k16"], c["k8"], c["ks"], c["v8"],
                             c["vs"], od.pack_row(last), np.full(B, Lk), tile, G)
    assert np.abs(out[:, :, 0] - ref).max() < 1e-12 and np.abs(lse[:, :, 0] - ref_lse).max() < 1e-12
    q8_row, dq_row = od.quantize_query(np.ascontiguousarray(c["chunk"]["q16"][:, :, 0]))
    assert np.array_equal(q8_row, c["chunk"]["q8"][:, :, 0]) and np.array_equal(dq_row, c["chunk"]["qs"][:, :, 0])


def test_chunk_v8_brute_force_loops():
    B, Hq, Hk, Lk, Lq, d, tile, G = 1, 2, 1, 96, 32, 8, 32, 2
    c = _chunk_case(B, Hq, Hk, Lk, Lq, d, tile, G, seed=13)
    out, lse = _chunk_run(c)
    half = lambda bits: float(np.array(bits, np.uint16).view(np.float16))
    scale = 1.0 / math.sqrt(d)
    for hq in range(Hq):
        for i in (0, 5, 31):
            cpos = c["off"] + i
            s = []
            for j in range(cpos + 1):
                g = j // (tile * G)
                if (int(c["words"][0, 0, cpos // tile, g >> 5]) >> (g & 31)) & 1:
                    dot = sum(int(a) * int(b) for a, b in zip(c["chunk"]["q8"][0, hq, i], c["k8"][0, 0, j]))
                    s.append(float(c["chunk"]["qs"][0, hq, i // tile]) * float(c["ks"][0, 0, j // tile]) * dot * scale)
                else:
                    s.append(sum(half(a) * half(b) for a, b in zip(c["chunk"]["q16"][0, hq, i], c["k16"][0, 0, j])) * scale)
            m = max(s)
            w = [math.exp(x - m) for x in s]
            for e in range(d):
                o = sum(w[j] * float(c["vs"][0, 0, j // tile]) * int(c["v8"][0, 0, j, e]) for j in range(cpos + 1)) / sum(w)
                assert abs(o - out[0, hq, i, e]) < 1e-12
            assert abs(m + math.log(sum(w)) - lse[0, hq, i]) < 1e-12
    assert c["route"].any() and not c["route"].all()
