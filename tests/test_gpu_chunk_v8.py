"""Chunked prefill against an INT8 value cache (tilemix_attention_fwd_chunk_v8) on the GPU: against the float64
oracle on every row, and bit for bit against the FP16-value chunk entry point where the two must coincide."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from oracle import decode as od
from paper_2608_17336_b200 import synth
from tests.helpers import ATOL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _bits(t):
    return np.ascontiguousarray(t.cpu().view(torch.int16).numpy()).view(np.uint16)


def _setup(B, Hq, Hk, Lk, Lq, d, tile, G, seed, f8=0.5):
    from paper_2608_17336_b200 import binding as tm
    gen = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, Hq, Lk, d), generator=gen).half().to(DEV)      # the whole context's queries; the chunk = last Lq
    k = torch.randn((B, Hk, Lk, d), generator=gen).half().to(DEV)
    v = (torch.randn((B, Hk, Lk, d), generator=gen) * 1.5).half().to(DEV)
    p_ctx = tm.problem(B, Hq, Hk, Lk, d, tile, tile, G)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p_ctx, q, k)
    # the value cache: the library's blockwise quantiser with V as its K operand (as for the decode step)
    _, v8, _, vs = tm.tilemix_quantize_qk(tm.problem(B, Hk, Hk, Lk, d, tile, tile), k, v)
    T_m, T_mask = -(-Lk // tile), -(-Lk // (tile * G))
    rng = np.random.default_rng(seed + 1)
    route = (rng.random((1, Hk, T_m, T_mask)) < f8).astype(np.uint8)
    words, _ = tm.tilemix_pack_routing_mask(p_ctx, torch.from_numpy(route).to(DEV), False)
    off = Lk - Lq
    chunk = dict(q=q[:, :, off:].contiguous(), q8=q8[:, :, off:].contiguous(), qs=qs[:, :, off // tile:].contiguous())
    return dict(tm=tm, q=q, k=k, v=v, q8=q8, k8=k8, qs=qs, ks=ks, v8=v8, vs=vs, route=route, words=words, off=off,
                chunk=chunk, p_chunk=tm.problem(B, Hq, Hk, Lq, d, tile, tile, G), shape=(B, Hq, Hk, Lk, Lq, d, tile, G))


def _check_against_oracle(c):
    tm = c["tm"]
    B, Hq, Hk, Lk, Lq, d, tile, G = c["shape"]
    ch = c["chunk"]
    res = tm.tilemix_attention_fwd_chunk_v8(c["p_chunk"], Lk, ch["q"], c["k"], c["v8"], c["vs"], ch["q8"], c["k8"],
                                            ch["qs"], c["ks"], c["words"], want_lse=True)
    torch.cuda.synchronize()
    assert tm.tilemix_read_status(res["workspace"])[0] == 0
    # what the oracle is given from the CUDA path is checked first: the quantised operands and the value cache
    v8_ref, vs_ref = oracle.quantize(_bits(c["v"]), tile)
    assert np.array_equal(c["v8"].cpu().numpy(), v8_ref)
    assert np.array_equal(c["vs"].cpu().numpy().view(np.uint32), vs_ref.view(np.uint32))
    q8_ref, qs_ref = oracle.quantize(_bits(c["q"]), tile)
    k8_ref, ks_ref = oracle.quantize(_bits(c["k"]), tile)
    assert np.array_equal(c["q8"].cpu().numpy(), q8_ref) and np.array_equal(c["k8"].cpu().numpy(), k8_ref)
    words_ref, _ = oracle.pack(oracle.Problem(B, Hq, Hk, Lk, d, tile, tile, G), c["route"])
    assert np.array_equal(c["words"].cpu().numpy().view(np.uint32), words_ref)
    off = c["off"]
    ref, ref_lse = od.chunk_v8(_bits(ch["q"]), q8_ref[:, :, off:], qs_ref[:, :, off // tile:], _bits(c["k"]), k8_ref,
                               ks_ref, v8_ref, vs_ref, words_ref, tile, G)
    out = res["out"].float().cpu().numpy().astype(np.float64)
    err = np.abs(out - ref)
    assert (err <= ATOL * np.maximum(1.0, np.abs(ref))).all(), f"max err {err.max():.3e}"
    assert np.abs(res["lse"].cpu().numpy().astype(np.float64) - ref_lse).max() < 2e-3
    return res


@pytest.mark.parametrize("d,tile,Lk,Lq", [(128, 128, 1024, 384), (128, 128, 900, 260), (64, 64, 640, 192)])
def test_chunk_v8_every_row_against_the_oracle(d, tile, Lk, Lq):
    _check_against_oracle(_setup(2, 4, 2, Lk, Lq, d, tile, 2, seed=61))


def test_chunk_v8_whole_context_and_single_tile_chunks():
    _check_against_oracle(_setup(1, 2, 1, 512, 512, 128, 128, 1, seed=62))      # a prefill against a fresh cache
    _check_against_oracle(_setup(1, 8, 1, 640, 128, 128, 128, 3, seed=63, f8=0.8))   # one tile of new queries, GQA 8


def test_chunk_v8_equals_the_fp16_value_chunk_when_the_cache_is_lossless():
    """Integer values with unit block scales: the FP16 image of the cache is the FP16 V operand itself and the
    probabilities are multiplied by 1, so the two entry points must agree bit for bit.  With power-of-two scales
    delta_V * V8 is still exact in FP16 and only the rounding of the probabilities differs (a probability that is
    subnormal in FP16 before or after the scaling keeps a different number of bits): equal within FP16 rounding."""
    c = _setup(2, 4, 2, 768, 256, 128, 128, 2, seed=64)
    tm = c["tm"]
    B, Hq, Hk, Lk, Lq, d, tile, G = c["shape"]
    rng = np.random.default_rng(65)
    v8 = torch.from_numpy(rng.integers(-127, 128, (B, Hk, Lk, d)).astype(np.int8)).to(DEV)
    ch = c["chunk"]
    for pow2 in (False, True):
        k2 = rng.integers(-5, 1, (B, Hk, Lk // tile)) if pow2 else np.zeros((B, Hk, Lk // tile))
        vs = torch.from_numpy((2.0 ** k2).astype(np.float32)).to(DEV)
        v16 = (v8.float() * vs.repeat_interleave(tile, 2)[..., None]).half()
        assert torch.equal(v16.float(), v8.float() * vs.repeat_interleave(tile, 2)[..., None])
        a = tm.tilemix_attention_fwd_chunk_v8(c["p_chunk"], Lk, ch["q"], c["k"], v8, vs, ch["q8"], c["k8"], ch["qs"],
                                              c["ks"], c["words"], want_lse=True)
        b = tm.tilemix_attention_fwd_chunk(c["p_chunk"], Lk, ch["q"], c["k"], v16, ch["q8"], c["k8"], ch["qs"], c["ks"],
                                           c["words"], want_lse=True)
        assert torch.equal(a["lse"], b["lse"])
        if pow2:
            assert (a["out"].float() - b["out"].float()).abs().max().item() <= 2e-3 * b["out"].float().abs().max().item()
        else:
            assert torch.equal(a["out"], b["out"])


def test_chunk_v8_scale_really_is_applied_per_block():
    """Doubling delta_V of one block must change the rows that see that block and no row before it."""
    c = _setup(1, 2, 1, 512, 512, 128, 128, 1, seed=66)
    tm = c["tm"]
    ch = c["chunk"]
    run = lambda vs: tm.tilemix_attention_fwd_chunk_v8(c["p_chunk"], 512, ch["q"], c["k"], c["v8"], vs, ch["q8"], c["k8"],
                                                       ch["qs"], c["ks"], c["words"])["out"]
    base = run(c["vs"])
    vs2 = c["vs"].clone(); vs2[:, :, 2] *= 2.0
    other = run(vs2)
    assert torch.equal(base[:, :, :256], other[:, :, :256]) and not torch.equal(base[:, :, 256:], other[:, :, 256:])
