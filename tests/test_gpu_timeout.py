"""The bounded waits of the kernels, seen running out -- without a fault, a trap or an endless loop.

A testing switch of the library makes a producer leave out one copy, so that the wait for it runs out after a few
milliseconds; the CTA then records a status, every role stops, what is in flight is waited for and the kernel
returns.  The tests read the status record and then use the same workspace for a normal call."""
import numpy as np
import pytest
import torch

from oracle import decode as od
from paper_2608_17336_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# role / barrier numbers of the attention kernel's status record
ROLE_SOFTMAX_A, ROLE_SOFTMAX_B, ROLE_PRODUCER, ROLE_MMA = 0, 1, 2, 3
BAR_RING_FULL, BAR_RING_EMPTY, BAR_S = 1, 2, 3


@pytest.fixture
def drop():
    from paper_2608_17336_b200 import binding as tm
    yield tm.tilemix_test_drop_copy
    tm.tilemix_test_drop_copy(0)        # always back to normal operation


def test_attention_wait_runs_out_and_the_kernel_returns(drop):
    from paper_2608_17336_b200 import binding as tm
    w = synth.Workload("timeout", 1, 2, 1024, 128, 128, 1, seed=91, routing="bernoulli", int8_fraction=0.5)
    q, k, v = (t.to(DEV) for t in synth.make_qkv(w))
    route = torch.from_numpy(synth.make_route(w)).to(DEV)
    p = H.gpu_problem(w)
    q8, k8, qs, ks = tm.tilemix_quantize_qk(p, q, k)
    words, _ = tm.tilemix_pack_routing_mask(p, route, False)
    good = tm.tilemix_attention_fwd(p, q, k, v, q8, k8, qs, ks, words)
    assert tm.tilemix_read_status(good["workspace"])[0] == 0
    ws = good["workspace"]
    drop(1, 2_000_000)                  # the wait for operand bundle 1 runs out after 2 ms
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    bad = tm.tilemix_attention_fwd(p, q, k, v, q8, k8, qs, ks, words, workspace=ws)
    t1.record()
    code, rec = tm.tilemix_read_status(bad["workspace"])
    assert code == tm.ERR_DEVICE_TIMEOUT
    # Every role waits with the same limit and the first to run out writes the record: the issuer waiting for
    # bundle 1, the producer waiting for the ring slot that the stalled issuer never frees, or a softmax warp
    # waiting for the scores of the stalled step.  Which of them started its wait first is a matter of timing.
    role, index, bar = rec[1], rec[2], rec[3]
    assert ((role == ROLE_MMA and index == 1 and bar == BAR_RING_FULL)
            or (role == ROLE_PRODUCER and bar == BAR_RING_EMPTY)
            or (role in (ROLE_SOFTMAX_A, ROLE_SOFTMAX_B) and bar == BAR_S)), rec
    assert t0.elapsed_time(t1) < 500.0            # it returned after the short limit, not after the default 2 s
    drop(0)
    again = tm.tilemix_attention_fwd(p, q, k, v, q8, k8, qs, ks, words, workspace=ws)
    assert tm.tilemix_read_status(again["workspace"])[0] == 0
    assert torch.equal(again["out"], good["out"])


def test_decode_wait_runs_out_and_the_kernel_returns(drop):
    from paper_2608_17336_b200 import binding as tm
    B, Hq, Hk, L, d, tile = 2, 4, 2, 1500, 128, 128
    gen = torch.Generator(device="cpu").manual_seed(92)
    q = torch.randn((B, Hq, d), generator=gen).half().to(DEV)
    k = torch.randn((B, Hk, L, d), generator=gen).half().to(DEV)
    v = torch.randn((B, Hk, L, d), generator=gen).half().to(DEV)
    k8, v8, ks, vs = tm.tilemix_quantize_qk(tm.problem(B, Hk, Hk, L, d, tile, tile), k, v)
    route = (np.random.default_rng(1).random((1, Hk, -(-L // tile))) < 0.5).astype(np.uint8)
    words = torch.from_numpy(od.pack_row(route).view(np.int32)).to(DEV)
    lens = torch.from_numpy(np.asarray([1500, 900], np.int32)).to(DEV)
    p = tm.decode_problem(B, Hq, Hk, d, L, tile, 1, n_splits=2)      # every split has several tiles
    good = tm.tilemix_decode_int8kv(p, q, k, k8, ks, v8, vs, words, lens)
    assert tm.tilemix_read_status(good["workspace"])[0] == 0
    drop(2, 2_000_000)
    bad = tm.tilemix_decode_int8kv(p, q, k, k8, ks, v8, vs, words, lens, workspace=good["workspace"])
    code, rec = tm.tilemix_read_status(bad["workspace"])
    assert code == tm.ERR_DEVICE_TIMEOUT, rec
    drop(0)
    again = tm.tilemix_decode_int8kv(p, q, k, k8, ks, v8, vs, words, lens, workspace=good["workspace"])
    assert tm.tilemix_read_status(again["workspace"])[0] == 0
    assert torch.equal(again["out"], good["out"])


def test_quantiser_wait_runs_out_and_the_kernel_returns(drop):
    """The streaming quantiser has no status record: a CTA whose wait for a block runs out stops, waits for its copies
    in flight and marks the scales of the blocks it did not finish with NaN."""
    from paper_2608_17336_b200 import binding as tm
    B, Hh, L, d = 1, 32, 4096, 128                     # 2 x 1024 blocks: every persistent CTA has well over two
    gen = torch.Generator(device="cpu").manual_seed(93)
    q = torch.randn((B, Hh, L, d), generator=gen).half().to(DEV)
    k = torch.randn((B, Hh, L, d), generator=gen).half().to(DEV)
    p = tm.problem(B, Hh, Hh, L, d, 128, 128)
    good = tm.tilemix_quantize_qk(p, q, k)
    assert all(torch.isfinite(x).all() for x in good[2:])
    drop(3, 2_000_000)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    bad = tm.tilemix_quantize_qk(p, q, k)
    t1.record()
    torch.cuda.synchronize()
    scales = torch.cat([bad[2].flatten(), bad[3].flatten()])          # the launch's blocks in order: Q's, then K's
    n_ctas = torch.cuda.get_device_properties(0).multi_processor_count
    assert torch.isnan(scales[n_ctas:2 * n_ctas]).all()               # block 1 of CTA c is block c + n_ctas of the launch
    assert torch.isfinite(scales[:n_ctas]).all()                      # block 0 of every CTA was finished
    assert t0.elapsed_time(t1) < 500.0
    drop(0)
    again = tm.tilemix_quantize_qk(p, q, k)
    assert all(torch.equal(a, g) for a, g in zip(again, good))
