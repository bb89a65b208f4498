"""The entry point for callers that cannot allocate device memory (tilemix_attention_fwd_noalloc) must
give what tilemix_attention_fwd gives.  Kept in a file that pytest collects last."""
import pytest
import torch

from paper_2608_17336_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_noalloc_entry_matches_regular_entry_twice_in_a_row():
    """Two different problems, one after the other, through the built-in workspace: each must equal the
    regular entry point's output (same kernel, so bit for bit, which is within the 2e-3 the other tests
    use), the second call must not be disturbed by what the first left in the shared workspace, and the
    status record read back through the returned address must be clean.  The comparison is with the regular
    entry point, which the other tests compare with the oracle.  torch.cuda.memory_allocated() only sees torch's
    own allocator: that the entry point makes no allocation call of its own is a property of its source (it
    calls cudaGetSymbolAddress, cudaMemsetAsync and the launch, nothing else), not something this test can see."""
    from paper_2608_17336_b200 import binding as b
    dev = torch.device("cuda:0")
    cases = [
        synth.Workload("noalloc_a", 1, 2, 896, 128, 128, 2, seed=41, routing="bernoulli", int8_fraction=0.5),
        synth.Workload("noalloc_b", 2, 1, 333, 64, 64, 1, seed=42, routing="bernoulli", int8_fraction=0.7),
    ]
    addresses = []
    for w in cases:
        q, k, v = (t.to(dev) for t in synth.make_qkv(w))
        route = torch.from_numpy(synth.make_route(w)).to(dev)
        p = H.gpu_problem(w)
        q8, k8, qs, ks = b.tilemix_quantize_qk(p, q, k)
        words, _ = b.tilemix_pack_routing_mask(p, route, w.pin_diagonal)
        ref = b.tilemix_attention_fwd(p, q, k, v, q8, k8, qs, ks, words, want_lse=True)
        assert b.tilemix_read_status(ref["workspace"])[0] == 0
        # everything the call needs exists before it: the call itself allocates nothing
        out = torch.full_like(ref["out"], float("nan"))
        lse = torch.full_like(ref["lse"], float("nan"))
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        addr = b.tilemix_attention_fwd_noalloc(p, q, k, v, q8, k8, qs, ks, words, out, lse)
        code, rec = b.tilemix_read_status_at(addr)
        assert torch.cuda.memory_allocated() == before
        assert code == 0, rec
        addresses.append(addr)
        assert torch.isfinite(out).all()
        assert (out.float() - ref["out"].float()).abs().max().item() <= H.ATOL
        assert torch.equal(out, ref["out"]) and torch.equal(lse, ref["lse"])
    assert addresses[0] == addresses[1] and addresses[0] != 0      # one array per device, reused


def test_noalloc_entry_rejects_bad_arguments_before_launch():
    import ctypes
    from paper_2608_17336_b200 import binding as b
    p = b.problem(1, 2, 2, 512, 128, 128, 128)
    lib = b.lib()
    args = [ctypes.c_void_p(0x1000)] * 9
    assert lib.tilemix_attention_fwd_noalloc(None, *args, None, None, None, None) == b.ERR_NULL
    bad = b.problem(1, 2, 2, 0, 128, 128, 128)
    assert lib.tilemix_attention_fwd_noalloc(ctypes.byref(bad), *args, None, None, None, None) == b.ERR_SHAPE
    assert lib.tilemix_attention_fwd_noalloc(ctypes.byref(p), None, *args[1:], None, None, None, None) == b.ERR_NULL
    odd = b.problem(1, 2, 2, 512, 128, 64, 64)
    assert lib.tilemix_attention_fwd_noalloc(ctypes.byref(odd), *args, None, None, None, None) == b.ERR_UNSUPPORTED
    # a stride that is not a multiple of 16 bytes: the code tilemix_attention_fwd gives, not a generic one
    skew = b.problem(1, 2, 2, 512, 128, 128, 128)
    skew.q_stride[0], skew.q_stride[1], skew.q_stride[2] = 2 * 512 * 132, 512 * 132, 132
    ws = ctypes.c_void_p(0x1000)
    assert lib.tilemix_attention_fwd(ctypes.byref(skew), *args, None, ws, 4096, None, None) == b.ERR_ALIGN
    assert lib.tilemix_attention_fwd_noalloc(ctypes.byref(skew), *args, None, None, None, None) == b.ERR_ALIGN
