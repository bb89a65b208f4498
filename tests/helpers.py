"""Shared test plumbing: runs one synthetic workload through the CUDA path (via the C ABI
binding) and through the CPU oracle on the same seeded inputs.  The oracle is evaluated on a
subset of heads / rows so that it finishes in seconds at any size."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2608_17336_b200 import synth

ATOL = 2e-3          # max-abs tolerance on FP16 outputs of unit-scale inputs


def np_bits(t: torch.Tensor) -> np.ndarray:
    """CPU half tensor -> uint16 bit patterns (contiguous)."""
    return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy()).view(np.uint16)


def oracle_problem(w: synth.Workload, heads=None, batch=None) -> oracle.Problem:
    H = w.heads if heads is None else heads
    B = w.batch if batch is None else batch
    nb = w.mask_batch if w.mask_batch == 1 else B
    return oracle.Problem(B, H, H, w.seqlen, w.head_dim, w.tile, w.tile, w.group, mask_batch=nb)


def gpu_problem(w: synth.Workload, flags=0):
    from paper_2608_17336_b200 import binding
    return binding.problem(w.batch, w.heads, w.heads, w.seqlen, w.head_dim, w.tile, w.tile, w.group,
                           mask_batch=w.mask_batch, flags=flags)


def run_gpu(w: synth.Workload, q, k, v, route, debug_tiles=None, want_lse=True, flags=0):
    """Whole path on the GPU.  q,k,v: CPU half tensors; route: numpy uint8."""
    from paper_2608_17336_b200 import binding
    p = gpu_problem(w, flags)
    dev = torch.device("cuda:0")
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    rd = torch.from_numpy(route).to(dev)
    q8, k8, qs, ks = binding.tilemix_quantize_qk(p, qd, kd)
    words, counts = binding.tilemix_pack_routing_mask(p, rd, w.pin_diagonal)
    res = binding.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words, want_lse=want_lse,
                                        debug_tiles=debug_tiles)
    code, rec = binding.tilemix_read_status(res["workspace"])
    assert code == 0, f"device status {rec}"
    res.update(q8=q8, k8=k8, qs=qs, ks=ks, words=words, counts=counts)
    return res


def run_oracle(w: synth.Workload, q, k, v, route, heads, rows):
    """Oracle on the head subset `heads` (list) of batch entries `all`; rows = (b, h, i) with h
    indexing the ORIGINAL heads.  Returns dict with per-row outputs and the subset's operands."""
    heads = list(heads)
    hmap = {h: s for s, h in enumerate(heads)}
    p = oracle_problem(w, heads=len(heads))
    qb, kb, vb = (np_bits(t[:, heads]) for t in (q, k, v))
    q8, qs = oracle.quantize(qb, p.bq)
    k8, ks = oracle.quantize(kb, p.bk)
    words, counts = oracle.pack(p, np.ascontiguousarray(route[:, heads]), w.pin_diagonal)
    sub_rows = np.asarray([(b, hmap[h], i) for b, h, i in rows], np.int64)
    out, lse, rsum = oracle.attention_rows(p, qb, kb, vb, q8, k8, qs, ks, words, sub_rows)
    return dict(p=p, out=out, lse=lse, q8=q8, k8=k8, qs=qs, ks=ks, words=words, counts=counts,
                qb=qb, kb=kb, heads=heads)


def check_rows(gpu_out: torch.Tensor, ref: np.ndarray, rows, atol=ATOL):
    """|O_gpu - O_oracle| <= atol * max(1, |O_oracle|) on the listed rows; returns max abs error."""
    rows = np.asarray(rows, np.int64)
    idx = torch.from_numpy(rows)
    got = gpu_out[idx[:, 0], idx[:, 1], idx[:, 2]].float().cpu().numpy().astype(np.float64)
    err = np.abs(got - ref)
    bound = atol * np.maximum(1.0, np.abs(ref))
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), (f"max err {err.max():.3e}; worst row {rows[worst[0]].tolist()} col {worst[1]}: "
                                  f"gpu {got[worst]:.6f} oracle {ref[worst]:.6f}")
    return float(err.max())


def all_rows(w: synth.Workload, heads=None):
    heads = range(w.heads) if heads is None else heads
    return [(b, h, i) for b in range(w.batch) for h in heads for i in range(w.seqlen)]
