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


# ------------------------------------------------------------------ variable-length batches

def varlen_inputs(cu, heads_q, heads_kv, head_dim, tile, group, seed, int8_fraction=0.5):
    """Seeded packed batch: q [total,Hq,d], k/v [total,Hk,d] CPU half tensors and a byte map
    route [Hk, sum T_m, T_mask_max] with Bernoulli(int8_fraction) entries."""
    total = cu[-1]
    gen = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((total, heads_q, head_dim), generator=gen).half()
    k = torch.randn((total, heads_kv, head_dim), generator=gen).half()
    v = torch.randn((total, heads_kv, head_dim), generator=gen).half()
    lens = [cu[s + 1] - cu[s] for s in range(len(cu) - 1)]
    rows = sum(-(-L // tile) for L in lens)
    t_mask_max = max(1, -(-max(lens) // (group * tile)))
    rng = np.random.default_rng(seed + 1)
    route = (rng.random((heads_kv, rows, t_mask_max)) < int8_fraction).astype(np.uint8)
    return q, k, v, route


def varlen_oracle(cu, q, k, v, route, tile, group, pin_diagonal=False, seqs=None):
    """The dense oracle applied to every sequence of a packed batch on its own (a variable-length
    batch is, by definition, independent causal problems laid end to end).  Returns one dict per
    sequence (None for an empty or skipped one) with q8/k8/scales/words/out/lse and its offsets."""
    Hq, Hk, d = q.shape[1], k.shape[1], q.shape[2]
    res, row0 = [], 0
    for s in range(len(cu) - 1):
        t0, t1 = cu[s], cu[s + 1]
        L = t1 - t0
        T_m = -(-L // tile)
        if L == 0 or (seqs is not None and s not in seqs):
            res.append(None)
            row0 += T_m
            continue
        p = oracle.Problem(1, Hq, Hk, L, d, tile, tile, group)
        qb, kb, vb = (np_bits(t[t0:t1].permute(1, 0, 2)[None]) for t in (q, k, v))
        q8, qs = oracle.quantize(qb, p.bq)
        k8, ks = oracle.quantize(kb, p.bk)
        r = np.ascontiguousarray(route[None, :, row0:row0 + T_m, :p.T_mask])
        words, counts = oracle.pack(p, r, pin_diagonal)
        out, lse, _ = oracle.attention_full(p, qb, kb, vb, q8, k8, qs, ks, words)
        res.append(dict(p=p, tok0=t0, row0=row0, q8=q8, k8=k8, qs=qs, ks=ks, words=words, counts=counts,
                        out=out, lse=lse, qb=qb, kb=kb))
        row0 += T_m
    return res


def run_gpu_varlen(cu, q, k, v, route, tile, group, pin_diagonal=False, flags=0, debug_tiles=None,
                   max_seqlen=0):
    from paper_2608_17336_b200 import binding
    dev = torch.device("cuda:0")
    Hq, Hk, d = q.shape[1], k.shape[1], q.shape[2]
    p = binding.problem(1, Hq, Hk, cu[-1], d, tile, tile, group, flags=flags)
    vl = binding.Varlen(cu, max_seqlen)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    q8, k8, qs, ks = binding.tilemix_quantize_qk_varlen(p, vl, qd, kd)
    words, counts = binding.tilemix_pack_routing_mask_varlen(p, vl, torch.from_numpy(route).to(dev), pin_diagonal)
    res = binding.tilemix_attention_fwd_varlen(p, vl, qd, kd, vd, q8, k8, qs, ks, words, want_lse=True,
                                               debug_tiles=debug_tiles)
    code, rec = binding.tilemix_read_status(res["workspace"])
    assert code == 0, f"device status {rec}"
    res.update(q8=q8, k8=k8, qs=qs, ks=ks, words=words, counts=counts, p=p, vl=vl)
    return res
