#!/usr/bin/env python
"""Benchmark of the TileMix hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3_long32k] [--impl reference]

A step is one pass of the whole hot path -- tilemix_quantize_qk, tilemix_pack_routing_mask,
tilemix_attention_fwd -- over one synthetic batch that is already resident in HBM.  The metric
is effective causal-attention TFLOP/s (4*B*H*L^2*d/2 FLOP per step).  Prints ONE JSON line
(rank 0).  With N > 1 every rank runs its own batch of the same shape (no data-path
collective: every (batch, head) is independent), launched by torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2608_17336_b200 import synth  # noqa: E402

METRIC = "effective causal-attention TFLOP/s at 1 B200 vs INT8 fraction; % of mixed roofline"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
INT8_OVER_FP16 = 2.0     # nominal dense INT8 : FP16 tensor throughput ratio (4.5 : 2.25 PFLOP/s)
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from an ncu capture of the 8-head case of
# the workload (484.1 MB; the traffic scales with the head count).
NCU_DRAM_BYTES_PER_HEAD = {"cfg3_long32k": 484.1e6 / 8}


def effective_flops(w: synth.Workload) -> float:
    return 4.0 * w.batch * w.heads * float(w.seqlen) ** 2 * w.head_dim / 2.0


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = torch.cuda.get_device_properties(device_index).uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                get = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or nv.nvmlDeviceGetCurrentClocksThrottleReasons
                mask = get(self._h)
                self.reasons |= {k for k, bit in names.items() if mask & bit}
            except Exception:
                pass
            time.sleep(0.005)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample(w: synth.Workload, q, k, v, route, budget_pairs: float):
    """Times the CPU oracle, as it stands, on a bounded sample of `w`: hash-chosen query rows of
    head 0 of batch 0, as many as fit in about `budget_pairs` (query, key) pairs, plus the
    quantise and pack steps of that head.  Returns (seconds, pairs, n_rows, threads)."""
    import oracle

    def np_bits(t):      # CPU half tensor -> uint16 bit patterns
        return np.ascontiguousarray(t.contiguous().view(torch.int16).numpy()).view(np.uint16)

    order = np.argsort(synth.hash_uniform(w.seed + 77, 0, 0, np.arange(w.seqlen)), kind="stable")
    keep = np.cumsum(order + 1) <= budget_pairs
    keep[0] = True
    idx = np.sort(order[keep])
    rows = np.stack([np.zeros_like(idx), np.zeros_like(idx), idx], axis=1)
    p = oracle.Problem(1, 1, 1, w.seqlen, w.head_dim, w.tile, w.tile, w.group, mask_batch=1)
    qb, kb, vb = (np_bits(t[:1, :1]) for t in (q, k, v))
    t0 = time.perf_counter()
    q8, qs = oracle.quantize(qb, p.bq)
    k8, ks = oracle.quantize(kb, p.bk)
    words, _ = oracle.pack(p, np.ascontiguousarray(route[:1, :1]), w.pin_diagonal)
    oracle.attention_rows(p, qb, kb, vb, q8, k8, qs, ks, words, rows)
    dt = time.perf_counter() - t0
    return dt, int((rows[:, 2] + 1).sum()), len(rows), oracle.num_threads()


def rank_workload(w: synth.Workload, rank: int) -> synth.Workload:
    """Every rank runs its own batch of the same shape: same recipe, rank-dependent seed."""
    return w.scaled(seed=w.seed + 1000 * rank)


def max_over_ranks(values, device, world: int):
    """Element-wise maximum of per-rank device timings (the job is as slow as its slowest rank)."""
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def job_value(flops_per_rank: float, world: int, ms_per_step: float) -> float:
    """Whole-job effective TFLOP/s: all ranks' FLOPs over the slowest rank's step time."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def run_reference(args, w, rank, world):
    """--impl reference: the CPU oracle on the host cores, on a bounded sample per step."""
    if rank != 0:
        return
    q, k, v = synth.make_qkv(w.scaled(heads=1, batch=1))
    route = synth.make_route(w)
    w1 = w.scaled(heads=1, batch=1)
    times, pairs, n_rows, threads = [], 0, 0, 1
    for i in range(args.warmup + args.steps):
        dt, pairs, n_rows, threads = oracle_sample(w1, q, k, v, route, args.ref_pairs)
        if i >= args.warmup:
            times.append(dt)
    sec = sum(times) / len(times)
    tflops = 4.0 * w.head_dim * pairs / sec / 1e12
    sample = f"{n_rows} rows of head 0 ({pairs} query-key pairs) per step, incl. quantise+pack of that head"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": tflops, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "heads": w.heads, "seqlen": w.seqlen, "head_dim": w.head_dim,
                   "tile": w.tile, "group": w.group},
        "cpu_baseline": {"value": tflops, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": tflops, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def same_run_peaks(tm, dev) -> dict:
    """Tensor-throughput denominators measured in this run, on this GPU: (1) the library's own issue-rate probe
    (tcgen05.mma M128 N128 from shared memory, kind::f16 and kind::i8, one CTA per SM), (2) dense library GEMMs as a
    cross-check -- torch.matmul FP16 and torch._int_mm INT8 at 8192^3, as a short burst and as a ~1.5 s loop under
    the power cap.  Library calls serve as denominators only."""
    stream = torch.cuda.current_stream()
    out = {}
    ws = torch.zeros(16, dtype=torch.uint8, device=dev)
    for name, int8, k in (("tcgen05_f16", False, 16), ("tcgen05_i8", True, 32)):
        n_mma = 40000
        tm.tilemix_tensor_peak_probe(int8, 2000, ws)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ctas = tm.tilemix_tensor_peak_probe(int8, n_mma, ws)
        b.record(stream)
        torch.cuda.synchronize()
        if tm.tilemix_read_status(ws)[0] != 0:
            raise RuntimeError("tensor probe timed out")
        out[name] = ctas * n_mma * 2.0 * 128 * 128 * k / (a.elapsed_time(b) * 1e-3) / 1e12
    n = 8192
    x16 = torch.randn((n, n), device=dev, dtype=torch.float16)
    y16 = torch.randn((n, n), device=dev, dtype=torch.float16)
    x8 = torch.randint(-127, 128, (n, n), device=dev, dtype=torch.int8)
    y8 = torch.randint(-127, 128, (n, n), device=dev, dtype=torch.int8).t().contiguous().t()   # column-major operand
    ops = 2.0 * n ** 3

    def rate(fn, iters):
        for _ in range(3):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(iters):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return ops * iters / (a.elapsed_time(b) * 1e-3) / 1e12

    out["matmul_f16_burst"] = rate(lambda: torch.matmul(x16, y16), 10)
    out["matmul_f16_sustained"] = rate(lambda: torch.matmul(x16, y16), 1800)
    try:
        out["int_mm_i8_burst"] = rate(lambda: torch._int_mm(x8, y8), 10)
        out["int_mm_i8_sustained"] = rate(lambda: torch._int_mm(x8, y8), 3000)
    except Exception as exc:      # the INT8 library GEMM is optional: the probe above is the INT8 figure
        out["int_mm_i8_error"] = repr(exc)[:120]
    return out


def varlen_leg(tm, w: synth.Workload, dev, peaks) -> dict:
    """The same step over a packed variable-length batch (no padding): as many tokens as the dense
    workload, split into sequences of halving length (L/2, L/4, ... and two of the shortest), Bernoulli
    routing at the workload's INT8 fraction.  Reported beside the headline; not part of `value`."""
    total = w.batch * w.seqlen
    lens, rest = [], total
    while rest > 2 * 256 and len(lens) < 6:
        lens.append(rest // 2)
        rest -= lens[-1]
    lens += [rest // 2, rest - rest // 2]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64).tolist()
    gen = torch.Generator(device="cpu").manual_seed(w.seed + 7)
    qkv = [torch.randn((total, w.heads, w.head_dim), generator=gen).half().to(dev) for _ in range(3)]
    p = tm.problem(1, w.heads, w.heads, total, w.head_dim, w.tile, w.tile, w.group)
    vl = tm.Varlen(cu)
    c = tm.tilemix_varlen_counts(p, vl)
    rng = np.random.default_rng(w.seed + 8)
    route = torch.from_numpy((rng.random((w.heads, c["sum_T_m"], c["T_mask_max"])) < w.int8_fraction)
                             .astype(np.uint8)).to(dev)
    work = torch.empty(tm.tilemix_varlen_workspace_size(p, vl), dtype=torch.uint8, device=dev)
    out = torch.empty_like(qkv[0])
    stream = torch.cuda.current_stream()

    def step(ev=None):
        q8, k8, qs, ks = tm.tilemix_quantize_qk_varlen(p, vl, qkv[0], qkv[1], workspace=work)
        words, _ = tm.tilemix_pack_routing_mask_varlen(p, vl, route, w.pin_diagonal, workspace=work)
        if ev:
            ev[0].record(stream)
        tm.tilemix_attention_fwd_varlen(p, vl, *qkv, q8, k8, qs, ks, words, out=out, workspace=work)
        if ev:
            ev[1].record(stream)

    for _ in range(3):
        step()
    n = 5
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(stream)
    for i in range(n):
        step(evs[i])
    t1.record(stream)
    torch.cuda.synchronize()
    code, rec = tm.tilemix_read_status(work)
    if code != 0:
        raise RuntimeError(f"device status {rec}")
    flops = sum(4.0 * w.heads * float(L) ** 2 * w.head_dim / 2.0 for L in lens)
    step_ms = t0.elapsed_time(t1) / n
    attn_ms = sum(a.elapsed_time(b) for a, b in evs) / n
    return {"seqlens": lens, "tokens": total, "ms_per_step": step_ms, "attention_ms": attn_ms,
            "value": flops / (step_ms * 1e-3) / 1e12, "attention_tflops": flops / (attn_ms * 1e-3) / 1e12,
            "unit": "TFLOP/s"}


def decode_leg(tm, w: synth.Workload, dev, peaks) -> dict:
    """One decode step over an INT8 key/value cache of the workload's length: 8 sequences, the workload's
    heads as query heads over a quarter as many KV heads (GQA 4:1), Bernoulli routing at the workload's
    INT8 fraction.  HBM-bound: reported against the measured copy bandwidth.  Not part of `value`."""
    B, Hq, Hk, d, L = 8, w.heads, max(1, w.heads // 4), w.head_dim, w.seqlen
    gen = torch.Generator(device=dev).manual_seed(w.seed + 11)
    k = torch.randn((B, Hk, L, d), generator=gen, device=dev, dtype=torch.float16)
    v = torch.randn((B, Hk, L, d), generator=gen, device=dev, dtype=torch.float16)
    q = torch.randn((B, Hq, d), generator=gen, device=dev, dtype=torch.float16)
    k8, v8, ks, vs = tm.tilemix_quantize_qk(tm.problem(B, Hk, Hk, L, d, w.tile, w.tile), k, v)
    del v
    T_mask = -(-L // (w.tile * w.group))
    rng = np.random.default_rng(w.seed + 12)
    route = (rng.random((1, Hk, T_mask)) < w.int8_fraction)
    words = np.zeros((1, Hk, -(-T_mask // 32)), np.uint32)
    for g in range(T_mask):
        words[..., g >> 5] |= route[..., g].astype(np.uint32) << np.uint32(g & 31)
    f8 = float(route.mean())
    words_d = torch.from_numpy(words.view(np.int32)).to(dev)
    lens = torch.full((B,), L, dtype=torch.int32, device=dev)
    p = tm.decode_problem(B, Hq, Hk, d, L, w.tile, w.group)
    work = torch.empty(tm.tilemix_decode_workspace_size(p), dtype=torch.uint8, device=dev)
    out = torch.empty((B, Hq, d), dtype=torch.float16, device=dev)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        tm.tilemix_decode_int8kv(p, q, k, k8, ks, v8, vs, words_d, lens, out=out, workspace=work)
    n = 10
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    t0.record(stream)
    for _ in range(n):
        tm.tilemix_decode_int8kv(p, q, k, k8, ks, v8, vs, words_d, lens, out=out, workspace=work)
    t1.record(stream)
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / n
    # algorithmic bytes: per cached token d (V8) + d (K8, INT8 route) or 2d (FP16 K, FP16 route)
    nbytes = float(B) * Hk * L * d * (1.0 + f8 + 2.0 * (1.0 - f8))
    gbs = nbytes / (ms * 1e-3) / 1e9
    res = {"batch": B, "heads_q": Hq, "heads_kv": Hk, "cache_len": L, "int8_groups": f8, "ms_per_step": ms,
           "tokens_per_s": B / (ms * 1e-3), "bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]),
           "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]), "bytes_per_step": nbytes,
           "l2": "cache (0.8 GB) exceeds L2"}
    # the same cache with unequal lengths: the library's uniform split count against splits shared out over the
    # rows by the kernel (n_splits = -1)
    ragged = [L, L // 8, L // 16, L // 2, L // 32, L // 4, L // 64, (3 * L) // 4]
    lens_r = torch.tensor(ragged, dtype=torch.int32, device=dev)
    res["unequal_lengths"] = {"cache_len": ragged}
    for key, ns in (("uniform_splits_ms", 0), ("kernel_chosen_splits_ms", -1)):
        pr = tm.decode_problem(B, Hq, Hk, d, L, w.tile, w.group, n_splits=ns)
        work_r = torch.empty(tm.tilemix_decode_workspace_size(pr), dtype=torch.uint8, device=dev)
        for _ in range(3):
            tm.tilemix_decode_int8kv(pr, q, k, k8, ks, v8, vs, words_d, lens_r, out=out, workspace=work_r)
        torch.cuda.synchronize()
        t0.record(stream)
        for _ in range(n):
            tm.tilemix_decode_int8kv(pr, q, k, k8, ks, v8, vs, words_d, lens_r, out=out, workspace=work_r)
        t1.record(stream)
        torch.cuda.synchronize()
        res["unequal_lengths"][key] = t0.elapsed_time(t1) / n
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3_long32k", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="tilemix", choices=["tilemix", "reference"])
    ap.add_argument("--int8-fraction", type=float, default=None, help="override the workload's INT8 coverage")
    ap.add_argument("--ref-pairs", type=float, default=6e7, help="oracle sample size (query-key pairs per step)")
    ap.add_argument("--cpu-pairs", type=float, default=4e8, help="cpu_baseline sample size (pairs)")
    ap.add_argument("--heads", type=int, default=None, help="override the head count (smaller profiling cases)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the INT8-fraction sweep of the attention kernel")
    ap.add_argument("--no-varlen", action="store_true", help="skip the variable-length (packed batch) measurement")
    ap.add_argument("--no-decode", action="store_true", help="skip the INT8 KV-cache decode measurement")
    ap.add_argument("--no-peaks", action="store_true", help="skip the same-run tensor peak measurements")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "tilemix" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = synth.WORKLOADS[args.workload]
    if args.heads is not None:
        w = w.scaled(heads=args.heads)
    if args.int8_fraction is not None:
        routing = "zero" if args.int8_fraction <= 0 else "one" if args.int8_fraction >= 1 else w.routing
        w = w.scaled(int8_fraction=args.int8_fraction, routing=routing)

    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return

    from paper_2608_17336_b200 import binding as tm
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    w_rank = rank_workload(w, rank)

    q, k, v = synth.make_qkv(w_rank)
    route = synth.make_route(w_rank)
    p = tm.problem(w.batch, w.heads, w.heads, w.seqlen, w.head_dim, w.tile, w.tile, w.group, mask_batch=w.mask_batch)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    rd = torch.from_numpy(route).to(dev)
    out = torch.empty_like(qd)
    work = torch.empty(tm.tilemix_workspace_size(p), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(record=None):
        if record is not None:
            record[2].record(stream)
        q8, k8, qs, ks = tm.tilemix_quantize_qk(p, qd, kd)
        if record is not None:
            record[3].record(stream)
        words, counts = tm.tilemix_pack_routing_mask(p, rd, w.pin_diagonal)
        if record is not None:
            record[0].record(stream)
        tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words, out=out, workspace=work)
        if record is not None:
            record[1].record(stream)
        return counts

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        counts = step()
    code, rec = tm.tilemix_read_status(work)
    if code != 0:
        raise RuntimeError(f"device status {rec}")
    counts_h = counts.cpu().numpy()
    rho_groups = float(counts_h[..., 1].sum() / counts_h[..., 0].sum())

    # ---- timed region: K steps, device-timed, inputs (1 GiB+) far larger than L2 ----------------------
    launches0 = tm.tilemix_launch_count()
    kern_ev = [tuple(torch.cuda.Event(enable_timing=True) for _ in range(4)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    with ClockSampler(local_rank) as clocks:
        e0.record(stream)
        for i in range(args.steps):
            step(kern_ev[i])
        e1.record(stream)
        sync_all()
    launches = tm.tilemix_launch_count() - launches0
    total_ms = e0.elapsed_time(e1)
    attn_steps = sorted(ev[0].elapsed_time(ev[1]) for ev in kern_ev)
    attn_ms = sum(attn_steps) / args.steps
    quant_ms = sum(ev[2].elapsed_time(ev[3]) for ev in kern_ev) / args.steps
    pack_ms = sum(ev[3].elapsed_time(ev[0]) for ev in kern_ev) / args.steps
    code, rec = tm.tilemix_read_status(work)
    if code != 0:
        raise RuntimeError(f"device status {rec}")

    # ---- end to end through the host-buffer entry point (copies inside the timed region) ---------------
    e2e = None
    if not args.no_e2e:
        qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
        rh = torch.from_numpy(route).pin_memory()
        oh = torch.empty(q.shape, dtype=torch.float16).pin_memory()
        arena = torch.empty(tm.tilemix_arena_size(p), dtype=torch.uint8, device=dev)
        for _ in range(2):
            tm.tilemix_prefill_host(p, qh, kh, vh, rh, oh, arena, w.pin_diagonal)
        sync_all()
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(args.steps):
            tm.tilemix_prefill_host(p, qh, kh, vh, rh, oh, arena, w.pin_diagonal)
        h1.record(stream)
        sync_all()
        e2e_ms = h0.elapsed_time(h1) / args.steps
        e2e = {"ms": e2e_ms, "h2d": q.numel() * 2 * 3 + route.size, "d2h": q.numel() * 2,
               "checksum": float(oh.float().abs().mean())}
        del arena

    # ---- max over ranks ----------------------------------------------------------------------------------
    total_ms, attn_ms, e2e_ms = max_over_ranks([total_ms, attn_ms, e2e["ms"] if e2e else 0.0], dev, world)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    F = effective_flops(w)
    ms_per_step = total_ms / args.steps
    value = job_value(F, world, ms_per_step)
    peaks, peak_kind = load_peaks()
    # mask-weighted roofline: T = F_pv/P16 + F_qk*((1-f8)/P16 + f8/P8); f8 = INT8 share of legal tiles.
    # f8 from the realised mask: expand groups to tiles on or below the diagonal
    words, _ = tm.tilemix_pack_routing_mask(p, rd, w.pin_diagonal)
    wh = words.cpu().numpy().view(np.uint32)
    mm, nn = np.tril_indices(w.T_m)
    gg = nn // w.group
    bits = (wh[:, :, mm, gg >> 5] >> (gg & 31).astype(np.uint32)) & 1
    f8 = float(bits.mean())
    p16 = float(peaks["bf16_tflops"])
    p16_sus = float(peaks.get("bf16_tflops_sustained", p16))
    peak_eff = p16 / (1.0 - f8 * (1.0 - 1.0 / INT8_OVER_FP16) / 2.0)
    peak_eff_sus = p16_sus / (1.0 - f8 * (1.0 - 1.0 / INT8_OVER_FP16) / 2.0)
    achieved = F / (attn_ms * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f16+i8 (f32/s32 accumulate)", "data": "synthetic",
        "config": {"workload": w.name, "batch": w.batch, "heads": w.heads, "seqlen": w.seqlen, "head_dim": w.head_dim,
                   "tile": w.tile, "group": w.group, "int8_groups": rho_groups, "int8_tiles": f8,
                   "step": "quantize_qk + pack_routing_mask + attention_fwd", "l2": "inputs_exceed_l2",
                   "parallelism": f"replicas x{world}"},
        "gpu_launches": int(launches),
        "clocks": clocks.summary(),
        "roofline": {"bound": "tensor", "kernel": "attention_kernel", "achieved": achieved, "peak": peak_eff,
                     "unit": "TFLOP/s", "frac": achieved / peak_eff,
                     "traffic": (NCU_DRAM_BYTES_PER_HEAD[w.name] * w.heads * w.batch if w.name in NCU_DRAM_BYTES_PER_HEAD else None),
                     "traffic_unit": "bytes per launch (ncu dram read+write, scaled from an 8-head capture)",
                     "peak_source": f"{peak_kind}: bf16 burst {p16} TFLOP/s, INT8 = {INT8_OVER_FP16}x nominal ratio, "
                                    f"mask-weighted with f8={f8:.4f}",
                     "attention_ms": attn_ms, "attention_ms_min": attn_steps[0],
                     "attention_ms_median": statistics.median(attn_steps),
                     "peak_sustained": peak_eff_sus, "frac_sustained": achieved / peak_eff_sus,
                     "frac_note": "frac (against the burst peak) is the figure; frac_sustained is context"},
    }
    if world == 1 and not args.no_peaks:
        # the same mask-weighted roofline from denominators measured in this run
        sp = same_run_peaks(tm, dev)
        line["roofline"]["peaks_same_run"] = {k_: (round(v_, 1) if isinstance(v_, float) else v_) for k_, v_ in sp.items()}
        for tag, p16s, p8s in (("tcgen05", sp["tcgen05_f16"], sp["tcgen05_i8"]),
                               ("library", sp["matmul_f16_burst"], sp.get("int_mm_i8_burst"))):
            if p8s:
                t_roof = (F / 2) / p16s + (F / 2) * ((1.0 - f8) / p16s + f8 / p8s)
                line["roofline"]["frac_same_run_" + tag] = (F / t_roof) and achieved / (F / t_roof)
    # the HBM-bound pre-pass: 3 bytes per element of Q and K (2 read, 1 written)
    quant_bytes = 3.0 * 2 * w.batch * w.heads * w.seqlen * w.head_dim
    line["other_kernels"] = {
        "quantize_qk": {"ms": quant_ms, "bound": "hbm", "achieved": quant_bytes / (quant_ms * 1e-3) / 1e9,
                        "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                        "frac": quant_bytes / (quant_ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"])},
        "pack_routing_mask": {"ms": pack_ms}}
    if e2e:
        line["e2e"] = {"value": job_value(F, world, e2e_ms), "unit": "TFLOP/s", "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": int(e2e["h2d"]), "d2h_bytes_per_step": int(e2e["d2h"])}
    if world == 1 and not args.no_sweep:
        # the metric's "vs INT8 fraction" axis: same shapes and inputs, attention kernel only
        q8, k8, qs, ks = tm.tilemix_quantize_qk(p, qd, kd)
        sweep = []
        for frac in (0.0, 0.25, 0.5, 0.75, 1.0):
            ws = w_rank.scaled(int8_fraction=frac, pin_diagonal=False,
                               routing="zero" if frac == 0.0 else "one" if frac == 1.0 else "row_exact")
            words_s, _ = tm.tilemix_pack_routing_mask(p, torch.from_numpy(synth.make_route(ws)).to(dev), False)
            whs = words_s.cpu().numpy().view(np.uint32)
            f8s = float(((whs[:, :, mm, gg >> 5] >> (gg & 31).astype(np.uint32)) & 1).mean())
            for _ in range(3):
                tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words_s, out=out, workspace=work)
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(7)]
            for s0, s1 in evs:
                s0.record(stream)
                tm.tilemix_attention_fwd(p, qd, kd, vd, q8, k8, qs, ks, words_s, out=out, workspace=work)
                s1.record(stream)
            torch.cuda.synchronize()
            ms = statistics.median(s0.elapsed_time(s1) for s0, s1 in evs)   # median of 7 launches
            pk = p16 / (1.0 - f8s * (1.0 - 1.0 / INT8_OVER_FP16) / 2.0)
            sweep.append({"int8_tiles": round(f8s, 4), "attention_ms": round(ms, 4),
                          "tflops": round(F / (ms * 1e-3) / 1e12, 1), "frac": round(F / (ms * 1e-3) / 1e12 / pk, 4)})
        line["int8_sweep"] = sweep
    if world == 1 and not args.no_varlen and w.tile == 128:
        line["varlen"] = varlen_leg(tm, w, dev, peaks)
    if world == 1 and not args.no_decode and w.tile == 128:
        line["decode"] = decode_leg(tm, w, dev, peaks)
    if world == 1 and not args.no_varlen and w.tile == 128 and w.batch == 1 and w.seqlen >= 8 * w.tile:
        # chunked prefill: the last eighth of the context as a chunk against all of its keys (same tensors)
        Lq = (w.seqlen // 8) // w.tile * w.tile
        off = w.seqlen - Lq
        pc = tm.problem(1, w.heads, w.heads, Lq, w.head_dim, w.tile, w.tile, w.group)
        q8f, k8f, qsf, ksf = tm.tilemix_quantize_qk(p, qd, kd)
        words_f, _ = tm.tilemix_pack_routing_mask(p, rd, w.pin_diagonal)
        qc, q8c, qsc = qd[:, :, off:].contiguous(), q8f[:, :, off:].contiguous(), qsf[:, :, off // w.tile:].contiguous()
        oc = torch.empty_like(qc)
        for _ in range(3):
            tm.tilemix_attention_fwd_chunk(pc, w.seqlen, qc, kd, vd, q8c, k8f, qsc, ksf, words_f, out=oc, workspace=work)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        for _ in range(5):
            tm.tilemix_attention_fwd_chunk(pc, w.seqlen, qc, kd, vd, q8c, k8f, qsc, ksf, words_f, out=oc, workspace=work)
        c1.record(stream)
        torch.cuda.synchronize()
        ms = c0.elapsed_time(c1) / 5
        fl = 4.0 * w.heads * w.head_dim * (float(Lq) * off + float(Lq) ** 2 / 2.0)
        line["chunk"] = {"chunk_len": Lq, "context_len": w.seqlen, "attention_ms": ms,
                         "tflops": fl / (ms * 1e-3) / 1e12, "unit": "TFLOP/s"}
        # the same chunk against an INT8 value cache (conversion kernel + fused kernel with delta_V folded into P)
        _, v8f, _, vsf = tm.tilemix_quantize_qk(p, kd, vd)
        work8 = torch.empty(tm.tilemix_chunk_v8_workspace_size(pc, w.seqlen), dtype=torch.uint8, device=dev)
        for _ in range(3):
            tm.tilemix_attention_fwd_chunk_v8(pc, w.seqlen, qc, kd, v8f, vsf, q8c, k8f, qsc, ksf, words_f, out=oc, workspace=work8)
        c0.record(stream)
        for _ in range(5):
            tm.tilemix_attention_fwd_chunk_v8(pc, w.seqlen, qc, kd, v8f, vsf, q8c, k8f, qsc, ksf, words_f, out=oc, workspace=work8)
        c1.record(stream)
        torch.cuda.synchronize()
        ms8 = c0.elapsed_time(c1) / 5
        line["chunk"]["int8_value_cache_ms"] = ms8
        line["chunk"]["int8_value_cache_tflops"] = fl / (ms8 * 1e-3) / 1e12
        del v8f, vsf, work8
    if world == 1 and not args.no_varlen and w.tile == 128 and w.head_dim == 128:
        # on-the-fly operand mode: no INT8 copies of Q and K and no scales in device memory; the kernel makes
        # them in shared memory (same mask, same result bit for bit -- checked here on the full workload)
        po = tm.problem(w.batch, w.heads, w.heads, w.seqlen, w.head_dim, w.tile, w.tile, w.group,
                        mask_batch=w.mask_batch, flags=tm.QUANT_ON_THE_FLY)
        q8f, k8f, qsf, ksf = tm.tilemix_quantize_qk(p, qd, kd)
        words_f, _ = tm.tilemix_pack_routing_mask(p, rd, w.pin_diagonal)
        ref = tm.tilemix_attention_fwd(p, qd, kd, vd, q8f, k8f, qsf, ksf, words_f, workspace=work)["out"]
        oo = torch.empty_like(ref)
        for _ in range(2):
            tm.tilemix_attention_fwd(po, qd, kd, vd, None, None, None, None, words_f, out=oo, workspace=work)
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        o0.record(stream)
        for _ in range(3):
            tm.tilemix_attention_fwd(po, qd, kd, vd, None, None, None, None, words_f, out=oo, workspace=work)
        o1.record(stream)
        torch.cuda.synchronize()
        ms = o0.elapsed_time(o1) / 3
        line["on_the_fly"] = {"attention_ms": ms, "tflops": F / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                              "equals_quantize_once": bool(torch.equal(oo.view(torch.int16), ref.view(torch.int16))),
                              "int8_scratch_bytes_saved": int(q8f.numel() + k8f.numel() + 4 * (qsf.numel() + ksf.numel()))}
        del q8f, k8f, ref, oo
    if world == 1 and not args.no_cpu_baseline:
        dt, pairs, n_rows, threads = oracle_sample(w.scaled(heads=1, batch=1), q, k, v, route, args.cpu_pairs)
        line["cpu_baseline"] = {"value": 4.0 * w.head_dim * pairs / dt / 1e12, "unit": "TFLOP/s", "cores": threads,
                                "kind": "oracle", "seconds": dt,
                                "sample": f"{n_rows} rows of head 0 ({pairs} query-key pairs), incl. quantise+pack of that head"}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
