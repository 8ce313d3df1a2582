#!/usr/bin/env python
"""Benchmark of the template-recovery hot path: observed-entry gradient updates per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl reference]

A step is one full-batch gradient step (both gradient passes, fix-ups, clip + update with the shadow
refresh of bf16 templates) over the whole synthetic template, inputs resident in HBM: K epochs of one
tsid_fit call, or K tsid_grad_step calls where L2 is flushed between steps.  Every timed region is
repeated REPS times (best and median reported; the headline is the median).  One JSON line is printed
by rank 0: the headline workload (the 1e9-entry template on the path TSID_PATH_AUTO picks), and under
"secondary" the same measurement of the other configurations (the dense tensor-core variant on C4
among them).  With N > 1 (torchrun) every rank runs an independent replica of the same template (the
path is single-GPU; there is no data-path collective); a "sharded" sub-record times the row-sharded
form as well.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "observed-entry gradient updates/sec"
UNIT = "updates/s"
L2_BYTES = 126 * 1024 * 1024
REPS = 5
SEG_LEN = 512        # kSegLen of the library build the traffic figures were captured on
N_SMS = 148

# What the paper itself reports (another machine, whole-run seconds; context, never the target).
PAPER_CONTEXT = {
    "hardware": "2x Intel Xeon Gold 6426Y, 512 GB RAM, 4x NVIDIA A100 40 GB, CUDA 12.4, PyTorch AMP fp16/fp32 (Sec. 6.1, Test Platform)",
    "stage1_time_s": "2.0-2.2 s for template recovery on 10K..100K synthetic matrices; SVD in its place 3.4-8.6 s; 4.09x faster (Sec. 6.5)",
    "tensor_core_vs_cuda_core_s": {"16Kx16K": [30.7, 22.18], "32Kx32K": [62.16, 47.88], "64Kx64K": [158.21, 136.25],
                                   "80Kx80K": [283.4, 216.7], "what": "whole run, CUDA cores -> Tensor Cores (Sec. 6.4)"},
    "conflict_free_stage1_s": "8.30 -> 4.71 s end to end on 1Kx3K, up to 43 % (Sec. 6.3 ablation)",
    "memory_gb": {"1Kx3K": 0.30, "3Kx3K": 0.47, "3Kx10K": 0.79, "Last.fm": 0.85, "MovieLens-25M": 27, "MovieLens-33M": 38,
                  "Netflix": 22, "Yahoo": 23, "what": "peak GPU memory, both stages (Table 6)"},
    "headline": "up to 11,647x faster than CSNN, up to 8.5x lower peak memory, up to 99.7 % lower NMAE (abstract; end to end)",
    "per_step_throughput": "not reported by the paper (no updates/s, GB/s or kernel time for Stage I)",
}


def load_traffic():
    """ncu figures per launch of the dominant kernels (profiles/traffic.json, written beside the summaries)."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f)
    return {}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops_sustained"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1400.0, 1590.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(x, dist, device):
    """The slowest rank's time (replicas run independently; the job is as slow as its slowest rank)."""
    if dist is None:
        return float(x)
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(world, units_per_rank_step, steps, seconds):
    """Whole-job throughput: every rank processed units_per_rank_step * steps units in `seconds`."""
    return world * units_per_rank_step * steps / seconds


def run_reference(args, W):
    """The oracle, as it stands, on the host cores: each step is one oracle step over a bounded
    sample (a prefix of the row-sorted COO) of the workload."""
    import numpy as np
    import oracle
    w = W.CONFIGS[args.workload]
    sample_nnz = min(w.nnz, max(20_000, int(4.0e8 / w.k)))
    frac = sample_nnz / w.nnz
    m = max(8, int(math.ceil(w.m * min(1.0, frac * 4))))
    n = max(8, int(math.ceil(w.n * min(1.0, frac * 4))))
    sw = W.scaled(w, w.name + "-cpu-sample", m, n, min(sample_nnz, m * n // 2))
    tpl = W.make_template(sw, "cpu")
    r, c, v = tpl.rows.numpy(), tpl.cols.numpy(), tpl.vals.numpy()
    P, Q = tpl.P0.numpy(), tpl.Q0.numpy()
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        st = oracle.grad_step(sw.m, sw.n, sw.k, r, c, v, P, Q, sw.eta, sw.lam, sw.xi, sw.clip, sw.norm_p, sw.norm_q)
        dt = time.perf_counter() - t0
        P, Q = st.P, st.Q
        if it >= args.warmup:
            times.append(dt)
    total = sum(times)
    val = tpl.nnz * len(times) / total
    sample = "%dx%d k=%d nnz=%d template with the recipe of %s (oracle grad_step, double, single thread)" % (
        sw.m, sw.n, sw.k, tpl.nnz, args.workload)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def _oracle_slice(a):
    """One single-threaded oracle step over one row slice (runs in a child process)."""
    import oracle
    m_used, n, k, r, c, v, P, Q, eta, lam, xi, clip, norm_p, norm_q = a
    t0 = time.perf_counter()
    oracle.grad_step(m_used, n, k, r, c, v, P, Q, eta, lam, xi, clip, norm_p, norm_q)
    return time.perf_counter() - t0


def cpu_baseline(w, tpl_dev, P0, Q0, budget_s=20.0):
    """Times the oracle, as it stands, on a prefix of the template's (row-sorted) COO entries with the full
    factor matrices: once on one core, and once as N single-threaded oracle processes on disjoint row slices
    of such a prefix (N = the host's cores; the oracle itself has no threads).  Sized from a short calibration
    run so that each leg takes about budget_s seconds."""
    import multiprocessing as mp
    import numpy as np
    import oracle
    nnz = tpl_dev.nnz
    P, Q = P0.cpu().numpy(), Q0.cpu().numpy()

    def prefix(count):
        r = tpl_dev.rows[:count].cpu().numpy(); c = tpl_dev.cols[:count].cpu().numpy()
        v = tpl_dev.vals[:count].cpu().numpy()
        return r, c, v, (int(r.max()) + 1 if count else 1)     # the prefix touches rows [0, m_used)

    def run(count):
        r, c, v, m_used = prefix(count)
        t0 = time.perf_counter()
        oracle.grad_step(m_used, w.n, w.k, r, c, v, P[:m_used], Q, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
        return time.perf_counter() - t0, m_used

    count = min(nnz, 1_000_000)
    t, m_used = run(count)
    if t < 0.5 * budget_s and count < nnz:   # the first run also pays fixed costs: rescale once
        count = int(min(nnz, count * budget_s / max(t, 1e-3)))
        t, m_used = run(count)
    out = {"value": count / t, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": "first %d of %d row-sorted entries (rows 0..%d, all %d columns), one oracle grad_step, "
                     "%.1f s" % (count, nnz, m_used - 1, w.n, t)}
    ncores = os.cpu_count() or 1
    if ncores > 1:
        total = int(min(nnz, count * ncores))
        r, c, v, m_all = prefix(total)
        cuts = [int(np.searchsorted(r, m_all * i // ncores)) for i in range(ncores + 1)]
        cuts[-1] = total
        jobs = []
        for i in range(ncores):
            a, b = cuts[i], cuts[i + 1]
            if b <= a:
                continue
            r0 = int(r[a]); m_i = int(r[b - 1]) - r0 + 1
            jobs.append((m_i, w.n, w.k, r[a:b] - r0, c[a:b], v[a:b], P[r0:r0 + m_i], Q, w.eta, w.lam, w.xi, w.clip,
                         w.norm_p, w.norm_q))
        try:
            with mp.get_context("fork").Pool(len(jobs)) as pool:
                t0 = time.perf_counter()
                pool.map(_oracle_slice, jobs, chunksize=1)
                wall = time.perf_counter() - t0
            out["all_cores"] = {"value": total / wall, "unit": UNIT, "cores": len(jobs), "kind": "oracle",
                                "sample": "first %d entries cut into %d row slices, one single-threaded oracle process per "
                                          "slice, all at once, %.1f s wall" % (total, len(jobs), wall)}
        except Exception as ex:   # a host that cannot fork: the single-core figure stands alone
            out["all_cores"] = {"unavailable": repr(ex)}
    return out


def measure_sampling(args, w, tpl, B, dev):
    """Times tsid_sample_template (alpha = 0.5) on the workload's COO triples taken as the full matrix."""
    import ctypes as C
    nnz = tpl.nnz
    alpha, seed = 0.5, 12345
    need = C.c_size_t(0)
    B.lib().tsid_sample_workspace_bytes(w.n, nnz, C.byref(need))
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    base = (ws.data_ptr() + 255) & ~255
    colmap = torch.empty(w.n, dtype=torch.int32, device=dev)
    ro, co = torch.empty(nnz, dtype=torch.int32, device=dev), torch.empty(nnz, dtype=torch.int32, device=dev)
    vo = torch.empty(nnz, dtype=torch.float32, device=dev)
    d, kept = C.c_int32(0), C.c_int64(0)
    stream = torch.cuda.current_stream(dev)

    def call():
        st = B.lib().tsid_sample_template(w.m, w.n, nnz, alpha, seed, tpl.rows.data_ptr(), tpl.cols.data_ptr(),
                                          tpl.vals.data_ptr(), stream.cuda_stream, base, need.value, colmap.data_ptr(),
                                          ro.data_ptr(), co.data_ptr(), vo.data_ptr(), C.byref(d), C.byref(kept))
        assert st == B.TSID_OK, st
    for _ in range(args.warmup):
        call()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        call()
    b.record(stream)
    torch.cuda.synchronize(dev)
    ms = a.elapsed_time(b) / args.steps
    peak = load_peaks()[0]
    # per entry: the column index once for the per-block counts (4) and the triple once for the selection (12);
    # per kept entry: the triple written (12).  (The chosen columns sit in shared memory as a bitmap.)
    alg = nnz * 16 + kept.value * 12
    print(json.dumps({"metric": "matrix entries sampled/sec", "value": nnz / (ms * 1e-3), "unit": "entries/s",
                      "ms_per_call": ms, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "config": {"workload": w.name, "alpha": alpha, "d": d.value, "kept": kept.value},
                      "roofline": {"bound": "hbm", "achieved": alg / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": alg / (ms * 1e-3) / 1e9 / peak, "alg_bytes": alg}}))


def measure_layout(args, w, tpl, B, dev):
    """Times the layout pass (tsid_template_create on the sparse path: COO -> CSR, CSC, perm, pointers,
    segments) of the workload's entries in the order `--order` gives them, workspace already allocated."""
    import ctypes as C
    nnz = tpl.nnz
    prec = B.TSID_BF16_SHADOW if w.precision == "bf16" else B.TSID_F32
    cfg = B.make_config(w.m, w.n, w.k, nnz, prec, B.TSID_PATH_SPARSE, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q, 0)
    need = C.c_size_t(0)
    assert B.lib().tsid_workspace_bytes(C.byref(cfg), C.byref(need)) == B.TSID_OK
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=dev)
    cfg.workspace = (ws.data_ptr() + 255) & ~255
    cfg.workspace_bytes = need.value
    stream = torch.cuda.current_stream(dev)
    cfg.stream = stream.cuda_stream
    times = []
    for it in range(args.warmup + args.steps):
        h = C.c_void_p()
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        st = B.lib().tsid_template_create(C.byref(cfg), tpl.rows.data_ptr(), tpl.cols.data_ptr(), tpl.vals.data_ptr(),
                                          C.byref(h))
        torch.cuda.synchronize(dev)
        dt = time.perf_counter() - t0
        assert st == B.TSID_OK, st
        B.lib().tsid_destroy(h)
        if it >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    peak = load_peaks()[0]
    # compulsory: the COO triples in (12 B), col_idx + val_csr out (8 B), row_idx + val_csc + perm out (12 B) per
    # entry.  The radix passes of the implemented algorithm move more: per entry and pass 4 B (histogram) + the
    # key and its payload words in and out; the third sort starts from the identity, so its first pass reads 12 B
    # and writes 16 B.  Input check 8 B, the two pointer builds 8 B.
    compulsory = nnz * 32 + (w.m + w.n + 2) * 8
    pc = max(1, (max(w.n - 1, 1).bit_length() + 7) // 8)
    pr = max(1, (max(w.m - 1, 1).bit_length() + 7) // 8)
    third = pc * 4 + 28 + (pc - 1) * 32
    per_entry = 16 + third + ((pc + pr) * 28 if args.order == "shuffled" else 16)
    alg = nnz * per_entry
    print(json.dumps({"metric": "entries laid out/sec", "value": nnz / t, "unit": "entries/s", "ms_per_call": t * 1e3,
                      "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "config": {"workload": w.name, "order": args.order, "m": w.m, "n": w.n, "nnz": nnz,
                                 "workspace_gb": need.value / 1e9},
                      "roofline": {"bound": "hbm", "achieved": alg / t / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": alg / t / 1e9 / peak, "alg_bytes": alg, "alg_bytes_per_entry": per_entry,
                                   "compulsory_bytes": compulsory, "compulsory_frac": compulsory / t / 1e9 / peak}}))


def measure_extend(args, w, tpl, B, dev):
    """Times tsid_extend: the workload's matrix (all n columns, host-resident, column-compressed) is extended
    from a template of d = n/4 columns (random-init factors of the workload's rank), `iters` Adam steps per
    chunk, 16 chunks.  The timed region is the whole call: H2D of the entries, compute, D2H of C."""
    d = max(8, w.n // 4)
    iters = 10
    chunk = max(1, (w.n + 15) // 16)
    order = torch.argsort(tpl.cols.long() * w.m + tpl.rows.long())
    rows = tpl.rows[order].cpu().pin_memory()
    vals = tpl.vals[order].cpu().pin_memory()
    counts = torch.bincount(tpl.cols.long(), minlength=w.n)
    col_ptr = torch.zeros(w.n + 1, dtype=torch.int64)
    col_ptr[1:] = torch.cumsum(counts.cpu(), 0)
    col_ptr = col_ptr.pin_memory()
    P = tpl.P0
    Q = tpl.Q0[:d].contiguous()
    Ch = torch.zeros(w.n, d).pin_memory()
    times = []
    for it in range(args.warmup + args.steps):
        Ch.zero_()
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        B.tsid_extend(P, Q, col_ptr, rows, vals, Ch, chunk, iters, 0.02, 0.05, cold_start=True, tensor_cores=args.extend_tc)
        torch.cuda.synchronize(dev)
        if it >= args.warmup:
            times.append(time.perf_counter() - t0)
    t = sum(times) / len(times)
    nnz = tpl.nnz
    # per Adam step: C, m, v read + written (24 B per coefficient) + C read by the first GEMM (4 B)
    # + the entry pass (8 + 4k B per entry, fp32 gathers); per call: entries in (8 B) and C in/out (8 B)
    alg_dev = iters * (w.n * d * 28 + nnz * (8 + 4 * w.k))
    flops = iters * (4.0 * w.n * d * w.k + 4.0 * nnz * w.k)
    peak = load_peaks()[0]
    print(json.dumps({"metric": "Stage II observed-entry Adam updates/sec", "value": nnz * iters / t, "unit": "updates/s",
                      "s_per_call": t, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
                      "config": {"workload": w.name, "m": w.m, "n_cols": w.n, "d": d, "k": w.k, "nnz": nnz,
                                 "iters": iters, "chunk_cols": chunk,
                                 "dtype": "bf16 operands / fp32 accumulation for the gradient product, fp32 elsewhere"
                                          if args.extend_tc else "f32"},
                      "h2d_bytes_per_call": nnz * 8 + (w.n + 1) * 8, "d2h_bytes_per_call": w.n * d * 4,
                      "roofline": {"bound": "hbm", "achieved": alg_dev / t / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": alg_dev / t / 1e9 / peak, "alg_bytes": alg_dev,
                                   "fp32_tflops": flops / t / 1e12}}))


def run_row_sharded(args, w, tpl, B, dev, dist, rank, world):
    """One template sharded by rows over the ranks: per step tsid_grad, one all-reduce (sum) of G_Q over
    NCCL, tsid_apply.  Total work is fixed as the rank count grows."""
    from paper_2608_00977_b200 import sharded as S
    r0, r1 = S.row_block(w.m, rank, world)
    rows, cols, vals = S.shard_coo(tpl.rows, tpl.cols, tpl.vals, r0, r1)
    prec = B.TSID_BF16_SHADOW if w.precision == "bf16" else B.TSID_F32
    sh = S.RowShard(r1 - r0, w.n, w.k, rows, cols, vals, precision=prec, eta=w.eta, lam=w.lam, xi=w.xi, clip=w.clip,
                    norm_p=w.norm_p, norm_q=w.norm_q, dist=dist)
    P, Q = tpl.P0[r0:r1].clone().contiguous(), tpl.Q0.clone()
    stream = torch.cuda.current_stream(dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)
    step = lambda: sh.step(P, Q)
    if args.exchange == "peer":
        # the exchange folded into the update kernel: G_Q parts and Q replicas mapped into every rank
        if world > 1:
            gq, gq_ptrs, gq_bar = S.symmetric_buffers(w.n * w.k, dev, dist)
            qs, q_ptrs, q_bar = S.symmetric_buffers(w.n * w.k, dev, dist)
            qs.copy_(Q.view(-1))
            Q = qs.view(w.n, w.k)
            sh.GQ = gq
        else:
            gq_ptrs, q_ptrs, gq_bar, q_bar = [sh.GQ.data_ptr()], [Q.data_ptr()], (lambda: None), (lambda: None)

        def step():
            sh.grad(P, Q)
            gq_bar()                                   # all parts complete
            sh.apply_sliced(P, q_ptrs, gq_ptrs, rank)
            q_bar()                                    # all slices stored
    for _ in range(args.warmup):
        step()
    sh.T.tsid_check()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    sampler.start()
    time.sleep(0.3)
    barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        step()
    b.record(stream)
    barrier()
    ms = max_over_ranks(a.elapsed_time(b), dist, dev)
    clocks = sampler.stop()
    sh.T.tsid_check()
    sse = sh.sse(P, Q)
    rec = None
    if rank == 0:
        _, launches = sh.T.tsid_get_info()
        rec = ({"metric": METRIC, "value": tpl.nnz * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                          "dtype": "bf16" if w.precision == "bf16" else "f32", "data": "synthetic",
                          "config": {"workload": w.name, "m": w.m, "n": w.n, "k": w.k, "nnz": tpl.nnz,
                                     "parallelism": ("rows/%d, exchange of G_Q (%d bytes) folded into the update kernel over peer memory"
                                                     if args.exchange == "peer" else
                                                     "rows/%d, all-reduce(sum) of G_Q (%d bytes) per step") % (world, w.n * w.k * 4),
                                     "l2": "inputs larger than L2, steps timed back to back"},
                          "clocks": clocks, "e2e": None, "gpu_launches": launches * args.steps, "roofline": None,
                          "cpu_baseline": None, "rmse_after": (sse / tpl.nnz) ** 0.5})
    sh.destroy()
    return rec


def alg_bytes_pass(w, entries, rows, nseg, value_bytes=4):
    """Algorithmic bytes of one gather-reduce pass launch over `entries` entries of `rows` staged rows."""
    b = 2 if w.precision == "bf16" else 4
    return entries * (4 + value_bytes + w.k * b) + rows * w.k * (b + 4) + nseg * 16


class StepBench:
    """One workload on one kernel path: template, warm-up, REPS timed regions of K steps, per-kernel times."""

    def __init__(self, args, W, B, wname, path_name, dev, dist, local, values="f32"):
        self.args, self.W, self.B, self.dev, self.dist, self.local = args, W, B, dev, dist, local
        self.wname, self.path_name, self.values = wname, path_name, values
        self.w = W.CONFIGS[wname]
        self.tpl = None
        self.T = None

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize(self.dev)

    def create(self, tpl=None):
        B, w = self.B, self.w
        t0 = time.perf_counter()
        self.tpl = tpl if tpl is not None else self.W.make_template(w, self.dev, order="sorted")
        torch.cuda.synchronize(self.dev)
        t1 = time.perf_counter()
        want = {"auto": B.TSID_PATH_AUTO, "sparse": B.TSID_PATH_SPARSE, "dense": B.TSID_PATH_DENSE_TC,
                "hybrid": B.TSID_PATH_HYBRID}[self.path_name]
        self.want_path = want
        vflags = B.TSID_VALUES_U8 if self.values == "u8" else 0
        self.T = B.template_from_workload(self.tpl, path=want, flags=vflags)
        torch.cuda.synchronize(self.dev)
        self.gen_s, self.create_s = t1 - t0, time.perf_counter() - t1
        self.path, self.launches = self.T.tsid_get_info()
        self.P, self.Q = self.tpl.P0.clone(), self.tpl.Q0.clone()
        return self

    def measure(self, steps, warmup, long_seconds=0.0):
        """Returns the record of this workload (timings in ms per step)."""
        B, w, T, P, Q, dev = self.B, self.w, self.T, self.P, self.Q, self.dev
        nnz = self.tpl.nnz
        stream = torch.cuda.current_stream(dev)
        resident = nnz * 16 + (w.m + w.n) * w.k * 4
        flush = resident < 4 * L2_BYTES
        scrub = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if flush else None
        for _ in range(warmup):
            T.tsid_grad_step(P, Q)
        T.tsid_check()
        sampler = ClockSampler(self.local)
        sampler.start()
        time.sleep(0.3)

        def timed(profiled=False, nsteps=steps):
            self.barrier()
            if flush:
                evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(nsteps)]
                for a, b in evs:
                    scrub.fill_(1)
                    a.record(stream)
                    T.tsid_grad_step(P, Q)
                    b.record(stream)
                self.barrier()
                return sum(a.elapsed_time(b) for a, b in evs)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            # K steps of one tsid_fit: replayed from the library's captured graph, or (profiled) the same kernels
            # launched one by one with the library's events between them
            T.tsid_fit(P, Q, nsteps)
            b.record(stream)
            self.barrier()
            return a.elapsed_time(b)

        # The headline loop carries no events between its kernels; the same K steps are then repeated with the
        # library's per-kernel events on the launching stream, and the roofline of the dominant kernel uses those.
        if not flush:
            T.tsid_fit(P, Q, steps)          # untimed: the call that captures the graph of K steps
            T.tsid_check()
        reps = [max_over_ranks(timed(), self.dist, dev) / steps for _ in range(REPS)]
        clocks = sampler.stop()
        long_run = None
        if long_seconds > 0 and not flush:
            # a region long enough for the power cap to set in (the regime of the sustained peak)
            nlong = max(steps, int(math.ceil(long_seconds * 1e3 / min(reps) / 8.0)) * 8)
            s2 = ClockSampler(self.local)
            s2.start()
            T.tsid_fit(P, Q, 8)
            ms_long = max_over_ranks(timed(nsteps=nlong), self.dist, dev) / nlong
            long_run = {"steps": nlong, "ms_per_step": ms_long, "clocks": s2.stop()}
        T.tsid_set_profiling(True)
        ms_prof = timed(profiled=True) / steps
        nrec, row_ms, col_ms, upd_ms, tile_ms = T.tsid_get_step_times()
        T.tsid_set_profiling(False)
        T.tsid_check()
        nrec = max(1, nrec)
        self.flush = flush
        shadow = 1 if w.precision == "bf16" else 0
        return {"reps_ms_per_step": reps, "best": min(reps), "median": statistics.median(reps), "clocks": clocks,
                "long_run": long_run, "ms_per_step_with_events": ms_prof,
                "kernel_ms": {"row_pass": row_ms / nrec, "col_pass": col_ms / nrec, "update": upd_ms / nrec,
                              "tile_passes": tile_ms / nrec},
                "gpu_launches_per_rep": self.launches * steps if flush else T.tsid_get_fit_launches(steps),
                "resident_bytes": resident}

    def roofline(self, rec, traffic):
        """Roofline record of the dominant kernel of this path, from the live launch durations."""
        B, w, T = self.B, self.w, self.T
        nnz = self.tpl.nnz
        peak, tf_sustained, tf_burst, peak_kind = load_peaks()
        km = rec["kernel_ms"]
        ms_step = rec["median"]
        mhz = rec["clocks"].get("sm_mhz") or 1965.0
        tkey = "%s-%s" % (self.wname, "dense" if self.path == B.TSID_PATH_DENSE_TC else
                          ("hybrid" if self.path == B.TSID_PATH_HYBRID else "sparse"))
        tr = traffic.get(tkey, {})
        if self.path == B.TSID_PATH_DENSE_TC:
            # dense variant: the dominant kernel is the tcgen05 pass (two launches per step); algorithmic flops
            # are the three GEMMs of the method, 6 m n k per step, i.e. 3 m n k per launch (four are executed)
            pass_ms = (km["row_pass"] + km["col_pass"]) / 2
            fl = 3.0 * w.m * w.n * w.k
            tfl_short = fl / (pass_ms * 1e-3) / 1e12
            out = {"bound": "tensor", "kernel": "dense_pass_kernel (tcgen05; pass over R and pass over R^T)",
                   "unit": "TFLOP/s", "alg_flops_per_launch": fl, "executed_flops_per_launch": 4.0 * w.m * w.n * w.k,
                   "avg_launch_ms": pass_ms, "traffic": tr.get("dram_bytes_per_launch"),
                   "pass_R": {"ms": km["row_pass"]}, "pass_RT": {"ms": km["col_pass"]}, "update": {"ms": km["update"]},
                   "short_run": {"what": "launch durations of the %d-step runs (clock %s MHz: burst regime)" % (
                                     self.args.steps, rec["clocks"].get("sm_mhz")),
                                 "kernel_tflops": tfl_short, "kernel_frac_of_burst": tfl_short / tf_burst,
                                 "step_frac_of_burst": 6.0 * w.m * w.n * w.k / (ms_step * 1e-3) / 1e12 / tf_burst},
                   "peak_burst": tf_burst, "peak_sustained": tf_sustained, "frac_of_nominal_2250": tfl_short / 2250.0}
            lr = rec.get("long_run")
            if lr:
                # like for like: a seconds-long region against the sustained peak; the pass kernels' share of a step
                # is taken from the per-kernel events of the short run
                share = 2 * pass_ms / max(1e-9, rec["ms_per_step_with_events"])
                step_tfl = 6.0 * w.m * w.n * w.k / (lr["ms_per_step"] * 1e-3) / 1e12
                out["long_run"] = {"steps": lr["steps"], "ms_per_step": lr["ms_per_step"], "clocks": lr["clocks"],
                                   "step_tflops": step_tfl, "step_frac_of_sustained": step_tfl / tf_sustained,
                                   "kernel_frac_of_sustained": step_tfl / max(share, 1e-9) / tf_sustained if share < 1 else None}
                out.update({"achieved": step_tfl, "peak": tf_sustained, "frac": step_tfl / tf_sustained,
                            "peak_source": "of %s (sustained bf16, against a %d-step region under the power cap)" % (
                                peak_kind, lr["steps"]),
                            "frac_is": "whole step (both passes + update), algorithmic flops, long run / sustained peak"})
            else:
                out.update({"achieved": tfl_short, "peak": tf_burst, "frac": tfl_short / tf_burst,
                            "peak_source": "of %s (burst bf16: short run at full clock)" % peak_kind})
            return out
        # gather-reduce passes (all entries on the sparse path, the tail entries on the hybrid path)
        tiles, min_tile, tail = T.tsid_get_hybrid_info()
        ent = tail if self.path == B.TSID_PATH_HYBRID else nnz
        vb = 1 if self.values == "u8" else 4
        b_row = alg_bytes_pass(w, ent, w.m, w.m + ent // SEG_LEN, vb)
        b_col = alg_bytes_pass(w, ent, w.n, w.n + ent // SEG_LEN, vb)
        b = 2 if w.precision == "bf16" else 4
        b_upd = (w.m + w.n) * w.k * (4 + 4 + 4 + (b if b == 2 else 0)) + (w.m + w.n) * 4
        pass_ms = (km["row_pass"] + km["col_pass"]) / 2
        bytes_per_launch = (b_row + b_col) / 2
        achieved = bytes_per_launch / (pass_ms * 1e-3) / 1e9 if pass_ms > 0 else 0.0
        step_alg = nnz * (8 + vb * 2 + 2 * w.k * b) + (w.m + w.n) * w.k * 20 + (w.m + w.n + 2) * 8
        step_min = nnz * 16 + (w.m + w.n) * w.k * 20
        out = {"bound": "hbm",
               "kernel": "pass_staged_kernel (gather-reduce: CSR row pass + CSC column pass, 2 launches per step%s)" % (
                   "; the %d entries outside the dense tiles" % ent if self.path == B.TSID_PATH_HYBRID else ""),
               "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "alg_frac": achieved / peak,
               "peak_source": "of %s" % peak_kind,
               "note": "frac = alg_frac charges every gathered factor row at HBM rate although L2 serves many of them, so it "
                       "can exceed 1; hbm_frac is what HBM itself carried (ncu DRAM bytes / launch time / peak)",
               "alg_bytes_per_launch": bytes_per_launch, "avg_launch_ms": pass_ms,
               "row_pass": {"ms": km["row_pass"], "alg_bytes": b_row},
               "col_pass": {"ms": km["col_pass"], "alg_bytes": b_col},
               "update": {"ms": km["update"], "alg_bytes": b_upd,
                          "gbs": b_upd / (km["update"] * 1e-3) / 1e9 if km["update"] else None},
               "step_alg_bytes": step_alg, "step_compulsory_bytes": step_min,
               "step_frac": step_alg / (ms_step * 1e-3) / 1e9 / peak,
               "frac_compulsory": step_min / (ms_step * 1e-3) / 1e9 / peak,
               "frac_of_nominal_8TBs": achieved / 8000.0}
        out["traffic"] = tr.get("dram_bytes_per_launch")
        if tr:
            out["traffic_from"] = tr.get("from")
            if tr.get("seg_len") not in (None, SEG_LEN):
                out["traffic_stale"] = "captured with segments of %s entries, this build uses %d" % (tr.get("seg_len"), SEG_LEN)
            if tr.get("dram_bytes_per_launch") and pass_ms > 0:
                out["dram_gbs"] = tr["dram_bytes_per_launch"] / (pass_ms * 1e-3) / 1e9
                out["hbm_frac"] = out["frac_dram"] = out["dram_gbs"] / peak
            if tr.get("warp_insts_per_entry") and pass_ms > 0:
                # share of the issue slots the pass uses: warp instructions / (SMs x 4 schedulers x clock x time)
                out["issue"] = {"warp_insts_per_entry": tr["warp_insts_per_entry"], "sm_mhz": mhz,
                                "frac": tr["warp_insts_per_entry"] * ent / (pass_ms * 1e-3) / (N_SMS * 4 * mhz * 1e6)}
        if self.path == B.TSID_PATH_HYBRID:
            fl_alg = 6.0 * 128 * 128 * w.k * tiles   # per step, both tile passes: S, E Y and E^T X of every stored tile
            out["tile_passes"] = {"tiles": tiles, "min_entries_per_tile": min_tile, "entries_in_tiles": nnz - tail,
                                  "ms": km["tile_passes"],
                                  "what": "tcgen05 tile pass over R tiles and over R^T tiles (their sums are added by the update kernel, which also keeps the rank-ordered shadow copies current)",
                                  "alg_tflops": fl_alg / (km["tile_passes"] * 1e-3) / 1e12 if km["tile_passes"] else None,
                                  "frac_of_burst_peak": fl_alg / (km["tile_passes"] * 1e-3) / 1e12 / tf_burst if km["tile_passes"] else None}
        return out

    def destroy(self):
        if self.T is not None:
            self.T.tsid_destroy()
            self.T = None
        self.P = self.Q = None
        torch.cuda.empty_cache()


def path_label(B, path):
    return {B.TSID_PATH_SPARSE: "sparse", B.TSID_PATH_DENSE_TC: "dense_tc", B.TSID_PATH_HYBRID: "hybrid"}.get(path, str(path))


def workload_config(B, sb, world):
    w, nnz = sb.w, sb.tpl.nnz
    return {"workload": w.name, "m": w.m, "n": w.n, "k": w.k, "nnz": nnz,
            "precision": "bf16 shadow factors, fp32 master and accumulation" if w.precision == "bf16" else "fp32",
            "path": path_label(B, sb.path), "path_requested": sb.path_name,
            "values": "one byte per rating" if sb.values == "u8" else "fp32",
            "step": "%s (eta=%g lambda=%g xi=%g clip=%d norm=%d/%d)" % (
                "K calls of tsid_grad_step" if sb.flush else "one tsid_fit of K epochs (graph replay)",
                w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q),
            "l2": "L2 flushed between timed steps (resident set %.0f MB)" % (sb.resident / 1e6) if sb.flush
                  else "inputs larger than L2 (resident set %.1f GB), steps timed back to back" % (sb.resident / 1e9),
            "repetitions": REPS, "replicas": world}


def secondary_record(args, W, B, wname, path_name, dev, local, traffic, tpl=None, long_seconds=0.0):
    """One more workload measured like the headline (no e2e, no CPU leg)."""
    sb = StepBench(args, W, B, wname, path_name, dev, None, local).create(tpl)
    rec = sb.measure(args.steps, args.warmup, long_seconds)
    sb.resident = rec["resident_bytes"]
    roof = sb.roofline(rec, traffic)
    nnz = sb.tpl.nnz
    out = {"config": workload_config(B, sb, 1), "ms_per_step": rec["median"], "best_ms_per_step": rec["best"],
           "reps_ms_per_step": rec["reps_ms_per_step"], "value": nnz / (rec["median"] * 1e-3), "unit": UNIT,
           "clocks": rec["clocks"], "roofline": roof, "layout_s": sb.create_s,
           "workspace_gb": sb.T.workspace.numel() / 1e9}
    sb.destroy()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=os.environ.get("TSID_BENCH_WORKLOAD", "C5"))
    ap.add_argument("--impl", default="tsid")
    ap.add_argument("--path", default="auto", choices=["auto", "sparse", "dense", "hybrid"],
                    help="kernel path of the measured template (auto: what TSID_PATH_AUTO resolves to; the dense tcgen05 "
                         "variant needs a qualifying workload, e.g. C4)")
    ap.add_argument("--measure", default="step", choices=["step", "sample", "extend", "layout"],
                    help="step: the gradient step (default); sample: tsid_sample_template on the workload's COO; "
                         "extend: Stage II (tsid_extend) of the workload's matrix on a template of a quarter of its columns; "
                         "layout: the layout pass (tsid_template_create) on the workload's COO in --order")
    ap.add_argument("--order", default="shuffled", choices=["sorted", "shuffled"],
                    help="entry order of the COO input for --measure layout")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "rows"],
                    help="N > 1: independent replicas of the template (default), or ONE template sharded by rows "
                         "with one all-reduce of G_Q per step")
    ap.add_argument("--extend-tc", action="store_true",
                    help="--measure extend: the gradient product on the tensor cores (TSID_EXTEND_TC, mixed precision)")
    ap.add_argument("--exchange", default="nccl", choices=["nccl", "peer"],
                    help="--shard rows: NCCL all-reduce of G_Q, or the exchange folded into the update kernel "
                         "(tsid_apply_sliced over symmetric memory)")
    ap.add_argument("--values", default="f32", choices=["f32", "u8"],
                    help="u8: stream the ratings as one byte each (TSID_VALUES_U8; needs integer values, e.g. C2, C3, C5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="only the headline workload (no C5-sparse / C4 / C3 / C2 records)")
    ap.add_argument("--e2e-epochs", type=int, default=0, help="epochs per host-buffer call (0: the workload's)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2608_00977_b200 import workloads as W
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, W)
        return

    import __graft_entry__ as G
    from paper_2608_00977_b200 import binding as B
    if rank == 0:
        G.build()
    dist = None
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    B.lib()

    w = W.CONFIGS[args.workload]
    if args.measure != "step" or args.shard == "rows":
        tpl = W.make_template(w, dev, order=args.order if args.measure == "layout" else "sorted")
        torch.cuda.synchronize(dev)
        if args.measure == "sample":
            measure_sampling(args, w, tpl, B, dev)
        elif args.measure == "extend":
            measure_extend(args, w, tpl, B, dev)
        elif args.measure == "layout":
            measure_layout(args, w, tpl, B, dev)
        else:
            rec = run_row_sharded(args, w, tpl, B, dev, dist, rank, world)
            if rank == 0:
                print(json.dumps(rec))
        return

    traffic = load_traffic()
    sb = StepBench(args, W, B, args.workload, args.path, dev, dist, local, args.values).create()
    tpl, nnz = sb.tpl, sb.tpl.nnz
    if rank == 0:
        sys.stderr.write("[bench] %s: generated %d entries in %.1f s, create (layout pass) %.2f s, workspace %.2f GB, path %s\n" % (
            w.name, nnz, sb.gen_s, sb.create_s, sb.T.workspace.numel() / 1e9, path_label(B, sb.path)))
    dense_headline = sb.path == B.TSID_PATH_DENSE_TC
    rec = sb.measure(args.steps, args.warmup, long_seconds=2.5 if dense_headline else 0.0)
    sb.resident = rec["resident_bytes"]
    ms_step = rec["median"]
    value = aggregate_value(world, nnz, 1, ms_step * 1e-3)
    roofline = sb.roofline(rec, traffic)
    roofline.update({"launch_times_from": "the same %d steps repeated with the library's per-kernel CUDA events" % args.steps,
                     "ms_per_step_with_events": rec["ms_per_step_with_events"]})
    config = workload_config(B, sb, world)
    prec = B.TSID_BF16_SHADOW if w.precision == "bf16" else B.TSID_F32
    want_path = sb.want_path
    ws_gb = sb.T.workspace.numel() / 1e9
    create_s = sb.create_s
    sb.destroy()

    # ---- end to end: host buffers through tsid_fit_host ----------------------------------------------
    e2e = None
    if not args.no_e2e:
        epochs = args.e2e_epochs or w.epochs
        cfg = B.make_config(w.m, w.n, w.k, nnz, prec, want_path, w.eta, w.lam, w.xi, w.clip, w.norm_p, w.norm_q)
        hb = [x.cpu().pin_memory() for x in (tpl.rows, tpl.cols, tpl.vals)]
        hP0, hQ0 = tpl.P0.cpu(), tpl.Q0.cpu()
        hP, hQ = hP0.clone().pin_memory(), hQ0.clone().pin_memory()
        ws = torch.empty(B.tsid_workspace_bytes_host(cfg) + 256, dtype=torch.uint8, device=dev)
        reps = 2
        sb.barrier()
        t_e2e = 0.0
        for rep in range(reps + 1):
            hP.copy_(hP0); hQ.copy_(hQ0)
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            B.tsid_fit_host(cfg, hb[0], hb[1], hb[2], hP, hQ, epochs, ws)
            torch.cuda.synchronize(dev)
            if rep > 0:   # the first call warms the pinned pages and the allocator
                t_e2e += time.perf_counter() - t0
        t_e2e = max_over_ranks(t_e2e, dist, dev)
        h2d = nnz * 12 + (w.m + w.n) * w.k * 4
        d2h = (w.m + w.n) * w.k * 4
        e2e = {"value": world * nnz * epochs * reps / t_e2e, "unit": UNIT,
               "h2d_bytes_per_step": h2d / epochs, "d2h_bytes_per_step": d2h / epochs,
               "epochs_per_call": epochs, "h2d_bytes_per_call": h2d, "d2h_bytes_per_call": d2h,
               "s_per_call": t_e2e / reps, "input_order": "COO sorted by (row, col); a shuffled COO adds two sorts to the layout pass",
               "what": "tsid_fit_host: pinned host COO + factors -> device, layout pass (and tile build), epochs steps, "
                       "factors -> host; the paper runs 100 - 10,000 iterations per template, which would amortise the "
                       "copies and the layout further"}
        del ws, hb, hP, hQ
        torch.cuda.empty_cache()

    # ---- the row-sharded form of the same template, when there is more than one rank ------------------
    sharded = None
    if world > 1:
        try:
            sharded = run_row_sharded(args, w, tpl, B, dev, dist, rank, world)
        except Exception as ex:   # the replica line above stands on its own
            sharded = {"unavailable": repr(ex)}

    # ---- the other configurations, measured the same way (rank 0 of a single-GPU run) -----------------
    secondary = None
    if rank == 0 and world == 1 and not args.no_secondary:
        secondary = {}
        try:
            if sb.path != B.TSID_PATH_SPARSE:
                secondary["%s-sparse" % args.workload] = secondary_record(args, W, B, args.workload, "sparse", dev, local,
                                                                          traffic, tpl=tpl)
        except Exception as ex:
            secondary["%s-sparse" % args.workload] = {"unavailable": repr(ex)}
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w, tpl, tpl.P0, tpl.Q0)
    del tpl
    sb.tpl = None
    torch.cuda.empty_cache()
    if secondary is not None:
        for key, wname, pname, long_s in (("C4-dense", "C4", "dense", 2.5), ("C3", "C3", "auto", 0.0), ("C2", "C2", "auto", 0.0)):
            if wname == args.workload:
                continue
            try:
                secondary[key] = secondary_record(args, W, B, wname, pname, dev, local, traffic, long_seconds=long_s)
            except Exception as ex:
                secondary[key] = {"unavailable": repr(ex)}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.precision == "bf16" else "f32",
                "data": "synthetic", "config": config,
                "timing": {"repetitions": REPS, "reps_ms_per_step": rec["reps_ms_per_step"], "best_ms_per_step": rec["best"],
                           "median_ms_per_step": rec["median"], "headline": "median of the repetitions, each exactly K steps",
                           "create_s": create_s, "workspace_gb": ws_gb},
                "clocks": rec["clocks"], "e2e": e2e, "gpu_launches": rec["gpu_launches_per_rep"],
                "roofline": roofline, "cpu_baseline": cpu, "secondary": secondary, "sharded": sharded,
                "paper_context": PAPER_CONTEXT}
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
