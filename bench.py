#!/usr/bin/env python
"""Benchmark of the paged-KV serving iteration (KV append + GQA attention).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config 2|3|4|5]

A step is one pass of the whole hot path over one synthetic batch: KV append,
split-K decode attention, LSE merge and (for batches with prefill chunks)
prefill attention.  The headline workload (`value`) is the decode-heavy ragged
batch on the Llama-3-8B attention shape (64 sequences, contexts log-uniform in
128..8192).  Without --config the same run also times the mixed iteration
(both dispatch modes), the long-context decode and the workload-shift trace and
reports them under `configs`, so that the HBM-bound and the tensor-bound kernel
each have a measured roofline fraction in the one line.  Prints ONE JSON line
(rank 0).

Timing: CUDA events on the launching stream around K steps (repeated back to
back until the region lasts about a second, so that clock samples fall inside it)
after W warm-up steps, barrier + synchronize on both sides, max over ranks.  Every
step reads a different copy of the KV pool (rotation among copies whose
combined size is many times the L2), so KV reads are cold.  The plan (host
work list + one H2D copy) is built once per batch outside `value`'s timed
region -- a serving engine builds it once per iteration and reuses it for
every layer -- and is inside the `e2e` region, which goes through
ap_serving_iteration_host with pinned host buffers every step.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "serving_iteration_attention_kv_tokens_per_s"
UNIT = "KV-tokens/s"

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of a kernel on a bench
# workload (ncu captures summarised under profiles/), keyed by (kernel, config, hash of
# the kernel's source file the counters were taken from); a changed kernel reports null.
NCU_TRAFFIC = {
    # profiles/decode_splitk_config2.md: 536.5 MB read + 3.8 MB written per launch (algorithmic 535.0 MB)
    ("decode_splitk", 2, "e7670ad945da38e5"): 540.3e6,
    # profiles/prefill_tcgen05_config3.md: 149.4 MB read + 18.0 MB written per launch (K/V re-reads are served by the L2)
    ("prefill_tcgen05", 3, "080aa46481f9814f"): 167.4e6,
}


def kernel_source_hash(*source_files: str) -> str:
    """Hash of the files a kernel's device code lives in (its .cu, the .cuh with the body, the PTX wrappers)."""
    h = hashlib.sha256()
    for f in source_files + ("ptx.cuh",):
        with open(os.path.join(ROOT, "paper_2604_07144_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def make_batch(config: int, seed_offset: int = 0, with_pool: bool = True):
    from paper_2604_07144_b200 import workloads as W
    gen = {1: W.config1, 2: W.config2, 3: W.config3, 4: W.config4}[config]
    kw = {} if config == 1 else {"with_pool": with_pool}
    from paper_2604_07144_b200 import replicas
    return gen(seed=replicas.replica_seed(W.SEED_BASE + config, seed_offset), **kw)


def algorithmic_bytes(batch, info):
    """Bytes the method must move per step (one attention layer)."""
    hq, hkv, d = batch.num_q_heads, batch.num_kv_heads, batch.head_dim
    per_kv_token = 2 * hkv * d * 2
    per_row = 2 * hq * d * 2 + hq * 4                      # q read, out write, lse write
    dec = batch.q_lens == 1
    decode_kv = int(batch.ctx_lens[dec].astype(np.int64).sum())
    decode_bytes = decode_kv * per_kv_token + int(dec.sum()) * per_row + int(((batch.ctx_lens[dec] + 15) // 16).sum()) * 4
    append_bytes = 2 * info["n_new"] * 2 * hkv * d * 2     # read + write, K and V
    total = info["kv_tokens"] * per_kv_token + info["n_new"] * per_row + append_bytes
    pre = batch.q_lens > 1
    prefill_rows = int(batch.q_lens[pre].astype(np.int64).sum())
    prefill_kv = int(batch.ctx_lens[pre].astype(np.int64).sum())
    prefill_bytes = prefill_kv * per_kv_token + prefill_rows * per_row
    return {"per_kv_token": per_kv_token, "decode_kernel": decode_bytes, "prefill_kernel": prefill_bytes,
            "append_kernel": append_bytes, "total": total,
            "decode_flops": 4 * hq * d * decode_kv, "prefill_flops": 4 * hq * d * info["prefill_pairs"]}


def paper_model_us(flops: float, bytes_: float, peaks) -> float:
    """Operator time by the paper's own cost model (App. B, Eq. "roofline"):
    pi = min(F/A * B_g, F_g), T_op = F / pi, with the measured copy bandwidth and bf16 peak of this GPU."""
    if flops <= 0 or bytes_ <= 0:
        return 0.0
    pi = min(flops / bytes_ * peaks["hbm_gbs"] * 1e9, peaks["bf16_tflops"] * 1e12)
    return flops / pi * 1e6


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w": None}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                try:
                    pw.append(float(f[3]))
                except ValueError:
                    pass
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w=(statistics.median(pw) if pw else None))
        return out


def pick_sequences(active, cost, run_seconds, target_s):
    """Whole sequences of the batch, in batch order, whose estimated oracle time stays within
    target_s.  The rate comes from a probe on the median-cost sequence and is refined once from a
    real run if the probe (dominated by fixed overheads) underestimated it."""
    probe = sorted(active, key=lambda s: cost[s])[len(active) // 2]
    rate = cost[probe] / max(run_seconds([probe]), 1e-6)
    chosen = []
    for _ in range(3):
        chosen, est = [], 0.0
        for s in active:
            if chosen and est + cost[s] / rate > target_s:
                continue
            chosen.append(s)
            est += cost[s] / rate
        if len(chosen) == len(active):
            break
        new_rate = sum(cost[s] for s in chosen) / max(run_seconds(chosen), 1e-6)
        if new_rate < 1.5 * rate:
            break
        rate = new_rate
    return chosen


def cpu_oracle_baseline(batch, target_s: float = 12.0):
    """The oracle as it stands, timed on the host cores on a bounded sample of
    the same workload: whole sequences of the batch, in batch order, until the
    estimated time reaches target_s (first a one-sequence probe)."""
    import oracle
    oracle.lib()
    k, v = batch.k_pool.copy(), batch.v_pool.copy()
    oracle.kv_append(k, v, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.k_new, batch.v_new)
    rows = batch.q_indptr

    def run(seqs):
        ql = np.zeros_like(batch.q_lens)
        ql[seqs] = batch.q_lens[seqs]
        qsel = np.concatenate([batch.q[rows[s]:rows[s + 1]] for s in seqs])
        t0 = time.perf_counter()
        oracle.attention(k, v, ql, batch.ctx_lens, batch.block_tables, qsel)
        return time.perf_counter() - t0, int(batch.ctx_lens[seqs].astype(np.int64).sum())

    active = [int(s) for s in np.nonzero(batch.q_lens > 0)[0]]
    # cost of a sequence ~ q_len * ctx_len
    cost = {s: float(batch.q_lens[s]) * float(batch.ctx_lens[s]) for s in active}
    chosen = pick_sequences(active, cost, lambda seqs: run(seqs)[0], target_s)
    # the sample is repeated until about 10 s of oracle time have been spent (a workload the oracle
    # finishes in a fraction of a second would otherwise give a noisy figure)
    t, toks, reps = 0.0, 0, 0
    while reps == 0 or (t < 10.0 and reps < 1000):
        dt, n = run(chosen)
        t, toks, reps = t + dt, toks + n, reps + 1
    return {"value": toks / t, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{len(chosen)} of {len(active)} sequences of the workload ({toks // reps} KV-tokens, "
                      f"all heads, fp64), repeated {reps} times, {t:.2f} s in all"}


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    batch = make_batch(args.config)
    oracle.lib()
    k, v = batch.k_pool.copy(), batch.v_pool.copy()
    rows = batch.q_indptr
    active = [int(s) for s in np.nonzero(batch.q_lens > 0)[0]]
    # bounded sample: whole sequences in batch order, ~2 s of oracle time per step
    oracle.kv_append(k, v, batch.q_lens, batch.ctx_lens, batch.block_tables, batch.k_new, batch.v_new)
    cost = {s: float(batch.q_lens[s]) * float(batch.ctx_lens[s]) for s in active}

    def run_seconds(seqs):
        ql_ = np.zeros_like(batch.q_lens); ql_[seqs] = batch.q_lens[seqs]
        q_ = np.concatenate([batch.q[rows[s]:rows[s + 1]] for s in seqs])
        t1 = time.perf_counter()
        oracle.attention(k, v, ql_, batch.ctx_lens, batch.block_tables, q_)
        return time.perf_counter() - t1

    chosen = pick_sequences(active, cost, run_seconds, 2.0)
    ql = np.zeros_like(batch.q_lens); ql[chosen] = batch.q_lens[chosen]
    qsel = np.concatenate([batch.q[rows[s]:rows[s + 1]] for s in chosen])
    knew = np.concatenate([batch.k_new[rows[s]:rows[s + 1]] for s in chosen])
    vnew = np.concatenate([batch.v_new[rows[s]:rows[s + 1]] for s in chosen])
    toks = int(batch.ctx_lens[chosen].astype(np.int64).sum())

    def step():
        oracle.kv_append(k, v, ql, batch.ctx_lens, batch.block_tables, knew, vnew)
        oracle.attention(k, v, ql, batch.ctx_lens, batch.block_tables, qsel)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = toks * args.steps / dt
    sample = f"{len(chosen)} of {len(active)} sequences of the workload per step ({toks} KV-tokens, all heads, fp64)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": batch.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_trace_bench(args):
    """--config 5: the 200-iteration workload-shift trace (single GPU).  The trace is replayed once
    untimed (warm-up) and once timed; a "step" is one serving iteration, timed with CUDA events around
    append + attention; the aggregate is sum(KV-tokens) / sum(device time) over non-empty iterations."""
    import torch
    import paper_2604_07144_b200 as ap
    from paper_2604_07144_b200.trace_runner import TraceRun
    torch.cuda.set_device(0)
    iterations = 200
    per_iter = []
    launches = 0
    for replay in range(2):
        run = TraceRun(iterations=iterations)
        ap.profile_enable(run.pool, replay == 1)
        sampler = ClockSampler(0)
        if replay == 1:
            sampler.start()
        for st in run.steps():
            if replay == 1 and st.kv_tokens:
                per_iter.append((st.index, st.kv_tokens, st.gpu_ms, st.n_prefill, st.n_decode,
                                 int(st.q_lens.sum()), st.info["launches_append"] + st.info["launches_attention"]))
        clocks = sampler.stop() if replay == 1 else None
        kt = ap.profile_collect(run.pool) if replay == 1 else None
        peak_pages, num_pages = run.peak_pages, run.num_pages
        run.close()
    toks = sum(p[1] for p in per_iter)
    ms = sum(p[2] for p in per_iter)
    launches = sum(p[6] for p in per_iter)
    phases = []
    for lo in range(0, iterations, 50):
        sel = [p for p in per_iter if lo <= p[0] < lo + 50]
        t, m = sum(p[1] for p in sel), sum(p[2] for p in sel)
        phases.append({"iterations": f"{lo}-{lo + 49}", "rate_req_s": 2 if (lo // 50) % 2 == 0 else 20,
                       "kv_tokens": t, "device_ms": m, "kv_tokens_per_s": (t / (m * 1e-3) if m else None),
                       "new_tokens": sum(p[5] for p in sel)})
    rates = sorted(p[1] / (p[2] * 1e-3) for p in per_iter)
    return ({
        "metric": METRIC, "value": toks / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": len(per_iter),
        "warmup": iterations, "ms_per_step": ms / max(len(per_iter), 1), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "config5_workload_shift_trace_8b", "iterations": iterations,
                   "non_empty_iterations": len(per_iter), "peak_pages": peak_pages, "pool_pages": num_pages,
                   "l2": "every iteration reads a different, growing working set (up to ~1 GB of KV)",
                   "timing": "CUDA events around append + attention of each iteration; plan build and H2D of the "
                             "new tokens outside"},
        "gpu_launches": launches,
        "per_iteration_kv_tokens_per_s": {"min": rates[0], "median": rates[len(rates) // 2], "max": rates[-1]},
        "phases": phases,
        "kernels": {k: {"launches": n, "us_per_launch": (1e3 * m / n if n else None)} for k, (m, n) in kt.items()},
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples")} if clocks else None,
    })


def run_policy_comparison(args):
    """--config 5 --policies: the workload-shift trace under fixed FCFS policies that differ in token
    budget and prefill chunk size.  Each replay is scored by Eq. "ttotal" of the paper's execution model
    with the measured device time of its iterations as the serving cost (a fixed policy never
    reschedules: one interval, no stale or reconfiguration cost)."""
    import torch
    from paper_2604_07144_b200 import execution_model as M
    from paper_2604_07144_b200.trace_runner import TraceRun
    torch.cuda.set_device(0)
    rows = []
    for budget, chunk in ((8192, 512), (8192, 256), (8192, 1024), (4096, 512), (2048, 256)):
        per_iter, toks, new = [], 0, 0
        for replay in range(2):                                  # first replay warms up
            run = TraceRun(iterations=200, token_budget=budget, chunk=chunk)
            for st in run.steps():
                if replay == 1 and st.kv_tokens:
                    per_iter.append(st.gpu_ms * 1e-3)
                    toks += st.kv_tokens
                    new += int(st.q_lens.sum())
            run.close()
        fb = M.artifact_feedback(M.intervals_from_iterations(per_iter))
        rows.append({"token_budget": budget, "chunk": chunk, "iterations": len(per_iter), "new_tokens": new,
                     "kv_tokens": toks, "T_total_s": fb["T_total"], "N": fb["N"],
                     "kv_tokens_per_s": toks / fb["T_total"], "new_tokens_per_s": new / fb["T_total"],
                     "worst_iteration_ms": 1e3 * max(per_iter)})
    best = min(rows, key=lambda r: r["T_total_s"] / max(r["new_tokens"], 1))
    print(json.dumps({"metric": "trace_completion_time_per_policy", "unit": "s", "n_gpus": 1, "data": "synthetic",
                      "config": {"workload": "config5_workload_shift_trace_8b", "iterations": 200,
                                 "score": "Eq. ttotal with measured append + attention device time of one layer as t_serve; "
                                          "policies that leave prompts unfinished at iteration 200 serve fewer new tokens, "
                                          "so compare T_total per new token"},
                      "policies": rows, "best_per_new_token": {k: best[k] for k in ("token_budget", "chunk")}}))


def run_page_copy_bench(args):
    """--page-copy: every used page of config 2 (534 MB of K+V) moves to a second pool in one call,
    alternating between two destination pools; bytes read + written against the measured copy bandwidth."""
    import torch
    import paper_2604_07144_b200 as ap
    torch.cuda.set_device(0)
    batch = make_batch(2)
    hkv, d = batch.num_kv_heads, batch.head_dim
    used = np.array(sorted({int(batch.block_tables[s, i]) for s in range(batch.batch)
                            for i in range((int(batch.ctx_lens[s]) + 15) // 16)}), np.int32)
    to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    src_planes = (to_dev(batch.k_pool), to_dev(batch.v_pool))
    src = ap.kv_pool_create(batch.num_pages, hkv, d, *src_planes)
    n_dst = len(used)
    dsts = []
    for i in range(3):
        planes = (torch.zeros((n_dst, hkv, 16, d), dtype=torch.bfloat16, device="cuda"),
                  torch.zeros((n_dst, hkv, 16, d), dtype=torch.bfloat16, device="cuda"))
        dsts.append((ap.kv_pool_create(n_dst, hkv, d, *planes), planes,
                     np.random.default_rng(i).permutation(n_dst).astype(np.int32)))
    page_bytes = 2 * hkv * 16 * d * 2
    moved = 2 * len(used) * page_bytes                        # read + written
    for i in range(max(args.warmup, 3)):
        ap.kv_copy_pages(dsts[i % 3][0], src, dsts[i % 3][2], used)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        ap.kv_copy_pages(dsts[i % 3][0], src, dsts[i % 3][2], used)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    # device-only time of the kernel: the pair list of every call is already queued behind the previous call
    peaks = measured_peaks()
    gbs = moved / (ms * 1e-3) / 1e9
    assert all(ap.last_device_status(p[0]) == 0 for p in dsts)
    print(json.dumps({
        "metric": "kv_page_copy_bytes_per_s", "value": gbs, "unit": "GB/s (read + written)", "n_gpus": 1,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": "config2_used_pages_to_a_second_pool", "pages": int(len(used)), "page_bytes": page_bytes,
                   "l2": "three destination pools in rotation; source 534 MB > 126 MB L2",
                   "includes": "upload of the page-pair list (65 KB) and the copy kernel"},
        "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "kernel": "kv_copy_pages", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}", "traffic": None,
                     "bytes_per_launch": moved, "us_per_launch": ms * 1e3},
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")} if clocks else None,
    }))
    for p, _, _ in dsts:
        ap.kv_pool_destroy(p)
    ap.kv_pool_destroy(src)


def measure_config(config: int, args, rank: int, world: int, local_rank: int, side_by_side=None, with_e2e=True,
                   min_region_s: float = 1.0):
    """Times one workload on this rank's GPU and returns every figure the JSON line carries for it.

    Pass 1 (the timed region): `repeats` blocks of K steps, kernels back to back in the stream, no events
    between them; `repeats` is chosen from the warm-up so that the region lasts at least min_region_s
    (clock samples need a region much longer than the sampling period).  Pass 2: the same steps with a
    CUDA-event pair around every kernel, for the per-kernel times.  Then the end-to-end loop through
    ap_serving_iteration_host with pinned host buffers."""
    import torch
    import paper_2604_07144_b200 as ap
    from paper_2604_07144_b200 import replicas

    dev = torch.device("cuda", local_rank)
    batch = make_batch(config, seed_offset=rank)
    hq, hkv, d = batch.num_q_heads, batch.num_kv_heads, batch.head_dim

    def dev_bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(dev).view(torch.bfloat16)

    kv_bytes = batch.kv_tokens * 2 * hkv * d * 2
    copies = args.pool_copies or max(3, int(np.ceil(2.0e9 / max(kv_bytes, 1))))
    copies = min(copies, 16)
    pools, plans, k_planes, v_planes = [], [], [], []
    k0, v0 = dev_bf16(batch.k_pool), dev_bf16(batch.v_pool)
    for c in range(copies):
        kp, vp = (k0, v0) if c == 0 else (k0.clone(), v0.clone())
        k_planes.append(kp); v_planes.append(vp)
        pools.append(ap.kv_pool_create(batch.num_pages, hkv, d, kp, vp, device=local_rank))
        if side_by_side is not None:
            ap.kv_pool_set_side_by_side(pools[-1], side_by_side)
        if args.two_streams:
            ap.kv_pool_set_single_launch(pools[-1], False)
        plans.append(ap.plan_create(pools[-1], batch.q_lens, batch.ctx_lens, batch.block_tables, hq))
    info = ap.plan_get_info(plans[0])
    q, k_new, v_new = dev_bf16(batch.q), dev_bf16(batch.k_new), dev_bf16(batch.v_new)
    out = torch.empty((batch.n_new, hq, d), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((batch.n_new, hq), dtype=torch.float32, device=dev)
    ws_bytes = ap.plan_workspace_bytes(plans[0])
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)

    def step(i):
        c = i % copies
        ap.kv_append(pools[c], plans[c], k_new, v_new)
        ap.attention_iteration(pools[c], plans[c], q, out, lse, ws, ws_bytes)

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier()
        torch.cuda.synchronize()

    reduce_max = lambda x: replicas.reduce_max(x, dev)
    reduce_sum = lambda x: replicas.reduce_sum(x, dev)

    # ---- warm-up, which also sizes the timed region
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(max(args.warmup - 3, 0)):
        step(i)
    torch.cuda.synchronize()
    e0.record()
    for i in range(3):
        step(i)
    e1.record()
    torch.cuda.synchronize()
    for p in pools:
        assert ap.last_device_status(p) == 0
    est_ms = reduce_max(e0.elapsed_time(e1)) / 3
    repeats = max(1, int(np.ceil(min_region_s * 1e3 / max(est_ms * args.steps, 1e-3))))
    n_timed = args.steps * repeats

    sampler = ClockSampler(local_rank)
    barrier()
    if rank == 0:
        sampler.start()
    e0.record()
    for i in range(n_timed):
        step(i)
    e1.record()
    barrier()
    ms_total = reduce_max(e0.elapsed_time(e1))
    for p in pools:
        ap.profile_enable(p, True)
    n_prof = args.steps * min(repeats, max(1, int(np.ceil(0.3e3 / max(est_ms * args.steps, 1e-3)))))
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for i in range(n_prof):
        step(i)
    e3.record()
    barrier()
    ms_total_profiled = reduce_max(e2.elapsed_time(e3))
    clocks = sampler.stop() if rank == 0 else None
    kt = {}
    for p in pools:
        for name, (ms, n) in ap.profile_collect(p).items():
            a = kt.setdefault(name, [0.0, 0])
            a[0] += ms; a[1] += n
        ap.profile_enable(p, False)
        assert ap.last_device_status(p) == 0
    total_tokens = reduce_sum(float(batch.kv_tokens))
    ms_per_step = ms_total / n_timed
    value = total_tokens / (ms_per_step * 1e-3)

    # ---- plan cost (host + upload), reported separately
    t0 = time.perf_counter()
    for _ in range(20):
        ap.plan_destroy(ap.plan_create(pools[0], batch.q_lens, batch.ctx_lens, batch.block_tables, hq))
    torch.cuda.synchronize()
    plan_ms = (time.perf_counter() - t0) / 20 * 1e3

    # ---- end to end through the host-buffer entry point
    e2e = None
    if with_e2e:
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
        hq_, hk_, hv_ = pin(batch.q), pin(batch.k_new), pin(batch.v_new)
        hout = torch.empty((batch.n_new, hq, d), dtype=torch.int16).pin_memory()
        hlse = torch.empty((batch.n_new, hq), dtype=torch.float32).pin_memory()

        def e2e_step(i):
            ap.serving_iteration_host(pools[i % copies], batch.q_lens, batch.ctx_lens, batch.block_tables, hq,
                                      hq_, hk_, hv_, hout, hlse)

        for i in range(3):
            e2e_step(i)
        barrier()
        t0 = time.perf_counter()
        e2e_step(0)
        torch.cuda.synchronize()
        est = (time.perf_counter() - t0) * 1e3
        e2e_steps = max(10, min(n_timed, int(np.ceil(0.5e3 / max(est, 1e-3)))))
        barrier()
        e0.record()
        for i in range(e2e_steps):
            e2e_step(i)
        e1.record()
        barrier()
        e2e_ms = reduce_max(e0.elapsed_time(e1)) / e2e_steps
        e2e = {"value": total_tokens / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(batch.q.nbytes + batch.k_new.nbytes + batch.v_new.nbytes),
               "d2h_bytes_per_step": int(hout.numel() * 2 + hlse.numel() * 4), "ms_per_step": e2e_ms,
               "steps": e2e_steps,
               "includes": "plan build + upload, H2D of q/k_new/v_new, append, attention, D2H of out/lse, sync (the status word is host memory the kernels write directly)"}
        got = torch.from_numpy(hout.numpy().copy()).view(torch.bfloat16).float()
        assert bool(torch.isfinite(got).all()) and bool(torch.isfinite(hlse).all())

    # sanity: the timed path produced finite numbers
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())

    res = None
    if rank == 0:
        peaks = measured_peaks()
        alg = algorithmic_bytes(batch, info)
        kernels = {name: {"launches": n, "us_per_launch": (1e3 * ms / n if n else None)} for name, (ms, n) in kt.items()}
        dec_us = kernels.get("decode_splitk", {}).get("us_per_launch")
        pre_us = kernels.get("prefill", {}).get("us_per_launch")
        fus_us = kernels.get("mixed_iteration", {}).get("us_per_launch")
        # the profile sums cover this rank's launches only
        achieved = alg["decode_kernel"] / (dec_us * 1e-6) / 1e9 if dec_us else 0.0
        decode_roofline = {
            "bound": "hbm", "kernel": "decode_splitk", "achieved": achieved, "peak": peaks["hbm_gbs"],
            "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "peak_source": f"of {peaks['source']}",
            "traffic": NCU_TRAFFIC.get(("decode_splitk", config, kernel_source_hash("decode_splitk.cu", "decode_splitk.cuh"))),
            "bytes_per_launch": alg["decode_kernel"], "us_per_launch": dec_us,
            "frac_of_nominal_8TBs": achieved / 8000.0,
        }
        concurrent = bool(info["side_by_side"]) or bool(fus_us)
        if concurrent:
            decode_roofline["note"] = ("in this plan decode shares the GPU with prefill, so its own time is not a "
                                       "whole-GPU bandwidth figure; see step_roofline")
        if not dec_us:
            decode_roofline.update(achieved=None, frac=None, frac_of_nominal_8TBs=None,
                                   note="no decode kernel of its own in this plan (one launch holds both parts, or the "
                                        "batch has no decode rows); see step_roofline")
        prefill_roofline = None
        if pre_us:
            tf = alg["prefill_flops"] / (pre_us * 1e-6) / 1e12
            prefill_roofline = {
                "bound": "tensor", "kernel": "prefill_tcgen05", "achieved": tf, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s", "frac": tf / peaks["bf16_tflops"], "peak_source": f"of {peaks['source']} (burst)",
                "peak_sustained": peaks["bf16_tflops_sustained"], "frac_of_sustained": tf / peaks["bf16_tflops_sustained"],
                "which_applies": "the kernel is timed inside a loop of about a second under the power limit (see clocks), "
                                 "which is the condition of the sustained figure; the burst figure is what a launch "
                                 "timed alone would be held against",
                "frac_of_nominal_2250": tf / 2250.0,
                "traffic": NCU_TRAFFIC.get(("prefill_tcgen05", config,
                                            kernel_source_hash("prefill_tcgen05.cu", "prefill_tcgen05.cuh"))),
                "flops_per_launch": alg["prefill_flops"], "us_per_launch": pre_us,
            }
            if concurrent:
                prefill_roofline["note"] = "runs next to the decode kernel in this plan: not a whole-GPU figure"
        # whole step against the slower of its two bounds: all algorithmic bytes at the measured copy
        # bandwidth, all algorithmic flops at the measured bf16 peak
        t_bytes = alg["total"] / (peaks["hbm_gbs"] * 1e9)
        t_flops = (alg["decode_flops"] + alg["prefill_flops"]) / (peaks["bf16_tflops"] * 1e12)
        step_roofline = {"bound_us": max(t_bytes, t_flops) * 1e6, "bytes_us": t_bytes * 1e6, "flops_us": t_flops * 1e6,
                         "sum_us": (t_bytes + t_flops) * 1e6, "step_us": ms_per_step * 1e3,
                         "frac": max(t_bytes, t_flops) / (ms_per_step * 1e-3),
                         "note": "bound = max(bytes / copy bandwidth, flops / bf16 peak): reachable only if the "
                                 "HBM-bound and the tensor-bound parts overlap perfectly; sum = no overlap"}
        launches_per_step = info["launches_append"] + info["launches_attention"]
        res = {
            "value": value, "ms_per_step": ms_per_step, "steps": args.steps, "repeats": repeats, "timed_steps": n_timed,
            "timed_ms": ms_total,
            "config": {"workload": batch.name, "num_q_heads": hq, "num_kv_heads": hkv, "head_dim": d,
                       "page_size": 16, "sequences": batch.batch, "new_tokens": batch.n_new,
                       "kv_tokens_per_step_per_gpu": batch.kv_tokens,
                       "dispatch": ("one launch: decode CTAs + prefill units" if fus_us else
                                    "two streams: decode beside prefill" if info["side_by_side"] else "sequential"),
                       "l2": f"rotation among {copies} pool copies ({copies * kv_bytes / 1e9:.2f} GB of KV, each step's "
                             f"{kv_bytes / 1e6:.0f} MB larger than the 126 MB L2)",
                       "timed_region": f"{repeats} x {args.steps} steps back to back ({ms_total:.0f} ms), sized from the warm-up "
                                       f"to last >= {min_region_s} s so the clock sampler sees it",
                       "parallelism": "replicas only (one independent batch per GPU, no collective)"},
            "gpu_launches": int(n_timed * launches_per_step),
            "e2e": e2e,
            "plan": {"host_ms": plan_ms, "in_value": False, "in_e2e": True, **{k: info[k] for k in (
                "decode_items", "decode_ctas", "merge_entries", "prefill_tiles", "side_by_side")}},
            "roofline": decode_roofline,
            "prefill_roofline": prefill_roofline,
            "step_roofline": step_roofline,
            "kernels": kernels,
            "kernel_timing": {"how": "second pass of the same steps with a CUDA-event pair around every kernel, "
                                     "right after the timed pass; the timed pass itself has no events between kernels",
                              "steps": n_prof, "ms_per_step_with_events": ms_total_profiled / n_prof},
            "paper_model_us": {"decode_splitk": paper_model_us(alg["decode_flops"], alg["decode_kernel"], peaks),
                               "prefill": paper_model_us(alg["prefill_flops"], alg["prefill_kernel"], peaks),
                               "note": "T_op = F / min(F/A * B, F_peak) with this GPU's measured copy bandwidth and "
                                       "bf16 peak; compare with kernels.*.us_per_launch"},
            "prediction": {**{k: v for k, v in ap.plan_predict(plans[0], peaks["hbm_gbs"], peaks["bf16_tflops"]).items()
                              if k.endswith("_us")},
                           "note": "ap_plan_predict: roofline_* = the paper's operator model computed by the library, "
                                   "model_* = the planner's calibrated cost model; compare model_step_us with ms_per_step"},
            "prefill_tflops": prefill_roofline["achieved"] if prefill_roofline else None,
            "step_gbs": alg["total"] / (ms_per_step * 1e-3) / 1e9,
            "clocks": ({**{k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples", "power_w")},
                        "ms_x_mhz": (ms_per_step * clocks["sm_mhz"] if clocks["sm_mhz"] else None)} if clocks else None),
        }
    for pl in plans:
        ap.plan_destroy(pl)
    for p in pools:
        ap.kv_pool_destroy(p)
    del k_planes, v_planes, k0, v0, q, k_new, v_new, out, lse, ws
    torch.cuda.empty_cache()
    return res, batch


def compact(res):
    """The figures of one extra workload that go under `configs` in the JSON line."""
    keep = ("value", "ms_per_step", "repeats", "timed_steps", "timed_ms", "gpu_launches", "kernels", "roofline",
            "prefill_roofline", "prefill_tflops", "step_roofline", "step_gbs", "e2e", "clocks", "prediction")
    out = {k: res[k] for k in keep if k in res}
    out["workload"] = res["config"]["workload"]
    out["dispatch"] = res["config"]["dispatch"]
    out["plan"] = res["plan"]
    for r in ("roofline", "prefill_roofline"):
        if out.get(r):
            out[r] = {k: v for k, v in out[r].items() if k not in ("note",)}
    return out


def main():
    ap_ = argparse.ArgumentParser()
    ap_.add_argument("--gpus", type=int, default=1)
    ap_.add_argument("--steps", type=int, default=100)
    ap_.add_argument("--warmup", type=int, default=10)
    ap_.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap_.add_argument("--config", type=int, default=0, choices=[0, 2, 3, 4, 5],
                     help="0 (default): config 2 is the headline value and configs 3 (both dispatch modes), 4 and the "
                          "config-5 trace are timed in the same run and reported under `configs`; 2|3|4|5: that one only")
    ap_.add_argument("--pool-copies", type=int, default=0, help="0 = enough copies for >= 2 GB of KV")
    ap_.add_argument("--no-cpu-baseline", action="store_true")
    ap_.add_argument("--min-region-s", type=float, default=1.0,
                     help="the K steps are repeated until the timed region lasts at least this long")
    ap_.add_argument("--policies", action="store_true",
                     help="with --config 5: replay the trace under several fixed scheduling policies (token budget, "
                          "prefill chunk) and score each by the paper's trace completion time on measured iterations")
    ap_.add_argument("--page-copy", action="store_true",
                     help="time ap_kv_copy_pages on config 2's used pages instead of the serving iteration")
    ap_.add_argument("--two-streams", action="store_true",
                     help="mixed iterations: the decode and prefill kernels on two streams instead of one launch")
    ap_.add_argument("--side-by-side", type=int, default=None,
                     help="mixed iterations: 0 = decode then prefill, 1 = planner decides (library default), "
                          "k >= 2 = decode on k CTAs next to prefill")
    args = ap_.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    all_configs = args.config == 0
    if all_configs:
        args.config = 2

    if args.impl == "reference":
        run_reference(args)
        return

    if args.page_copy:
        run_page_copy_bench(args)
        return

    if args.config == 5 and args.policies:
        run_policy_comparison(args)
        return

    if args.config == 5:
        print(json.dumps(run_trace_bench(args)))
        return

    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # replicas only: every rank serves its own independent batch, no data-path collective
    res, batch = measure_config(args.config, args, rank, world, local_rank, side_by_side=args.side_by_side,
                                min_region_s=args.min_region_s)
    extras = {}
    if all_configs and world == 1:
        # the other roofline-bearing workloads, in the same process and on the same GPU
        r3s, _ = measure_config(3, args, rank, world, local_rank, side_by_side=0, min_region_s=args.min_region_s)
        extras["config3_sequential"] = compact(r3s)
        r3, _ = measure_config(3, args, rank, world, local_rank, min_region_s=args.min_region_s)
        extras["config3"] = compact(r3)
        r4, _ = measure_config(4, args, rank, world, local_rank, min_region_s=args.min_region_s)
        extras["config4"] = compact(r4)
        t5 = run_trace_bench(args)
        extras["config5"] = {k: t5[k] for k in ("value", "ms_per_step", "steps", "gpu_launches", "phases",
                                                "per_iteration_kv_tokens_per_s", "kernels", "clocks")}
        extras["config5"]["workload"] = t5["config"]["workload"]

    if rank == 0:
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        }
        line.update({k: v for k, v in res.items() if k not in ("value", "ms_per_step", "steps")})
        if extras:
            line["configs"] = extras
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_baseline(batch)
        print(json.dumps(line))

    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
