#!/usr/bin/env python
"""Benchmark of the FCP attention hot path: forward over the block plan with the merge on the fly
(`fcp_attn_fwd_fused`) + backward (`fcp_attn_bwd`) on one synthetic packed batch per step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

Prints one JSON line.  The default workload is the largest single-GPU configuration (`extreme_512k`);
short runs of the other long-context workloads are reported under `other_workloads`.  With N > 1 the
script starts its own N ranks through torch.distributed.run unless it already runs under one (one
rank per GPU); every rank processes its own batch (seed = rank): the path has no data-path
collective, so scaling is weak and the time is the max over ranks.  `--impl reference` times the
fp64 CPU oracle on a bounded sample of the same workload.

Bench inputs are N(0,1) bf16 tensors drawn on the device by a seeded generator (no parity is checked
here; the parity tests use the host generator whose bits also feed the oracle).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fwd+bwd attention TFLOPS/GPU on packed varlen batches"
NOMINAL_BF16_TFLOPS = 2250.0      # vendor's public dense BF16 figure, for context only
OTHER_WORKLOADS = ("longtail_256k", "bimodal_128k", "bimodal_128k_spans")
KERNEL_KINDS = ["attn_fwd", "lse_merge", "bwd_preprocess", "attn_bwd", "dq_convert"]

# DRAM bytes (read + write) of one backward-kernel launch of the timed workload from an ncu capture, with the digest
# of the sources that decide the kernel and its work order: reported only while they still match.  The default
# workload has no entry: its launch runs for seconds and the DRAM counters take several replay passes, so it is
# captured on a small case only; the traffic of a launch does not scale from a small case in proportion (it depends
# on what stays in L2), so `roofline.traffic` is null and the small-case capture is reported beside it.
NCU_BWD_TRAFFIC = {}
NCU_BWD_TRAFFIC_SMALL_CASE = {
    "workload": "longtail_256k cut to 5 query heads on 1 KV head", "traffic": 4035786000 + 2922308000,
    "algorithmic_bytes": 2282000000, "ms": 52.8, "summary": "profiles/bwd_kernel_longtail_256k_5heads.md"}


def bwd_kernel_digest():
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2602_21788_b200", "csrc")
    for f in ("fcp_bwd.cuh", "sm100_ptx.cuh", "fcp_plan.cpp", "fcp_plan.hpp"):
        with open(os.path.join(csrc, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(w, args):
    rec = NCU_BWD_TRAFFIC.get(w.name)
    if rec is None or args.max_heads > 0 or args.seed != 0:
        return None
    return rec["bytes"] if rec["digest"] == bwd_kernel_digest() else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


def config_of(w, seed):
    """The keys both arms print for the workload."""
    return {"workload": w.name, "tokens": w.total_tokens, "sequences": int(len(w.seqlens)), "hq": w.hq, "hkv": w.hkv,
            "head_dim": w.head_dim, "seed": seed, "sum_len_sq": w.sum_sq,
            "cp_degrees": sorted(set(int(x) for x in w.cp_degrees)),
            "spans": sum(len(x) for x in w.spans) if w.spans else 0,
            "flops": "7 * sum(L^2) * hq * head_dim per step" + (" (+ 14 * hq * head_dim per pair a span adds)" if w.spans else "")}


# --------------------------------------------------------------------------------------------
# CPU oracle leg
# --------------------------------------------------------------------------------------------
def host_sequence_inputs(w, b, h):
    """N(0,1) bf16 inputs (as float64) of one (sequence, query head) problem, seeded by (seed, b, h)."""
    from paper_2602_21788_b200 import synth
    rng = np.random.Generator(np.random.PCG64([w.seed, 0xB0, int(b), int(h)]))
    L = int(w.seqlens[b])
    return [synth.bf16_bits_to_f64(synth.normal_bf16(rng, (L, w.head_dim))) for _ in range(4)]


def oracle_sample(w, budget_s: float):
    """Runs the oracle (as it stands) on (sequence, head) problems of the workload, longest sequences
    of at most 8192 tokens first, head 0 then 1 ..., until `budget_s` seconds are spent.  Returns
    (useful FLOPs by the headline accounting, seconds, description)."""
    from oracle import attention_ref as A
    order = np.argsort(-w.seqlens, kind="stable")
    order = [int(b) for b in order if w.seqlens[b] <= 8192] or [int(order[-1])]
    flops, done, spent = 0.0, 0, 0.0
    for h in range(w.hq):
        for b in order:
            qs, ks, vs, dos = host_sequence_inputs(w, b, h)
            L = int(w.seqlens[b])
            t0 = time.perf_counter()
            for rows in A._slabs(L, 2048):
                A.attention_fwd_seq(qs, ks, vs, rows)
                A.attention_bwd_seq(qs, ks, vs, dos, rows)
            spent += time.perf_counter() - t0
            flops += 7.0 * float(L) ** 2 * w.head_dim
            done += 1
            if spent > budget_s:
                return flops, spent, f"{done} (sequence, head) problems, sequences <= 8192 tokens, longest first"
    return flops, spent, f"all {done} (sequence, head) problems with sequences <= 8192 tokens"


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    per_step = 4.0
    for _ in range(max(args.warmup, 0)):
        oracle_sample(w, per_step / 4)
    tot_f, tot_t, desc = 0.0, 0.0, ""
    for _ in range(args.steps):
        fl, dt, desc = oracle_sample(w, per_step)
        tot_f += fl
        tot_t += dt
    val = tot_f / tot_t / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOPS", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, args.seed),
        "cpu_baseline": {"value": val, "unit": "TFLOPS", "cores": blas_threads(), "kind": "oracle",
                         "sample": f"each step: {desc}, about {per_step:.0f} s"},
        "e2e": {"value": val, "unit": "TFLOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.samples, self.proc = [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.perf_counter(), line.strip()))

    def window(self, t_begin, t_end):
        """Median SM clock, maximum and the throttle reasons seen between two perf_counter instants."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [s for t, s in self.samples if t_begin <= t <= t_end] or [s for _, s in self.samples[-3:]]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except Exception:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def per_ghz(tflops, clocks):
    """Clock-normalised throughput: TFLOPS per GHz of the median SM clock sampled during the timed region."""
    mhz = (clocks or {}).get("sm_mhz")
    return tflops / (mhz / 1000.0) if mhz else None


def time_planner(w, reps=20):
    """Host time of the two planner calls alone (no CUDA call inside the timers), microseconds."""
    from paper_2602_21788_b200 import costfit, fcp
    lens = w.seqlens
    coeffs = dict(costfit.B200_COEFFS, alpha3=0.0, beta2=0.0, v=1.0)
    budget = float(max(8192, int(np.ceil(lens.max() / 8))))     # activation budget per rank, in tokens
    N = 16
    out = {}
    t = []
    for _ in range(reps):
        t0 = time.perf_counter()
        plan = fcp.fcp_plan_blocks(lens, w.cp_degrees, w.hq, w.hkv, w.head_dim)
        t.append(time.perf_counter() - t0)
        del plan
    out["plan_blocks_us"] = 1e6 * statistics.median(t)
    t = []
    res = None
    for _ in range(reps):
        t0 = time.perf_counter()
        try:
            res = fcp.fcp_plan_strategy(lens, N, budget, 1.0, 0.0, coeffs)
        except fcp.FcpError:
            res = None
        t.append(time.perf_counter() - t0)
    out["plan_strategy_us"] = 1e6 * statistics.median(t)
    out["plan_strategy_case"] = {"sequences": int(len(lens)), "ranks": N, "budget_tokens_per_rank": budget,
                                 "groups": None if res is None else int(res["n_groups"]),
                                 "paper_solver_ms": "20-86 (Sec. 6.3, its own batches, host CPU and language unstated)"}
    return out


def measure(w, seed, steps, warmup, sampler, dist_ctx, heads_per_pass=0, want_partial_path=False):
    """Times `steps` passes of fused forward + backward on workload `w`.  Returns a dict of raw results."""
    import torch

    from paper_2602_21788_b200 import ranks
    from paper_2602_21788_b200.runner import DeviceState

    q, k, v, do = w.device_tensors()
    ds = DeviceState(w, q, k, v, do, heads_per_pass=heads_per_pass or None, partials=False)
    del q, k, v, do
    plan = ds.plan

    def step():
        ds.forward_fused()
        ds.backward()

    def barrier():
        torch.cuda.synchronize()
        if dist_ctx is not None:
            dist_ctx.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step()
    barrier()
    ds.check_status()
    plan.set_profiling(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.perf_counter()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    barrier()
    t_end = time.perf_counter()
    ms = ev0.elapsed_time(ev1)
    ds.check_status()
    clocks = sampler.window(t_begin, t_end) if sampler else None
    kern = {}
    for kind, name in enumerate(KERNEL_KINDS):
        n, kms = plan.kernel_ms(kind)
        kern[name] = {"launches": n, "mean_ms": kms}
    plan.set_profiling(False)
    ms_all, flops_total = ranks.aggregate(ms, w.flops_fwd_bwd(), "cuda")
    res = dict(ds=ds, ms=ms_all, ms_local=ms, wall_s=t_end - t_begin, flops_total=flops_total, clocks=clocks, kernels=kern,
               passes=-(-w.hq // ds.hpp), value=ranks.throughput_tflops(ms_all, steps, flops_total))

    if want_partial_path:
        # The partial-producing path of the same plan (forward per item -> fp32 partials -> merge kernel), in
        # head passes that keep the partial buffers below about 20 GB: evidence for the merge kernel's HBM rate.
        R = plan.info("R")
        hpp = max(1, min(w.hq, int(20e9 // (R * (4 * w.head_dim + 4)))))
        ds.hpp = hpp
        ds.o_part = torch.empty((R, hpp, w.head_dim), dtype=torch.float32, device="cuda")
        ds.lse_part = torch.empty((R, hpp), dtype=torch.float32, device="cuda")
        ds.forward(merged=True)
        torch.cuda.synchronize()
        plan.set_profiling(True)
        ds.forward(merged=True)
        torch.cuda.synchronize()
        n_f, f_ms = plan.kernel_ms(0)
        n_m, m_ms = plan.kernel_ms(1)
        plan.set_profiling(False)
        ds.check_status()
        mu = plan.table("merge_units")[: plan.info("n_merge_multi")]
        so = plan.table("slot_offset")
        n_slots = (so[mu[:, 2] + 1] - so[mu[:, 2]]).astype(np.int64)
        merge_tokens = int(mu[:, 1].sum())
        merge_bytes = (int((mu[:, 1] * n_slots).sum()) * w.hq * (4 * w.head_dim + 4)
                       + merge_tokens * w.hq * (2 * w.head_dim + 4))
        passes = -(-w.hq // hpp)
        res["partial_path"] = {
            "call": "fcp_attn_fwd_merged (per-item partials + fcp_lse_merge kernel)", "head_passes": passes,
            "partial_rows": R, "merged_tokens": merge_tokens,
            "attn_fwd_ms": f_ms * passes, "attn_fwd_tflops": w.flops_fwd() / (f_ms * passes * 1e-3) / 1e12 if f_ms > 0 else None,
            "lse_merge_ms": m_ms * passes, "merge_bytes": merge_bytes,
            "merge_gbs": merge_bytes / (m_ms * passes * 1e-3) / 1e9 if m_ms > 0 else None}
        del ds.o_part, ds.lse_part
    return res


def run_e2e(w, ds, n_e2e, barrier):
    """The same step through the host entry point: pinned host buffers in, pinned host buffers out."""
    import torch

    from paper_2602_21788_b200 import fcp
    T, hq, hkv, D = w.total_tokens, w.hq, w.hkv, w.head_dim
    plan = ds.plan

    def pinned_copy(t):
        h = torch.empty(t.shape, dtype=torch.int16, pin_memory=True)
        h.copy_(t.view(torch.int16))
        return h

    hq_, hk_, hv_, hdo_ = pinned_copy(ds.q), pinned_copy(ds.k), pinned_copy(ds.v), pinned_copy(ds.do)
    for name in ("q", "k", "v", "do", "o", "lse", "dq", "dk", "dv", "scratch"):
        setattr(ds, name, None)
    torch.cuda.empty_cache()
    ho = torch.empty((T, hq, D), dtype=torch.int16, pin_memory=True)
    hdq = torch.empty((T, hq, D), dtype=torch.int16, pin_memory=True)
    hdk = torch.empty((T, hkv, D), dtype=torch.int16, pin_memory=True)
    hdv = torch.empty((T, hkv, D), dtype=torch.int16, pin_memory=True)
    hlse = torch.empty((T, hq), dtype=torch.float32, pin_memory=True)
    nbytes = plan.host_workspace_bytes()
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    call = lambda: fcp.fcp_attn_fwd_bwd_host(plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, nbytes, st)
    call()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n_e2e):
        call()
    e1.record()
    barrier()
    st_words = plan.device_status()
    if st_words[0] != 0:
        raise RuntimeError(f"device status {int(st_words[0])} after the host entry point")
    h2d = 2 * (2 * T * hq * D + 2 * T * hkv * D)
    d2h = 2 * (2 * T * hq * D + 2 * T * hkv * D) + 4 * T * hq
    return e0.elapsed_time(e1) / n_e2e, h2d, d2h


def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2602_21788_b200 import ranks, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()

    # each rank has its own batch: independent problems, no data-path collective
    if world > 1:
        w = ranks.rank_workload(args.workload, args.seed, rank, world, args.max_heads)
    sampler = ClockSampler(local) if rank == 0 else None
    planner = time_planner(w) if rank == 0 else None

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    main = measure(w, args.seed + rank, args.steps, args.warmup, sampler, dist if world > 1 else None,
                   heads_per_pass=args.heads_per_pass, want_partial_path=(rank == 0 and not args.no_partial_path))
    ds = main["ds"]
    value, ms_per_step = main["value"], main["ms"] / args.steps
    kern, clocks, passes = main["kernels"], main["clocks"], main["passes"]
    flops_total = main["flops_total"]

    # ---- end to end from pinned host buffers through the host entry point
    e2e = None
    # every rank of this node pins its own host copies of all inputs and outputs: leave the leg out (on all ranks
    # alike, it contains a reduction) rather than exhaust the host memory when N batches of this size do not fit
    pinned_need = world * (8 * w.total_tokens * (w.hq + w.hkv) * w.head_dim + 4 * w.total_tokens * w.hq)
    host_ok = True
    try:
        import psutil
        host_ok = pinned_need <= 0.6 * psutil.virtual_memory().available
    except Exception:
        pass
    if world > 1:
        flag = torch.tensor([1 if host_ok else 0], device="cuda")
        dist.all_reduce(flag, op=dist.ReduceOp.MIN)
        host_ok = bool(flag.item())
    if not args.no_e2e and not host_ok:
        e2e = {"value": None, "unit": "TFLOPS", "skipped": "pinned host buffers of %d ranks (%.0f GB) exceed the host memory"
               % (world, pinned_need / 1e9)}
    if not args.no_e2e and host_ok:
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        e_ms, h2d, d2h = run_e2e(w, ds, n_e2e, barrier)
        e_ms, _ = ranks.aggregate(e_ms, 0.0, "cuda")
        e2e = {"value": flops_total / (e_ms * 1e-3) / 1e12, "unit": "TFLOPS", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e,
               "call": "fcp_attn_fwd_bwd_host, pinned host buffers"}
    plan = ds.plan
    n_fused = plan.info("n_fused_units")
    n_bwd_units = plan.info("n_bwd_units")
    del ds, main["ds"]
    torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (backward attention): algorithmic FLOPs = 2.5 x forward.
    # Denominator from the run itself: the burst cuBLAS figure when the timed region is short or the SM clock
    # stayed near its maximum, the sustained one when the region ran for seconds under the power cap.
    bwd_ms = kern["attn_bwd"]["mean_ms"]
    fwd_ms = kern["attn_fwd"]["mean_ms"] * passes      # all head passes of one step
    bwd_flops = 2.5 * w.flops_fwd()
    achieved = bwd_flops / (bwd_ms * 1e-3) / 1e12 if bwd_ms > 0 else None
    sm, smx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    near_max = bool(sm and smx and sm >= 0.9 * smx)
    use_burst = main["wall_s"] < 2.0 or near_max
    peak = peaks["bf16_burst"] if use_burst else peaks["bf16_sustained"]
    why = (f"timed region {main['wall_s']:.1f} s, median SM clock {sm} of {smx} MHz: "
           + ("burst figure (short region or clock near maximum)" if use_burst
              else "sustained figure (seconds under the power cap, clock well below maximum)"))
    roofline = {"bound": "tensor", "kernel": "fcp_bwd_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None, "traffic": ncu_traffic(w, args),
                "traffic_small_case": NCU_BWD_TRAFFIC_SMALL_CASE,
                "flops_per_launch": bwd_flops, "ms_per_launch": bwd_ms,
                "peak_source": f"{peaks['source']} {'burst' if use_burst else 'sustained'} bf16 cuBLAS; {why}",
                "fwd_kernel": {"achieved": w.flops_fwd() / (fwd_ms * 1e-3) / 1e12 if fwd_ms > 0 else None, "ms": fwd_ms,
                               "frac": w.flops_fwd() / (fwd_ms * 1e-3) / 1e12 / peak if fwd_ms > 0 else None},
                "frac_of_burst": achieved / peaks["bf16_burst"] if achieved else None,
                "frac_of_sustained": achieved / peaks["bf16_sustained"] if achieved else None,
                "frac_of_vendor_dense_bf16": achieved / NOMINAL_BF16_TFLOPS if achieved else None}

    # ---- short runs of the other long-context workloads (N = 1 only)
    others = {}
    if world == 1 and not args.no_other_workloads and args.max_heads == 0:
        for name in OTHER_WORKLOADS:
            if name == w.name:
                continue
            ow = synth.make_workload(name, args.seed)
            r = measure(ow, args.seed, args.other_steps, 3, sampler, None)
            k2 = r["kernels"]
            others[name] = {
                "value": r["value"], "unit": "TFLOPS", "steps": args.other_steps, "warmup": 3,
                "ms_per_step": r["ms"] / args.other_steps, "config": config_of(ow, args.seed),
                "attn_fwd_ms": k2["attn_fwd"]["mean_ms"], "attn_bwd_ms": k2["attn_bwd"]["mean_ms"],
                "attn_fwd_tflops": ow.flops_fwd() / (k2["attn_fwd"]["mean_ms"] * 1e-3) / 1e12,
                "attn_bwd_tflops": 2.5 * ow.flops_fwd() / (k2["attn_bwd"]["mean_ms"] * 1e-3) / 1e12,
                "frac_of_burst": r["value"] / peaks["bf16_burst"], "frac_of_sustained": r["value"] / peaks["bf16_sustained"],
                "frac_of_vendor_dense_bf16": r["value"] / NOMINAL_BF16_TFLOPS, "clocks": r["clocks"],
                "tflops_per_sm_ghz": per_ghz(r["value"], r["clocks"])}
            del r
            torch.cuda.empty_cache()
    if sampler:
        sampler.stop()

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        fl, dt, desc = oracle_sample(w, args.cpu_seconds)
        cpu = {"value": fl / dt / 1e12, "unit": "TFLOPS", "cores": blas_threads(), "kind": "oracle",
               "sample": f"{desc}; {dt:.1f} s of fp64 numpy"}

    cfg = config_of(w, args.seed)
    cfg.update({"l2": "inputs larger than L2 (q alone is %d MB)" % (2 * w.total_tokens * w.hq * w.head_dim >> 20),
                "step": "fcp_attn_fwd_fused + fcp_attn_bwd", "head_passes": passes, "fused_units": n_fused,
                "bwd_units": n_bwd_units, "inputs": "N(0,1) bf16 drawn on the device, seeded"})
    cfg.update(planner or {})
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": cfg,
        "frac_of_peak": {"measured_sustained": value / world / peaks["bf16_sustained"],
                         "measured_burst": value / world / peaks["bf16_burst"],
                         "vendor_dense_bf16": value / world / NOMINAL_BF16_TFLOPS},
        "kernels": kern, "roofline": roofline, "partial_path": main.get("partial_path"), "other_workloads": others,
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": args.steps * (passes + 3), "clocks": clocks,
        "tflops_per_sm_ghz": per_ghz(value / world, clocks),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# launcher
# --------------------------------------------------------------------------------------------
def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def relaunch_ranks(n: int) -> int:
    """Starts this script as n ranks (one per GPU) through torch.distributed.run on this node."""
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")              # keep the communicator set-up lines in the log
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def run_launcher_selftest(args):
    """The rank plumbing of `run_ours` on CPU (`gloo`), with a sleep in place of the GPU step: no measurement."""
    import torch.distributed as dist

    from paper_2602_21788_b200 import ranks
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    w = ranks.rank_workload("tiny", args.seed, rank, world)
    t0 = time.perf_counter()
    time.sleep(0.01 * (rank + 1))
    ms = 1e3 * (time.perf_counter() - t0)
    ms_all, flops_total = ranks.aggregate(ms, w.flops_fwd_bwd(), "cpu")
    if rank == 0:
        print(json.dumps({"selftest": "launcher", "metric": METRIC, "value": None, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "scaling": "weak", "max_ms_over_ranks": ms_all,
                          "flops_all_ranks": flops_total, "flops_rank0": w.flops_fwd_bwd()}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="extreme_512k")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-other-workloads", action="store_true")
    ap.add_argument("--other-steps", type=int, default=10, help="timed steps of each workload under other_workloads")
    ap.add_argument("--no-partial-path", action="store_true")
    ap.add_argument("--heads-per-pass", type=int, default=0, help="query heads per forward pass (0 = all)")
    ap.add_argument("--max-heads", type=int, default=0,
                    help="keep at most this many query heads (query:KV ratio kept); a small case for profiler captures, "
                         "named <workload>_reduced in the output")
    ap.add_argument("--selftest-launcher", action="store_true",
                    help="CPU check of the rank plumbing (gloo, a sleep instead of the GPU step); prints no measurement")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    world = int(os.environ.get("WORLD_SIZE", "0"))
    if args.gpus > 1 and world == 0 and args.impl == "ours":
        sys.exit(relaunch_ranks(args.gpus))
    if args.selftest_launcher:
        run_launcher_selftest(args)
        return

    from paper_2602_21788_b200 import synth
    w = synth.make_workload(args.workload, args.seed)
    if args.max_heads > 0:
        w = synth.reduced(w, len_div=1, max_heads=args.max_heads)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
