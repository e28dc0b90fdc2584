#!/usr/bin/env python
"""Benchmark of the FCP attention hot path (forward over the block plan + LSE merge + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one synthetic packed batch.  Prints one JSON line.
With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank processes its own batch
(seed = rank): the path has no data-path collective, so scaling is weak; timing is the max over ranks.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
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

# DRAM bytes (read + write) of one backward-kernel launch from an ncu capture of this command line, with the
# digest of the kernel sources the counters were taken on: reported only while the sources still match.
NCU_BWD_TRAFFIC = {"llama8b_64k": (2499581440 + 1298159872, "4b313e6f3ea9283d")}


def bwd_kernel_digest():
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(os.path.dirname(os.path.abspath(__file__)), "paper_2602_21788_b200", "csrc")
    for f in ("fcp_bwd.cuh", "sm100_ptx.cuh"):
        with open(os.path.join(csrc, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(w, args):
    rec = NCU_BWD_TRAFFIC.get(w.name)
    if rec is None or args.max_heads > 0 or args.seed != 0:
        return None
    return rec[0] if rec[1] == bwd_kernel_digest() else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# --------------------------------------------------------------------------------------------
# CPU oracle leg
# --------------------------------------------------------------------------------------------
def oracle_sample(w, q, k, v, do, budget_s: float):
    """Runs the oracle (as it stands) on (sequence, head) problems of the workload, longest sequences
    first, head 0 then 1 ..., until `budget_s` seconds are spent.  Returns (useful FLOPs by the
    headline accounting, seconds, description)."""
    from oracle import attention_ref as A
    from paper_2602_21788_b200 import synth
    f = synth.bf16_bits_to_f64
    cu = w.cu_seqlens
    g = w.hq // w.hkv
    order = np.argsort(-w.seqlens, kind="stable")
    order = [b for b in order if w.seqlens[b] <= 8192] or [int(order[-1])]
    flops, done = 0.0, 0
    t0 = time.perf_counter()
    for h in range(w.hq):
        for b in order:
            a, e = int(cu[b]), int(cu[b + 1])
            qs, ks, vs, dos = f(q[a:e, h]), f(k[a:e, h // g]), f(v[a:e, h // g]), f(do[a:e, h])
            for rows in A._slabs(e - a, 2048):
                A.attention_fwd_seq(qs, ks, vs, rows)
                A.attention_bwd_seq(qs, ks, vs, dos, rows)
            flops += 7.0 * float(e - a) ** 2 * w.head_dim
            done += 1
            if time.perf_counter() - t0 > budget_s:
                dt = time.perf_counter() - t0
                return flops, dt, f"{done} (sequence, head) problems, sequences <= 8192 tokens, longest first"
    dt = time.perf_counter() - t0
    return flops, dt, f"all {done} (sequence, head) problems with sequences <= 8192 tokens"


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    q, k, v, do = w.tensors()
    per_step = 4.0
    for _ in range(max(args.warmup, 0)):
        oracle_sample(w, q, k, v, do, per_step / 4)
    tot_f, tot_t, desc = 0.0, 0.0, ""
    for _ in range(args.steps):
        fl, dt, desc = oracle_sample(w, q, k, v, do, per_step)
        tot_f += fl
        tot_t += dt
    val = tot_f / tot_t / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOPS", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "tokens": w.total_tokens, "hq": w.hq, "hkv": w.hkv, "head_dim": w.head_dim,
                   "seed": w.seed},
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

    def stop(self, t_begin, t_end):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        rows = [s for t, s in self.samples if t_begin <= t <= t_end] or [s for _, s in self.samples[-3:]]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for nm, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------
def run_ours(args, w):
    import torch
    import torch.distributed as dist

    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import DeviceState

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    peaks = load_peaks()

    # each rank has its own batch: independent problems, no data-path collective
    from paper_2602_21788_b200 import ranks
    if world > 1:
        w = ranks.rank_workload(args.workload, args.seed, rank, world, args.max_heads)
    q, k, v, do = w.tensors()
    t_plan0 = time.perf_counter()
    ds = DeviceState(w, q, k, v, do, heads_per_pass=args.heads_per_pass or None)
    plan_ms = 1e3 * (time.perf_counter() - t_plan0)
    plan = ds.plan

    def step():
        ds.forward(merged=True)
        ds.backward()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    ds.check_status()
    plan.set_profiling(True)
    sampler = ClockSampler(local) if rank == 0 else None
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin = time.perf_counter()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    t_end = time.perf_counter()
    ms = ev0.elapsed_time(ev1)
    ds.check_status()
    clocks = sampler.stop(t_begin, t_end) if sampler else None
    kern = {}
    for kind, name in enumerate(["attn_fwd", "lse_merge", "bwd_preprocess", "attn_bwd", "dq_convert"]):
        n, kms = plan.kernel_ms(kind)
        kern[name] = {"launches": n, "mean_ms": kms}
    plan.set_profiling(False)

    ms, flops_total = ranks.aggregate(ms, w.flops_fwd_bwd(), "cuda")
    ms_per_step = ms / args.steps
    value = ranks.throughput_tflops(ms, args.steps, flops_total)

    # ---- end to end from pinned host buffers through the host entry point
    e2e = None
    if (rank == 0 or world > 1) and not args.no_e2e:
        T, hq, hkv, D = w.total_tokens, w.hq, w.hkv, w.head_dim
        pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
        hq_, hk_, hv_, hdo_ = pin(q), pin(k), pin(v), pin(do)
        ho = torch.empty((T, hq, D), dtype=torch.int16).pin_memory()
        hdq = torch.empty((T, hq, D), dtype=torch.int16).pin_memory()
        hdk = torch.empty((T, hkv, D), dtype=torch.int16).pin_memory()
        hdv = torch.empty((T, hkv, D), dtype=torch.int16).pin_memory()
        hlse = torch.empty((T, hq), dtype=torch.float32).pin_memory()
        nbytes = plan.host_workspace_bytes()
        del ds.o_part, ds.lse_part, ds.scratch
        torch.cuda.empty_cache()
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        st = torch.cuda.current_stream().cuda_stream
        call = lambda: fcp.fcp_attn_fwd_bwd_host(plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, nbytes, st)
        call()
        barrier()
        n_e2e = max(1, min(args.steps, 5))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_e2e):
            call()
        e1.record()
        barrier()
        e_ms = e0.elapsed_time(e1) / n_e2e
        e_ms, _ = ranks.aggregate(e_ms, 0.0, "cuda")
        h2d = 2 * (2 * T * hq * D + 2 * T * hkv * D)
        d2h = 2 * (2 * T * hq * D + 2 * T * hkv * D) + 4 * T * hq
        e2e = {"value": flops_total / (e_ms * 1e-3) / 1e12, "unit": "TFLOPS", "ms_per_step": e_ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (backward attention): algorithmic FLOPs = 2.5 x forward
    passes = -(-w.hq // ds.hpp)
    bwd_ms = kern["attn_bwd"]["mean_ms"]
    fwd_ms = kern["attn_fwd"]["mean_ms"] * passes      # all head passes of one step
    bwd_flops = 2.5 * w.flops_fwd()
    achieved = bwd_flops / (bwd_ms * 1e-3) / 1e12 if bwd_ms > 0 else None
    peak = peaks["bf16_sustained"]
    roofline = {"bound": "tensor", "kernel": "fcp_bwd_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None, "traffic": ncu_traffic(w, args),
                "peak_source": f"{peaks['source']} sustained bf16 (kernel timed inside a long step)",
                "fwd_kernel": {"achieved": w.flops_fwd() / (fwd_ms * 1e-3) / 1e12 if fwd_ms > 0 else None, "ms": fwd_ms},
                "frac_of_burst": achieved / peaks["bf16_burst"] if achieved else None,
                "frac_of_vendor_dense_bf16": achieved / NOMINAL_BF16_TFLOPS if achieved else None}
    R = plan.info("R")
    # the merge launch only covers Q chunks with two or more slots (the forward kernel writes the others
    # straight to the output): per token of such a chunk it reads every slot's partial row and writes one row
    mu = plan.table("merge_units")[: plan.info("n_merge_multi")]
    so = plan.table("slot_offset")
    n_slots = (so[mu[:, 2] + 1] - so[mu[:, 2]]).astype(np.int64)
    merge_tokens = int(mu[:, 1].sum())
    merge_bytes = int((mu[:, 1] * n_slots).sum()) * w.hq * (4 * w.head_dim + 4) + merge_tokens * w.hq * (2 * w.head_dim + 4)
    mms = kern["lse_merge"]["mean_ms"] * passes
    merge = {"bound": "hbm", "achieved_gbs": merge_bytes / (mms * 1e-3) / 1e9 if mms > 0 else None,
             "peak_gbs": peaks["hbm_gbs"], "ms": mms}

    # ---- CPU oracle on a bounded sample of the same workload (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        fl, dt, desc = oracle_sample(w, q, k, v, do, args.cpu_seconds)
        cpu = {"value": fl / dt / 1e12, "unit": "TFLOPS", "cores": blas_threads(), "kind": "oracle",
               "sample": f"{desc}; {dt:.1f} s of fp64 numpy"}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOPS", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": w.name, "tokens": w.total_tokens, "sequences": int(len(w.seqlens)), "hq": w.hq,
                   "hkv": w.hkv, "head_dim": w.head_dim, "seed": args.seed, "sum_len_sq": w.sum_sq,
                   "cp_degrees": sorted(set(int(x) for x in w.cp_degrees)), "partial_rows": R, "merged_tokens": merge_tokens,
                   "l2": "inputs larger than L2 (q alone is %d MB)" % (2 * w.total_tokens * w.hq * w.head_dim >> 20),
                   "flops": "7 * sum(L^2) * hq * head_dim per step", "plan_ms_host": plan_ms, "head_passes": passes},
        "frac_of_peak": {"measured_sustained": value / world / peaks["bf16_sustained"],
                         "measured_burst": value / world / peaks["bf16_burst"],
                         "vendor_dense_bf16": value / world / NOMINAL_BF16_TFLOPS},
        "kernels": kern, "roofline": roofline, "merge_roofline": merge, "cpu_baseline": cpu, "e2e": e2e,
        "gpu_launches": args.steps * (2 * passes + 3), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b_64k")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--heads-per-pass", type=int, default=0, help="query heads per forward pass (0 = all)")
    ap.add_argument("--max-heads", type=int, default=0,
                    help="keep at most this many query heads (query:KV ratio kept); a small case for profiler captures, "
                         "named <workload>_reduced in the output")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

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
