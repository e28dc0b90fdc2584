"""Profiled coefficients of the paper's compute-time model on this GPU (Sec. 4.3, Eq. 4).

Eq. 4 models the compute time of one rank of a CP group as  sum_k (alpha1 (1 + eta_k) L_k^2 + alpha2 L_k)
/ d + beta1.  Here all d virtual ranks of a sequence run in one grid on one GPU, so what can be timed
is the sum over the ranks:  T(L, d) = alpha1 L^2 + alpha2 L + beta1 d  (causal attention: eta = 0).
`measure_grid` times the whole hot path (forward over the plan with the merge on the fly, backward) through the C ABI on
batches of equal-length sequences that fill the GPU; `fit` solves the least-squares problem for
(alpha1, alpha2, beta1); `relative_errors` gives the estimation error the paper reports in its
cost-model table (predicted against measured time of mixed batches).  The fitted coefficients are
the `coeffs` input of `fcp.fcp_plan_strategy`.

    python -m paper_2602_21788_b200.costfit [--out FILE.md]      (needs a GPU)
"""
from __future__ import annotations

import argparse

import numpy as np

# Last fit on a B200 (32 query / 8 KV heads, head_dim 128), ms units; see `main` for how it is taken.
B200_COEFFS = dict(alpha1=2.976196e-08, alpha2=1.734399e-05, beta1=0.0)   # beta1 fitted at -3e-5 ms: zero within noise


def design_row(seqlens, cp_degrees):
    """Regressors of one batch: (sum L^2, sum L, sum d)."""
    L = np.asarray(seqlens, dtype=np.float64)
    d = np.asarray(cp_degrees, dtype=np.float64)
    return np.array([np.sum(L * L), np.sum(L), np.sum(d)])


def fit(rows, times_ms):
    """Least squares for T = alpha1 * sum L^2 + alpha2 * sum L + beta1 * sum d, every equation weighted by
    1 / T so that the residual is the relative error.  Returns dict(alpha1, alpha2, beta1) in ms."""
    X = np.asarray(rows, dtype=np.float64)
    y = np.asarray(times_ms, dtype=np.float64)
    wgt = 1.0 / y
    sol, *_ = np.linalg.lstsq(X * wgt[:, None], y * wgt, rcond=None)
    return dict(alpha1=float(sol[0]), alpha2=float(sol[1]), beta1=float(sol[2]))


def predict(coeffs, seqlens, cp_degrees) -> float:
    r = design_row(seqlens, cp_degrees)
    return float(coeffs["alpha1"] * r[0] + coeffs["alpha2"] * r[1] + coeffs["beta1"] * r[2])


def relative_errors(coeffs, batches, times_ms):
    """|predicted - measured| / measured for each (seqlens, cp_degrees) batch."""
    return np.array([abs(predict(coeffs, l, d) - t) / t for (l, d), t in zip(batches, times_ms)])


# ------------------------------------------------------------------------------------------------
# measurement (GPU)
# ------------------------------------------------------------------------------------------------
def time_batch(seqlens, cp_degrees, hq, hkv, head_dim, reps=5, warmup=2, seed=0) -> float:
    """Median ms of fused forward + backward for one synthetic batch (inputs resident on the GPU)."""
    import torch

    from . import synth
    from .runner import DeviceState

    w = synth.Workload(name="costfit", seed=seed, seqlens=np.asarray(seqlens, dtype=np.int32),
                       cp_degrees=np.asarray(cp_degrees, dtype=np.int32), hq=hq, hkv=hkv, head_dim=head_dim)
    T = w.total_tokens
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)

    def draw(h):   # N(0,1) rounded to bf16, as in the workloads (values do not change the timing)
        return torch.randn((T, h, head_dim), device="cuda", generator=g, dtype=torch.bfloat16)

    ds = DeviceState(w, draw(hq), draw(hkv), draw(hkv), draw(hq), partials=False)
    for _ in range(warmup):
        ds.forward_fused()
        ds.backward()
    torch.cuda.synchronize()
    out = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ds.forward_fused()
        ds.backward()
        e1.record()
        torch.cuda.synchronize()
        out.append(e0.elapsed_time(e1))
    ds.check_status()
    return float(np.median(out))


def measure_grid(lengths, degrees, hq, hkv, head_dim, tokens=65536):
    """Batches of tokens // L sequences of length L, all at degree d.  Returns (rows, times, labels)."""
    rows, times, labels = [], [], []
    for L in lengths:
        n = max(1, tokens // L)
        for d in degrees:
            lens, degs = [L] * n, [d] * n
            rows.append(design_row(lens, degs))
            times.append(time_batch(lens, degs, hq, hkv, head_dim))
            labels.append((L, d, n))
    return rows, times, labels


def main():
    from . import fcp, synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--out", default="")
    args = ap.parse_args()
    hq, hkv, D = 32, 8, 128
    lengths, degrees = [1024, 2048, 4096, 8192, 16384, 32768], [1, 2, 3, 4, 6, 8]
    rows, times, labels = measure_grid(lengths, degrees, hq, hkv, D)
    c = fit(rows, times)
    grid_err = np.array([abs(float(np.dot(r, [c["alpha1"], c["alpha2"], c["beta1"]])) - t) / t for r, t in zip(rows, times)])
    # held-out mixed batches: the bench workload's recipe with other seeds
    batches, btimes = [], []
    for seed in range(5):
        w = synth.make_workload("llama8b_64k", seed=seed)
        batches.append((w.seqlens, w.cp_degrees))
        btimes.append(time_batch(w.seqlens, w.cp_degrees, hq, hkv, D, seed=seed))
    errs = relative_errors(c, batches, btimes)
    # the fitted coefficients drive the strategy search (no communication term on one GPU)
    w = synth.make_workload("llama8b_64k", seed=0)
    plan = fcp.fcp_plan_strategy(w.seqlens, N=16, E=8192.0, M_token=1.0, M_ms=0.0,
                                 coeffs=dict(alpha1=c["alpha1"], alpha2=c["alpha2"], alpha3=0.0, beta1=c["beta1"], beta2=0.0, v=1.0))
    lines = ["# Cost-model coefficients of Eq. 4 fitted on one B200 (`python -m paper_2602_21788_b200.costfit`)", "",
             f"Shape: {hq} query / {hkv} KV heads, head_dim {D}, causal, bf16; batches of 65536 tokens of equal-length sequences;",
             "time = forward over the plan with the merge on the fly + backward (median of 5, CUDA events).", "",
             f"alpha1 = {c['alpha1']:.6e} ms/token^2, alpha2 = {c['alpha2']:.6e} ms/token, beta1 = {c['beta1']:.6e} ms per virtual rank", "",
             f"Fit residual over the {len(times)} grid points: mean {100 * grid_err.mean():.2f} %, max {100 * grid_err.max():.2f} %.",
             "Estimation error on held-out mixed batches (`llama8b_64k` recipe, seeds 0-4): "
             + ", ".join(f"{100 * e:.2f} %" for e in errs) + f" (mean {100 * errs.mean():.2f} %).", "",
             "| L | d | sequences | measured ms | predicted ms |", "|---|---|---|---|---|"]
    for (L, d, n), r, t in zip(labels, rows, times):
        lines.append(f"| {L} | {d} | {n} | {t:.3f} | {float(np.dot(r, [c['alpha1'], c['alpha2'], c['beta1']])):.3f} |")
    lines += ["", f"Strategy search with these coefficients on `llama8b_64k` seed 0 (N = 16 ranks, E = 8192 tokens per rank): "
              f"{plan['n_groups']} groups, degrees {sorted(set(int(x) for x in plan['cp_degree']))}, makespan {plan['makespan']:.3f} ms."]
    text = "\n".join(lines) + "\n"
    print(text)
    if args.out:
        with open(args.out, "w") as f:
            f.write(text)


if __name__ == "__main__":
    main()
