"""GPU parity: the CUDA path (through the C ABI) against the fp64 oracle on the same seeded inputs.

Tolerances (stated for bf16 inputs with fp32 accumulation):
  O    max abs <= 1e-2, mean abs <= 1e-3     (checked on the fp32 output; the bf16 copy of O is
                                             allowed its own rounding, half an ulp = 2^-8 * |o|, on top)
  LSE  max abs <= 1e-3
  dQ, dK, dV   relative Frobenius error <= 2e-2
  plan tables  bit-exact (tests/test_host_plan.py, host only)
"""
import math

import numpy as np
import pytest

from oracle import attention_ref as A
from oracle import plan_ref as P
from paper_2602_21788_b200 import build, synth

pytestmark = pytest.mark.gpu

torch = pytest.importorskip("torch")

O_MAX, O_MEAN, LSE_MAX, GRAD_REL = 1e-2, 1e-3, 1e-3, 2e-2
f64 = synth.bf16_bits_to_f64


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    build.build()
    torch.cuda.set_device(0)


def _wl(lens, degs, hq, hkv, D, seed=0):
    return synth.Workload(name="case", seed=seed, seqlens=np.asarray(lens, np.int32),
                          cp_degrees=np.asarray(degs, np.int32), hq=hq, hkv=hkv, head_dim=D)


def _grad_ok(got, ref):
    """Relative Frobenius error <= 2e-2.  Only where the exact gradient is identically zero (a batch of
    single-token sequences has dq = dk = 0) is the ratio undefined; an absolute bound is used there."""
    err = np.linalg.norm(np.asarray(got, dtype=np.float64) - ref)
    nref = np.linalg.norm(ref)
    if nref == 0.0:
        return err <= 1e-4 * math.sqrt(ref.size), err
    return err <= GRAD_REL * nref, err / nref


def _check_full(w, heads_per_pass=None, bwd=True, check_partials=False):
    from paper_2602_21788_b200.runner import run_fwd_bwd
    q, k, v, do = w.tensors()
    res = run_fwd_bwd(w, q, k, v, do if bwd else None, heads_per_pass=heads_per_pass, keep_partials=check_partials)
    qf, kf, vf, dof = f64(q), f64(k), f64(v), f64(do)
    o_ref, lse_ref = A.attention_fwd_packed(qf, kf, vf, w.cu_seqlens)
    e = np.abs(res["o_f32"] - o_ref)
    assert e.max() <= O_MAX and e.mean() <= O_MEAN, (e.max(), e.mean())
    eb = np.abs(res["o"] - o_ref)
    assert np.all(eb <= O_MAX + np.abs(o_ref) * 2.0 ** -8) and eb.mean() <= O_MEAN, (eb.max(), eb.mean())
    assert np.abs(res["lse"] - lse_ref).max() <= LSE_MAX
    if check_partials:
        _check_partials(w, res, qf, kf, vf)
    if bwd:
        dq_ref, dk_ref, dv_ref = A.attention_bwd_packed(qf, kf, vf, dof, w.cu_seqlens)
        for name, ref in (("dq", dq_ref), ("dk", dk_ref), ("dv", dv_ref)):
            ok, rel = _grad_ok(res[name], ref)
            assert ok, (name, rel)
            assert np.isfinite(res[name]).all()
    return res


def _check_partials(w, res, qf, kf, vf):
    """Every item's normalised partial and its LSE against the oracle's partial over the same KV ranges."""
    lens, degs = w.seqlens.tolist(), w.cp_degrees.tolist()
    pl = P.plan_blocks(lens, degs)
    cb, co = pl["chunk_bounds"], pl["chunk_offset"]
    g = w.hq // w.hkv
    for (b, r, s, qc, slot, row0, n, first) in pl["items"]:
        t0 = cb[co[b]]
        qr = (cb[co[b] + qc] - t0, cb[co[b] + qc + 1] - t0)
        ranges = [(cb[co[b] + kc] - t0, cb[co[b] + kc + 1] - t0) for (_, _, _, _, kc, _) in pl["pairs"][first:first + n]]
        sl = slice(t0, t0 + lens[b])
        for h in range(w.hq):
            op, lp = A.partial_attention(qf[sl, h], kf[sl, h // g], vf[sl, h // g], qr, ranges)
            rows = slice(row0, row0 + qr[1] - qr[0])
            assert np.abs(res["o_partial"][rows, h] - op).max() <= O_MAX
            assert np.abs(res["lse_partial"][rows, h] - lp).max() <= LSE_MAX


EDGE_CASES = [
    # lens, degs, hq, hkv, D
    ([1], [1], 1, 1, 128),                    # single token
    ([1, 2, 3], [3, 2, 4], 2, 1, 64),         # L < 2d: empty chunks are dropped
    ([128], [1], 1, 1, 128),                  # exactly one tile
    ([129], [1], 2, 2, 64),                   # one row into the second tile
    ([256, 257, 255], [1, 1, 1], 2, 1, 128),  # around the two-tile unit
    ([100], [8], 4, 4, 64),                   # chunks shorter than a tile (6-7 tokens)
    ([1000], [7], 8, 1, 128),                 # non-power-of-two degree, GQA 8:1, L % 14 != 0
    ([1031], [5], 4, 2, 128),                 # prime length
    ([777, 64, 1500], [3, 1, 6], 4, 4, 64),   # hq == hkv
    ([2048], [8], 2, 1, 128),                 # d = 8, chunk = one tile exactly
    ([3000], [1], 2, 1, 128),                 # d = 1: plain varlen causal attention
    ([513], [64], 1, 1, 64),                  # largest supported degree
]


@pytest.mark.parametrize("lens,degs,hq,hkv,D", EDGE_CASES)
def test_edge_shapes(lens, degs, hq, hkv, D):
    _check_full(_wl(lens, degs, hq, hkv, D, seed=3), check_partials=True)


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_tiny_workload(seed):
    _check_full(synth.make_workload("tiny", seed), check_partials=True)


@pytest.mark.parametrize("name", ["llama8b_64k", "longtail_256k", "bimodal_128k", "extreme_512k"])
def test_reduced_workloads(name):
    """Same generators and degrees, lengths / 16, at most 8 query heads: the oracle runs in full."""
    w = synth.reduced(synth.make_workload(name, 0))
    _check_full(w)


def _check_fused(w, heads_per_pass=None):
    """fcp_attn_fwd_fused (merge on the fly, no partials) against the fp64 oracle, and against the
    partial-producing path of the same plan."""
    from paper_2602_21788_b200.runner import run_fwd_bwd
    q, k, v = w.tensors(with_do=False)
    res = run_fwd_bwd(w, q, k, v, None, heads_per_pass=heads_per_pass, fused=True)
    o_ref, lse_ref = A.attention_fwd_packed(f64(q), f64(k), f64(v), w.cu_seqlens)
    e = np.abs(res["o_f32"] - o_ref)
    assert e.max() <= O_MAX and e.mean() <= O_MEAN, (e.max(), e.mean())
    eb = np.abs(res["o"] - o_ref)
    assert np.all(eb <= O_MAX + np.abs(o_ref) * 2.0 ** -8) and eb.mean() <= O_MEAN, (eb.max(), eb.mean())
    assert np.abs(res["lse"] - lse_ref).max() <= LSE_MAX
    part = run_fwd_bwd(w, q, k, v, None, heads_per_pass=heads_per_pass)
    assert np.abs(part["o_f32"] - res["o_f32"]).max() <= O_MAX and np.abs(part["lse"] - res["lse"]).max() <= LSE_MAX


@pytest.mark.parametrize("lens,degs,hq,hkv,D", EDGE_CASES)
def test_fused_forward_edge_shapes(lens, degs, hq, hkv, D):
    _check_fused(_wl(lens, degs, hq, hkv, D, seed=3))


@pytest.mark.parametrize("name", ["tiny", "llama8b_64k", "longtail_256k", "bimodal_128k", "extreme_512k"])
def test_fused_forward_workloads(name):
    w = synth.make_workload(name, 0)
    _check_fused(w if name == "tiny" else synth.reduced(w), heads_per_pass=3 if name == "bimodal_128k" else None)


def test_fused_forward_is_bitwise_reproducible_and_independent_of_the_degrees():
    """One CTA sweeps a row's keys in position order whatever the plan's degrees, so the fused forward of
    the configured degrees and of all d = 1 give the same bits."""
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = synth.reduced(synth.make_workload("bimodal_128k", 1), len_div=8)
    q, k, v = w.tensors(with_do=False)
    a = run_fwd_bwd(w, q, k, v, None, fused=True)
    b = run_fwd_bwd(w, q, k, v, None, fused=True)
    assert np.array_equal(a["o"], b["o"]) and np.array_equal(a["lse"], b["lse"])
    w1 = _wl(w.seqlens, np.ones_like(w.cp_degrees), w.hq, w.hkv, w.head_dim, seed=w.seed)
    c = run_fwd_bwd(w1, q, k, v, None, fused=True)
    assert np.array_equal(a["o"], c["o"]) and np.array_equal(a["lse"], c["lse"])


def test_backward_in_kv_head_passes_gives_the_same_result():
    """fcp_attn_bwd_heads over disjoint KV-head ranges == fcp_attn_bwd over all heads: dK/dV bit for bit
    (no sum crosses KV heads, no atomics), dQ to the order of its fp32 reductions."""
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = _wl([700, 300, 129], [3, 2, 1], 8, 4, 128, seed=5)
    q, k, v, do = w.tensors()
    a = run_fwd_bwd(w, q, k, v, do)
    b = run_fwd_bwd(w, q, k, v, do, kv_heads_per_bwd_pass=3)      # passes of 3 + 1 KV heads
    assert np.array_equal(a["dk"], b["dk"]) and np.array_equal(a["dv"], b["dv"])
    assert np.linalg.norm(a["dq"] - b["dq"]) <= 1e-2 * np.linalg.norm(a["dq"])
    dq_ref, dk_ref, dv_ref = A.attention_bwd_packed(f64(q), f64(k), f64(v), f64(do), w.cu_seqlens)
    for name, ref in (("dq", dq_ref), ("dk", dk_ref), ("dv", dv_ref)):
        ok, rel = _grad_ok(b[name], ref)
        assert ok, (name, rel)
    ds = b["state"]
    assert ds.plan.bwd_scratch_bytes(3) < ds.plan.bwd_scratch_bytes(4) == ds.plan.workspace_bytes(1)[2]
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_attn_bwd_heads(ds.plan, ds.q, ds.k, ds.v, ds.o, ds.do, ds.lse, 3, 2, ds.dq, ds.dk, ds.dv, ds.scratch,
                               ds.scratch_bytes, 0)
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_head_passes_give_the_same_result():
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = _wl([700, 300], [3, 2], 8, 2, 128, seed=5)
    q, k, v, do = w.tensors()
    a = run_fwd_bwd(w, q, k, v, do)
    b = run_fwd_bwd(w, q, k, v, do, heads_per_pass=3)
    assert np.array_equal(a["o"], b["o"]) and np.array_equal(a["lse"], b["lse"])


MERGED_CASES = [
    ([700, 300], [3, 2], 8, 2, 128, None),       # mixed single-slot (first chunks) and multi-slot chunks
    ([3000, 129, 1], [1, 1, 1], 2, 1, 128, None),  # degree 1 everywhere: nothing left to merge
    ([777, 64, 1500], [3, 1, 6], 4, 4, 64, 3),   # head_dim 64, head passes
    ([1000], [7], 8, 1, 128, None),
]


@pytest.mark.parametrize("lens,degs,hq,hkv,D,hpp", MERGED_CASES)
def test_merged_forward_is_bit_identical_to_forward_plus_merge(lens, degs, hq, hkv, D, hpp):
    """fcp_attn_fwd_merged writes single-slot chunks straight to o / lse: same bits as the two calls,
    and within the stated tolerances of the fp64 oracle."""
    import torch
    from paper_2602_21788_b200.runner import DeviceState, bf16_dev_to_f64
    w = _wl(lens, degs, hq, hkv, D, seed=11)
    q, k, v = w.tensors(with_do=False)
    ds = DeviceState(w, q, k, v, None, heads_per_pass=hpp)
    ds.forward()
    torch.cuda.synchronize()
    o_a, lse_a = ds.o.clone(), ds.lse.clone()
    ds.o.fill_(float("nan"))
    ds.lse.fill_(float("nan"))
    ds.o_part.fill_(float("nan"))
    ds.lse_part.fill_(float("nan"))
    ds.forward(merged=True)
    torch.cuda.synchronize()
    ds.check_status()
    assert torch.equal(ds.o.view(torch.int16), o_a.view(torch.int16))
    assert torch.equal(ds.lse, lse_a)
    f = synth.bf16_bits_to_f64
    o_ref, lse_ref = A.attention_fwd_packed(f(q), f(k), f(v), w.cu_seqlens)
    assert np.abs(ds.lse.cpu().numpy() - lse_ref).max() <= 1e-3
    err = np.abs(bf16_dev_to_f64(ds.o) - o_ref)
    assert err.mean() <= 1e-3 and (err <= 1e-2 + 2.0 ** -8 * np.abs(o_ref)).all()


def test_forward_and_merge_are_bitwise_reproducible_and_backward_within_tolerance():
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = synth.make_workload("tiny", 1)
    q, k, v, do = w.tensors()
    a = run_fwd_bwd(w, q, k, v, do)
    b = run_fwd_bwd(w, q, k, v, do)
    assert np.array_equal(a["o"], b["o"]) and np.array_equal(a["lse"], b["lse"]) and np.array_equal(a["o_f32"], b["o_f32"])
    assert np.array_equal(a["dk"], b["dk"]) and np.array_equal(a["dv"], b["dv"])   # no atomics on dK/dV
    assert np.linalg.norm(a["dq"] - b["dq"]) <= 1e-2 * np.linalg.norm(a["dq"])       # fp32 atomics: order varies


def test_chunked_plan_agrees_with_degree_one_plan():
    """Self-consistency without the oracle: the configured degrees vs all d = 1."""
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = synth.reduced(synth.make_workload("bimodal_128k", 1), len_div=8)
    q, k, v, do = w.tensors()
    a = run_fwd_bwd(w, q, k, v, do)
    w1 = _wl(w.seqlens, np.ones_like(w.cp_degrees), w.hq, w.hkv, w.head_dim, seed=w.seed)
    w1.name = w.name
    b = run_fwd_bwd(w1, q, k, v, do)
    assert np.abs(a["o_f32"] - b["o_f32"]).max() <= O_MAX and np.abs(a["lse"] - b["lse"]).max() <= LSE_MAX
    for n in ("dq", "dk", "dv"):
        assert np.linalg.norm(a[n] - b[n]) <= GRAD_REL * np.linalg.norm(b[n])


@pytest.mark.parametrize("lens,degs", [
    ([900, 130], [3, 1]),                                              # one sequence group
    ([2100, 1800, 2500, 900, 3000, 1500, 2048, 4097, 700, 2600, 1900, 3100],
     [1, 2, 1, 1, 3, 1, 2, 1, 1, 2, 1, 3]),                           # three groups, pipelined copies and kernels
])
def test_host_buffer_entry_point_matches_device_path(lens, degs):
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = _wl(lens, degs, 4, 2, 128, seed=7)
    q, k, v, do = w.tensors()
    ref = run_fwd_bwd(w, q, k, v, do, fused=True)      # the host entry point runs the fused forward
    plan = ref["state"].plan
    T, hq, hkv, D = w.total_tokens, w.hq, w.hkv, w.head_dim
    pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
    hq_, hk_, hv_, hdo_ = pin(q), pin(k), pin(v), pin(do)
    ho = torch.empty((T, hq, D), dtype=torch.int16).pin_memory()
    hdq = torch.empty((T, hq, D), dtype=torch.int16).pin_memory()
    hdk = torch.empty((T, hkv, D), dtype=torch.int16).pin_memory()
    hdv = torch.empty((T, hkv, D), dtype=torch.int16).pin_memory()
    hlse = torch.empty((T, hq), dtype=torch.float32).pin_memory()
    nbytes = plan.host_workspace_bytes()
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    fcp.fcp_attn_fwd_bwd_host(plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, nbytes,
                              torch.cuda.current_stream().cuda_stream)
    back = lambda t: f64(t.numpy().view(np.uint16))
    assert np.array_equal(back(ho), ref["o"]) and np.array_equal(hlse.numpy(), ref["lse"])
    assert np.array_equal(back(hdk), ref["dk"]) and np.array_equal(back(hdv), ref["dv"])
    assert np.linalg.norm(back(hdq) - ref["dq"]) <= 1e-2 * np.linalg.norm(ref["dq"])
    assert plan.device_status()[0] == 0
    # a second call reuses the sequence groups built by the first
    ho.zero_(); hdk.zero_()
    fcp.fcp_attn_fwd_bwd_host(plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, nbytes,
                              torch.cuda.current_stream().cuda_stream)
    assert np.array_equal(back(ho), ref["o"]) and np.array_equal(back(hdk), ref["dk"])
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_attn_fwd_bwd_host(plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, 1024, 0)
    assert e.value.status == fcp.FCP_ERR_WORKSPACE


def test_host_buffer_entry_point_pipelines_a_long_sequence_by_kv_heads():
    """A group whose q slice exceeds 512 MB is also cut into passes over whole KV heads (strided 2-D copies, the
    forward by head range, the backward by KV-head range): same results as the device path, bit for bit where
    that path is deterministic."""
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import DeviceState
    w = _wl([61440, 4096], [5, 1], 40, 8, 128, seed=8)
    q, k, v, do = w.device_tensors()
    ds = DeviceState(w, q, k, v, do, partials=False)
    ds.forward_fused()
    ds.backward()
    torch.cuda.synchronize()
    ds.check_status()
    T, hq, hkv, D = w.total_tokens, w.hq, w.hkv, w.head_dim
    pin = lambda t: t.view(torch.int16).cpu().pin_memory()
    hq_, hk_, hv_, hdo_ = pin(q), pin(k), pin(v), pin(do)
    ho = torch.zeros((T, hq, D), dtype=torch.int16).pin_memory()
    hdq = torch.zeros((T, hq, D), dtype=torch.int16).pin_memory()
    hdk = torch.zeros((T, hkv, D), dtype=torch.int16).pin_memory()
    hdv = torch.zeros((T, hkv, D), dtype=torch.int16).pin_memory()
    hlse = torch.zeros((T, hq), dtype=torch.float32).pin_memory()
    nbytes = ds.plan.host_workspace_bytes()
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    fcp.fcp_attn_fwd_bwd_host(ds.plan, hq_, hk_, hv_, hdo_, ho, hlse, hdq, hdk, hdv, ws, nbytes,
                              torch.cuda.current_stream().cuda_stream)
    assert ds.plan.device_status()[0] == 0
    assert torch.equal(ho, ds.o.view(torch.int16).cpu()) and torch.equal(hlse, ds.lse.cpu())
    assert torch.equal(hdk, ds.dk.view(torch.int16).cpu()) and torch.equal(hdv, ds.dv.view(torch.int16).cpu())
    a, b = hdq.view(torch.bfloat16).float(), ds.dq.float().cpu()
    assert torch.isfinite(a).all() and (a - b).norm() <= 1e-2 * b.norm()


def test_workspace_too_small_is_reported():
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import DeviceState
    w = _wl([300], [1], 2, 1, 128)
    q, k, v, do = w.tensors()
    ds = DeviceState(w, q, k, v, do)
    ds.forward()
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_attn_bwd(ds.plan, ds.q, ds.k, ds.v, ds.o, ds.do, ds.lse, ds.dq, ds.dk, ds.dv, ds.scratch, 16, 0)
    assert e.value.status == fcp.FCP_ERR_WORKSPACE
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_attn_fwd(ds.plan, ds.q, ds.k, ds.v, ds.o_part, ds.lse_part, 1, 2, 0)   # heads [1,3) of 2
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    torch.cuda.synchronize()


# ----------------------------------------------------------------------------------------------
# Full-size workloads: results stay on the device, the oracle evaluates sampled outputs one by one.
# ----------------------------------------------------------------------------------------------
def _bits64(t):
    """bf16 device tensor (any slice) -> float64 host array, exactly."""
    return t.float().cpu().numpy().astype(np.float64)


def _sampled_check(w, n_rows=96, n_tail=24, seed=0, heads_per_pass=None, device_inputs=False):
    """Runs the partial path (forward + merge), the merged call, the fused forward and the backward at full
    size and compares sampled outputs with the oracle's per-row forms.  With `device_inputs` the tensors
    are drawn on the device (host draws of billions of values take minutes) and only the slices the
    oracle needs are brought to the host."""
    from paper_2602_21788_b200.runner import DeviceState
    if device_inputs:
        q, k, v, do = w.device_tensors()
    else:
        q, k, v, do = (torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16) for a in w.tensors())
    big = w.total_tokens * w.hq * w.head_dim > (1 << 31)
    ds = DeviceState(w, q, k, v, do, heads_per_pass=heads_per_pass, want_o_f32=not big)
    ds.forward()
    torch.cuda.synchronize()
    o_two_calls, lse_two_calls = ds.o.clone(), ds.lse.clone()
    o_f32 = ds.o_f32.clone() if ds.o_f32 is not None else None
    # the merged call (single-slot chunks straight to the output) gives the same bits
    ds.o.zero_()
    ds.lse.zero_()
    ds.forward(merged=True)
    torch.cuda.synchronize()
    ds.check_status()
    assert torch.equal(ds.o.view(torch.int16), o_two_calls.view(torch.int16)) and torch.equal(ds.lse, lse_two_calls)
    # the fused forward (the call the benchmark times) agrees with the partial path to rounding
    del ds.o_part, ds.lse_part
    ds.o.zero_()
    ds.lse.zero_()
    ds.forward_fused()
    torch.cuda.synchronize()
    ds.check_status()
    assert (ds.lse - lse_two_calls).abs().max().item() <= LSE_MAX
    T = w.total_tokens
    for t0 in range(0, T, 1 << 15):      # blockwise: the tensors may hold billions of elements
        a_, b_ = ds.o[t0:t0 + (1 << 15)].float(), o_two_calls[t0:t0 + (1 << 15)].float()
        assert ((a_ - b_).abs() <= O_MAX + 2.0 ** -7 * b_.abs()).all()
    del o_two_calls, lse_two_calls
    ds.backward()
    torch.cuda.synchronize()
    ds.check_status()

    rng = np.random.default_rng(seed)
    cu = w.cu_seqlens
    g = w.hq // w.hkv
    D = w.head_dim
    longest = int(np.argmax(w.seqlens))
    kv_cache = {}

    def kv_of(b, hk):
        """K and V of one (sequence, KV head) as float64, cached (the long sequence is fetched once per head)."""
        if (b, hk) not in kv_cache:
            if len(kv_cache) >= 3:
                kv_cache.pop(next(iter(kv_cache)))
            t0, t1 = int(cu[b]), int(cu[b + 1])
            kv_cache[(b, hk)] = (_bits64(k[t0:t1, hk]), _bits64(v[t0:t1, hk]))
        return kv_cache[(b, hk)]

    # forward rows and dQ rows: random (sequence, token, head), biased to the longest sequence, to the last
    # tokens of a sequence and to the edges of its chunks; few distinct KV heads so that the cache works
    heads = sorted(int(h) for h in rng.choice(w.hq, size=min(w.hq, 4), replace=False))
    o_err, l_err, dq_num, dq_den = [], [], 0.0, 0.0
    for n in range(n_rows):
        b = longest if n % 3 == 0 else int(rng.integers(len(w.seqlens)))
        L = int(w.seqlens[b])
        d = int(w.cp_degrees[b])
        if n % 4 == 0:
            i = L - 1 - int(rng.integers(min(L, 300)))
        elif n % 4 == 1 and d > 1:
            c = int(rng.integers(1, 2 * d))
            i = min(L - 1, max(0, c * L // (2 * d) + int(rng.integers(-2, 2))))     # around a chunk edge
        else:
            i = int(rng.integers(L))
        h = heads[n % len(heads)]
        t0 = int(cu[b])
        ks, vs = kv_of(b, h // g)
        qi, doi = _bits64(q[t0 + i, h]), _bits64(do[t0 + i, h])
        o_ref, lse_ref = A.attention_row(qi, ks[:i + 1], vs[:i + 1], i)
        dq_ref, _, _ = A.attention_row_grad(qi, ks[:i + 1], vs[:i + 1], doi, i)
        if o_f32 is not None:
            o_err.append(np.abs(o_f32[t0 + i, h].cpu().numpy().astype(np.float64) - o_ref))
        else:
            eb = np.abs(_bits64(ds.o[t0 + i, h]) - o_ref)
            assert np.all(eb <= O_MAX + np.abs(o_ref) * 2.0 ** -8)
            o_err.append(eb)
        l_err.append(abs(float(ds.lse[t0 + i, h]) - lse_ref))
        dq_num += np.sum((_bits64(ds.dq[t0 + i, h]) - dq_ref) ** 2)
        dq_den += np.sum(dq_ref ** 2)
    o_err = np.concatenate(o_err)
    assert (o_f32 is None or o_err.max() <= O_MAX) and o_err.mean() <= O_MEAN, (o_err.max(), o_err.mean())
    assert max(l_err) <= LSE_MAX
    assert math.sqrt(dq_num / dq_den) <= GRAD_REL
    # dK/dV columns: the last n_tail tokens of the longest sequence (every later row of every head of
    # the group contributes), one KV head
    b, L, t0 = longest, int(w.seqlens[longest]), int(cu[longest])
    hk = heads[0] // g
    ks, vs = kv_of(b, hk)
    j0 = L - n_tail
    dk_ref = np.zeros((n_tail, D)); dv_ref = np.zeros((n_tail, D))
    for h in range(hk * g, hk * g + g):
        qt, dot = _bits64(q[t0 + j0:t0 + L, h]), _bits64(do[t0 + j0:t0 + L, h])
        for i in range(j0, L):
            qi, doi = qt[i - j0], dot[i - j0]
            _, p, dsr = A.attention_row_grad(qi, ks[:i + 1], vs[:i + 1], doi, i)
            dv_ref[: i - j0 + 1] += p[j0:, None] * doi[None, :]
            dk_ref[: i - j0 + 1] += dsr[j0:, None] * qi[None, :] / math.sqrt(D)
    for name, ref, got in (("dk", dk_ref, ds.dk), ("dv", dv_ref, ds.dv)):
        assert np.linalg.norm(_bits64(got[t0 + j0:t0 + L, hk]) - ref) <= GRAD_REL * np.linalg.norm(ref), name
    kv_cache.clear()
    # two whole short sequences in full (all heads): every dK/dV column of them, every row
    short = [b for b in range(len(w.seqlens)) if w.seqlens[b] <= 1536][:2]
    for b in short:
        t0, t1 = int(cu[b]), int(cu[b + 1])
        sub_cu = np.array([0, t1 - t0])
        qf, kf, vf, dof = _bits64(q[t0:t1]), _bits64(k[t0:t1]), _bits64(v[t0:t1]), _bits64(do[t0:t1])
        o_ref, lse_ref = A.attention_fwd_packed(qf, kf, vf, sub_cu)
        dq_ref, dk_ref, dv_ref = A.attention_bwd_packed(qf, kf, vf, dof, sub_cu)
        e = np.abs(_bits64(ds.o[t0:t1]) - o_ref)
        assert np.all(e <= O_MAX + np.abs(o_ref) * 2.0 ** -8) and e.mean() <= O_MEAN
        assert np.abs(ds.lse[t0:t1].cpu().numpy() - lse_ref).max() <= LSE_MAX
        for name, ref, got in (("dq", dq_ref, ds.dq), ("dk", dk_ref, ds.dk), ("dv", dv_ref, ds.dv)):
            assert np.linalg.norm(_bits64(got[t0:t1]) - ref) <= GRAD_REL * np.linalg.norm(ref), name
    # properties that hold at any size
    for t in (ds.o, ds.lse, ds.dq, ds.dk, ds.dv):
        for t0 in range(0, T, 1 << 15):
            assert torch.isfinite(t[t0:t0 + (1 << 15)]).all()
    first = torch.from_numpy(cu[:-1].astype(np.int64)).cuda()
    assert torch.equal(ds.o[first].view(torch.int16),
                       v[first].repeat_interleave(g, dim=1).view(torch.int16))   # first token attends to itself only


def test_full_size_llama8b_64k_sampled():
    """All heads in one pass; inputs from the host generator."""
    _sampled_check(synth.make_workload("llama8b_64k", 0))


@pytest.mark.slow
def test_full_size_bimodal_128k_sampled():
    _sampled_check(synth.make_workload("bimodal_128k", 0), n_rows=48, n_tail=8, device_inputs=True)


@pytest.mark.slow
def test_full_size_longtail_256k_sampled():
    """One 128K-token sequence at degree 7 plus short ones, 40 query heads on 8 KV heads."""
    _sampled_check(synth.make_workload("longtail_256k", 0), n_rows=48, n_tail=8, device_inputs=True)


@pytest.mark.slow
def test_full_size_extreme_512k_all_heads_sampled():
    """The benchmark's configuration at its real shape: 512K tokens (one 384K sequence at degree 7), all 64
    query heads on 8 KV heads, so T*hq*D = 2^32 elements per tensor (element offsets beyond 32 bits), the
    partial path in 4 head passes of 16, the fused forward and the backward in one pass."""
    w = synth.make_workload("extreme_512k", 0)
    assert w.total_tokens * w.hq * w.head_dim >= 1 << 32
    _sampled_check(w, n_rows=32, n_tail=4, heads_per_pass=16, device_inputs=True)


# ----------------------------------------------------------------------------------------------
# dK/dV columns at chunk boundaries in the middle of a sequence, non-power-of-two degrees
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("L,d", [(12000, 3), (14000, 5), (15000, 6), (16000, 7)])
def test_dk_dv_columns_at_chunk_boundaries_mid_sequence(L, d):
    """Columns right at the chunk bounds b_c = floor(c*L/(2d)) receive contributions from the Q rows of every
    later chunk, across all ring steps; the oracle's slab form still gives the full dk/dv at this length."""
    from paper_2602_21788_b200.runner import run_fwd_bwd
    w = _wl([L], [d], 2, 1, 128, seed=13)
    q, k, v, do = w.tensors()
    res = run_fwd_bwd(w, q, k, v, do)
    qf, kf, vf, dof = f64(q), f64(k), f64(v), f64(do)
    dq_ref, dk_ref, dv_ref = A.attention_bwd_packed(qf, kf, vf, dof, w.cu_seqlens)
    cols = sorted({min(L - 1, max(0, c * L // (2 * d) + o)) for c in range(1, 2 * d) for o in (-2, -1, 0, 1)})
    assert len(cols) >= 4 * (2 * d - 1) - 2
    for name, ref in (("dk", dk_ref), ("dv", dv_ref), ("dq", dq_ref)):
        ok, rel = _grad_ok(res[name], ref)
        assert ok, (name, rel)
        for j in cols:                                 # each boundary column (and row of dq) on its own
            err = np.linalg.norm(res[name][j] - ref[j])
            assert err <= GRAD_REL * np.linalg.norm(ref[j]), (name, j, err / np.linalg.norm(ref[j]))
