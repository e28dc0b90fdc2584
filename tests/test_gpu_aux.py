"""GPU tests of the parts around the kernels: the timing leg of the cost-model fit and the bounded
device-side wait."""
import numpy as np
import pytest

from paper_2602_21788_b200 import build, costfit, synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    build.build()
    torch.cuda.set_device(0)


def test_cost_model_timing_leg_fit_and_predict_round_trip():
    """`costfit.measure_grid` on a 2 x 2 grid of (length, degree), then the fit of Eq. 4's coefficients on
    those timings: positive times that grow with the length, an exact fit/predict round trip on a system
    with as many equations as it can determine, and coefficients that `fcp_plan_strategy` accepts."""
    from paper_2602_21788_b200 import fcp
    rows, times, labels = costfit.measure_grid([1024, 4096], [1, 3], hq=8, hkv=2, head_dim=128, tokens=16384)
    assert [(L, d) for L, d, _ in labels] == [(1024, 1), (1024, 3), (4096, 1), (4096, 3)]
    assert all(t > 0 for t in times)
    assert times[2] > times[0] and times[3] > times[1]            # 4x the length at equal tokens: more work
    c = costfit.fit(rows, times)
    assert set(c) == {"alpha1", "alpha2", "beta1"} and c["alpha1"] > 0
    pred = [costfit.predict(c, [L] * n, [d] * n) for (L, d, n) in labels]
    errs = costfit.relative_errors(c, [([L] * n, [d] * n) for (L, d, n) in labels], times)
    assert np.allclose(pred, [float(np.dot(r, [c["alpha1"], c["alpha2"], c["beta1"]])) for r in rows])
    assert errs.max() < 0.5                                       # 4 points, 3 coefficients: a loose sanity bound
    w = synth.make_workload("tiny", 0)
    plan = fcp.fcp_plan_strategy(w.seqlens, 8, 4096.0, 1.0, 0.0,
                                 dict(alpha1=c["alpha1"], alpha2=max(c["alpha2"], 0.0), alpha3=0.0,
                                      beta1=max(c["beta1"], 0.0), beta2=0.0, v=1.0))
    assert int(plan["cp_degree"].min()) >= 1 and plan["makespan"] > 0


def test_bounded_wait_runs_out_reports_timeout_and_leaves_the_context_usable():
    """A wait on a barrier nobody arrives at, with a 1 ms limit: the kernel returns by itself, the status
    words say FCP_ERR_TIMEOUT and name the wait site, and the next ordinary calls run and pass parity."""
    import time
    from oracle import attention_ref as A
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import run_fwd_bwd
    t0 = time.perf_counter()
    st = fcp.fcp_selftest_bounded_wait(1000)
    assert time.perf_counter() - t0 < 5.0
    assert st.tolist() == [fcp.FCP_ERR_TIMEOUT, 901, 0, 0]
    assert fcp.status_string(int(st[0])) == "FCP_ERR_TIMEOUT"
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_selftest_bounded_wait(0)
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    w = synth.Workload(name="after", seed=2, seqlens=np.asarray([500, 131], np.int32), cp_degrees=np.asarray([3, 1], np.int32),
                       hq=2, hkv=1, head_dim=128)
    q, k, v, do = w.tensors()
    res = run_fwd_bwd(w, q, k, v, do)                             # checks the plan's own status words: still clean
    f = synth.bf16_bits_to_f64
    o_ref, lse_ref = A.attention_fwd_packed(f(q), f(k), f(v), w.cu_seqlens)
    assert np.abs(res["o_f32"] - o_ref).max() <= 1e-2 and np.abs(res["lse"] - lse_ref).max() <= 1e-3
    dq_ref, dk_ref, dv_ref = A.attention_bwd_packed(f(q), f(k), f(v), f(do), w.cu_seqlens)
    for name, ref in (("dq", dq_ref), ("dk", dk_ref), ("dv", dv_ref)):
        assert np.linalg.norm(res[name] - ref) <= 2e-2 * np.linalg.norm(ref)


def test_no_call_writes_outside_the_buffers_it_was_given():
    """Guard bands around every output and workspace buffer (64 KB of a byte pattern on both sides) stay
    untouched by the partial path, the merged and the fused forward and the backward pass, on a ragged batch
    (tiles cut by sequence ends, empty chunks, head passes)."""
    from paper_2602_21788_b200.runner import DeviceState
    GUARD = 1 << 16
    w = synth.Workload(name="guards", seed=6, seqlens=np.asarray([1, 700, 129, 3, 1031], np.int32),
                       cp_degrees=np.asarray([1, 3, 1, 4, 5], np.int32), hq=4, hkv=2, head_dim=128)
    q, k, v, do = w.tensors()
    ds = DeviceState(w, q, k, v, do, heads_per_pass=3, want_o_f32=True, kv_heads_per_bwd_pass=1)
    arenas = {}
    for name in ("o_part", "lse_part", "o", "lse", "o_f32", "dq", "dk", "dv", "scratch"):
        t = getattr(ds, name)
        nbytes = t.numel() * t.element_size()
        arena = torch.full((nbytes + 2 * GUARD,), 0xA5, dtype=torch.uint8, device="cuda")
        inner = arena[GUARD:GUARD + nbytes].view(t.dtype).view(t.shape)
        assert inner.data_ptr() % 256 == 0
        setattr(ds, name, inner)
        arenas[name] = (arena, nbytes)
    ds.forward()
    ds.forward(merged=True)
    ds.forward_fused()
    ds.backward()
    torch.cuda.synchronize()
    ds.check_status()
    for name, (arena, nbytes) in arenas.items():
        assert bool((arena[:GUARD] == 0xA5).all()) and bool((arena[GUARD + nbytes:] == 0xA5).all()), name
    assert torch.isfinite(ds.o.float()).all() and torch.isfinite(ds.dq.float()).all()
