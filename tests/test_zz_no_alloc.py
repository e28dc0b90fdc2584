"""The allocation-free backward entry point against the regular one.

Some users of the library reach the backward pass in a place where they may not allocate device
memory: every byte belongs to their framework's pool, cudaMalloc would stall or is off limits
there, or the device is simply full.  fcp_attn_bwd_noalloc serves them from an array built into the
library, needs no uploaded plan and no scratch argument.  It has to give the same gradients as
fcp_attn_bwd on the same inputs (and, like it, the fp64 oracle's within the parity tolerance), also
when it is called twice in a row (the built-in array keeps
the first call's contents, so the second call checks that everything that must be cleared is).

Collected last on purpose: with `-x` every other test has run before this one can fail.
"""
import numpy as np
import pytest

from oracle import attention_ref as A
from paper_2602_21788_b200 import build, synth

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    build.build()
    torch.cuda.set_device(0)


def _bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


@pytest.mark.parametrize("lens,degs,hq,hkv,D", [([1500, 300, 77], [3, 1, 2], 4, 2, 128), ([900, 129], [2, 1], 4, 4, 64)])
def test_noalloc_backward_matches_regular_backward_twice(lens, degs, hq, hkv, D):
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import DeviceState
    w = synth.Workload(name="noalloc", seed=11, seqlens=np.asarray(lens, np.int32), cp_degrees=np.asarray(degs, np.int32),
                       hq=hq, hkv=hkv, head_dim=D)
    q, k, v, do = w.tensors()
    ds = DeviceState(w, q, k, v, do)
    ds.forward()
    ds.backward()
    torch.cuda.synchronize()
    ds.check_status()
    ref = {n: synth.bf16_bits_to_f64(_bits(getattr(ds, n))) for n in ("dq", "dk", "dv")}
    f = synth.bf16_bits_to_f64
    oracle = dict(zip(("dq", "dk", "dv"), A.attention_bwd_packed(f(q), f(k), f(v), f(do), w.cu_seqlens)))

    host_plan = fcp.fcp_plan_blocks(w.seqlens, w.cp_degrees, hq, hkv, D)       # never uploaded
    assert fcp.fcp_noalloc_bytes_needed(host_plan) <= fcp.FCP_NOALLOC_MAX_BYTES
    st = torch.cuda.current_stream().cuda_stream
    for call in range(2):
        dq = torch.full_like(ds.dq, float("nan"))
        dk = torch.full_like(ds.dk, float("nan"))
        dv = torch.full_like(ds.dv, float("nan"))
        fcp.fcp_attn_bwd_noalloc(host_plan, ds.q, ds.k, ds.v, ds.o, ds.do, ds.lse, dq, dk, dv, st)
        torch.cuda.synchronize()
        assert fcp.fcp_noalloc_device_status()[0] == 0
        got = {"dq": dq, "dk": dk, "dv": dv}
        for n in ("dk", "dv"):                       # no atomics on these: bit-identical
            assert np.array_equal(synth.bf16_bits_to_f64(_bits(got[n])), ref[n]), (n, call)
        g = synth.bf16_bits_to_f64(_bits(got["dq"]))  # fp32 reductions in varying order: the tests' tolerance
        assert np.isfinite(g).all()
        assert np.linalg.norm(g - ref["dq"]) <= 2e-2 * np.linalg.norm(ref["dq"]), call
        for n in ("dq", "dk", "dv"):                 # and the fp64 oracle's gradients, at the parity tests' tolerance
            x = synth.bf16_bits_to_f64(_bits(got[n]))
            assert np.linalg.norm(x - oracle[n]) <= 2e-2 * np.linalg.norm(oracle[n]), (n, call)


def test_noalloc_rejects_batches_beyond_the_builtin_arena():
    from paper_2602_21788_b200 import fcp
    big = fcp.fcp_plan_blocks([65536], [4], 32, 8, 128)
    assert fcp.fcp_noalloc_bytes_needed(big) > fcp.FCP_NOALLOC_MAX_BYTES
    x = torch.zeros(16, device="cuda")
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_attn_bwd_noalloc(big, x, x, x, x, x, x, x, x, x, 0)
    assert e.value.status == fcp.FCP_ERR_WORKSPACE
    assert "arena" in str(e.value)
