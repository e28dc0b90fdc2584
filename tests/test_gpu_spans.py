"""GPU parity of the span mask (bidirectional spans inside causal sequences): fcp_attn_fwd_fused and
fcp_attn_bwd through the C ABI against the fp64 span oracle on the same seeded inputs."""
import numpy as np
import pytest

from oracle import span_attention_ref as S
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


def _check(w, kv_heads_per_bwd_pass=None):
    from paper_2602_21788_b200.runner import run_fwd_bwd
    q, k, v, do = w.tensors()
    res = run_fwd_bwd(w, q, k, v, do, fused=True, kv_heads_per_bwd_pass=kv_heads_per_bwd_pass)
    qf, kf, vf, dof = f64(q), f64(k), f64(v), f64(do)
    o_ref, lse_ref = S.span_attention_fwd_packed(qf, kf, vf, w.cu_seqlens, w.spans)
    e = np.abs(res["o_f32"] - o_ref)
    assert e.max() <= O_MAX and e.mean() <= O_MEAN, (e.max(), e.mean())
    assert np.abs(res["lse"] - lse_ref).max() <= LSE_MAX
    refs = S.span_attention_bwd_packed(qf, kf, vf, dof, w.cu_seqlens, w.spans)
    for name, ref in zip(("dq", "dk", "dv"), refs):
        rel = np.linalg.norm(res[name] - ref) / np.linalg.norm(ref)
        assert rel <= GRAD_REL and np.isfinite(res[name]).all(), (name, rel)
    return res


def _wl(lens, degs, spans, hq, hkv, D, seed=0):
    return synth.Workload(name="spans", seed=seed, seqlens=np.asarray(lens, np.int32), cp_degrees=np.asarray(degs, np.int32),
                          hq=hq, hkv=hkv, head_dim=D, spans=spans)


CASES = [
    # lens, degs, spans, hq, hkv, D
    ([300], [1], [[(100, 140)]], 2, 1, 128),                                 # inside tiles
    ([300], [1], [[(120, 135), (250, 300)]], 2, 2, 64),                      # across a tile edge; up to the sequence end
    ([700, 50], [3, 2], [[(0, 130), (230, 236), (400, 699)], []], 4, 2, 128),  # d = 3: across chunk edges (116, 233, 350, ...)
    ([1030], [6], [[(80, 95), (500, 860)]], 2, 1, 128),                      # d = 6: one span over several chunks
    ([257, 129, 1], [1, 1, 1], [[(0, 257)], [(1, 2)], []], 2, 1, 128),       # whole sequence bidirectional; one-token span
    ([2000], [3], [[(127, 129), (255, 257), (333, 334), (666, 1500)]], 8, 1, 128),  # spans straddling tile edges, GQA 8:1
    ([900, 640], [1, 5], [[(0, 900)], [(0, 640)]], 2, 2, 64),                # full attention everywhere (eta -> 1)
]


@pytest.mark.parametrize("lens,degs,spans,hq,hkv,D", CASES)
def test_span_mask_edge_shapes(lens, degs, spans, hq, hkv, D):
    _check(_wl(lens, degs, spans, hq, hkv, D, seed=4))


def test_span_plan_of_the_bimodal_workload_with_image_spans():
    """The bimodal batch with image spans, lengths / 16 so that the oracle runs in full; backward in two passes of KV heads."""
    w = synth.reduced(synth.make_workload("bimodal_128k_spans", 0))
    assert any(len(s) > 0 for s in w.spans)
    _check(w, kv_heads_per_bwd_pass=max(1, w.hkv // 2))


def test_rows_outside_spans_keep_their_causal_bits_and_partial_path_refuses_span_plans():
    """A query outside every span sees exactly its causal keys in the same order: same forward bits as the
    causal plan.  The per-item partial path is causal only and says so."""
    from paper_2602_21788_b200 import fcp
    from paper_2602_21788_b200.runner import DeviceState, run_fwd_bwd
    spans = [[(300, 420), (900, 1100)]]
    w = _wl([1500], [3], spans, 2, 1, 128, seed=9)
    wc = _wl([1500], [3], None, 2, 1, 128, seed=9)
    q, k, v = w.tensors(with_do=False)
    a = run_fwd_bwd(w, q, k, v, None, fused=True)
    c = run_fwd_bwd(wc, q, k, v, None, fused=True)
    outside = np.ones(1500, dtype=bool)
    for s0, s1 in spans[0]:
        outside[s0:s1] = False
    assert np.array_equal(a["o"][outside], c["o"][outside]) and np.array_equal(a["lse"][outside], c["lse"][outside])
    assert not np.array_equal(a["o"][~outside], c["o"][~outside])
    ds = DeviceState(w, q, k, v, None)
    with pytest.raises(fcp.FcpError) as e:
        ds.forward()
    assert e.value.status == fcp.FCP_ERR_UNSUPPORTED
    torch.cuda.synchronize()


@pytest.mark.slow
def test_full_size_bimodal_with_image_spans_sampled():
    """The benchmark's span workload at its real shape (131 072 tokens, 32 heads, 80 spans of 256-2048 tokens):
    sampled forward rows and dQ rows, inside spans, at their edges and outside, against the oracle's single-row
    form (a row with limit lim sees exactly what the causal row lim - 1 sees), plus dK/dV columns at the very end of
    the longest sequence."""
    import math
    from oracle import attention_ref as A
    from paper_2602_21788_b200.runner import DeviceState
    w = synth.make_workload("bimodal_128k_spans", 0)
    q, k, v, do = w.device_tensors()
    ds = DeviceState(w, q, k, v, do, partials=False, want_o_f32=True)
    ds.forward_fused()
    ds.backward()
    torch.cuda.synchronize()
    ds.check_status()
    b64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(0)
    cu, D = w.cu_seqlens, w.head_dim
    long_seqs = [b for b in range(len(w.seqlens)) if w.spans[b]]
    o_err, l_err, num, den = [], [], 0.0, 0.0
    for n in range(40):
        b = long_seqs[n % len(long_seqs)]
        L, t0 = int(w.seqlens[b]), int(cu[b])
        lim = S.row_limits(L, w.spans[b])
        a_, e_ = w.spans[b][int(rng.integers(len(w.spans[b])))]
        i = [a_, e_ - 1, int(rng.integers(a_, e_)), max(0, a_ - 1), min(L - 1, e_), int(rng.integers(L))][n % 6]
        h = int(rng.integers(w.hq))
        ks, vs = b64(k[t0:t0 + int(lim[i]), h]), b64(v[t0:t0 + int(lim[i]), h])      # hq == hkv in this workload
        qi, doi = b64(q[t0 + i, h]), b64(do[t0 + i, h])
        o_ref, lse_ref = A.attention_row(qi, ks, vs, int(lim[i]) - 1)
        dq_ref, _, _ = A.attention_row_grad(qi, ks, vs, doi, int(lim[i]) - 1)
        o_err.append(np.abs(ds.o_f32[t0 + i, h].cpu().numpy().astype(np.float64) - o_ref))
        l_err.append(abs(float(ds.lse[t0 + i, h]) - lse_ref))
        num += np.sum((b64(ds.dq[t0 + i, h]) - dq_ref) ** 2)
        den += np.sum(dq_ref ** 2)
    o_err = np.concatenate(o_err)
    assert o_err.max() <= O_MAX and o_err.mean() <= O_MEAN and max(l_err) <= LSE_MAX
    assert math.sqrt(num / den) <= GRAD_REL
    # dK/dV of the last 8 tokens of the longest sequence: every row from the first query that sees them on
    b = int(np.argmax(w.seqlens))
    L, t0 = int(w.seqlens[b]), int(cu[b])
    lim, first = S.row_limits(L, w.spans[b]), S.first_queries(L, w.spans[b])
    j0, hk = L - 8, 3
    ks, vs = b64(k[t0:t0 + L, hk]), b64(v[t0:t0 + L, hk])
    dk_ref, dv_ref = np.zeros((8, D)), np.zeros((8, D))
    for i in range(int(first[j0]), L):
        qi, doi = b64(q[t0 + i, hk]), b64(do[t0 + i, hk])
        n_i = int(lim[i])
        _, p, dsr = A.attention_row_grad(qi, ks[:n_i], vs[:n_i], doi, n_i - 1)
        lo = max(j0, 0)
        if n_i > lo:
            dv_ref[: n_i - lo] += p[lo:, None] * doi[None, :]
            dk_ref[: n_i - lo] += dsr[lo:, None] * qi[None, :] / math.sqrt(D)
    for name, ref, got in (("dk", dk_ref, ds.dk), ("dv", dv_ref, ds.dv)):
        assert np.linalg.norm(b64(got[t0 + j0:t0 + L, hk]) - ref) <= GRAD_REL * np.linalg.norm(ref), name
