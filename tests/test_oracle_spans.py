"""Pins of the span-mask oracle (oracle/span_attention_ref.py) to things other than itself."""
import math

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import attention_ref as A
from oracle import span_attention_ref as S


def _rand(L, D, seed):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((L, D)) for _ in range(4)]


def test_no_spans_is_the_causal_oracle():
    q, k, v, do = _rand(37, 8, 0)
    o, lse = S.span_attention_fwd_seq(q, k, v, [])
    o_ref, lse_ref = A.attention_fwd_seq(q, k, v)
    assert np.allclose(o, o_ref, atol=1e-13) and np.allclose(lse, lse_ref, atol=1e-13)
    for got, ref in zip(S.span_attention_bwd_seq(q, k, v, do, []), A.attention_bwd_seq(q, k, v, do)):
        assert np.allclose(got, ref, atol=1e-12)
    # spans of a single token change nothing either
    o1, lse1 = S.span_attention_fwd_seq(q, k, v, [(3, 4), (10, 11)])
    assert np.array_equal(o1, o) and np.array_equal(lse1, lse)


def test_span_over_the_whole_sequence_is_unmasked_library_softmax():
    L, D = 29, 16
    q, k, v, _ = _rand(L, D, 1)
    o, lse = S.span_attention_fwd_seq(q, k, v, [(0, L)])
    s = q @ k.T / math.sqrt(D)
    assert np.allclose(o, softmax(s, axis=1) @ v, atol=1e-13)
    assert np.allclose(lse, logsumexp(s, axis=1), atol=1e-13)


def test_rows_outside_spans_are_causal_rows_and_rows_inside_see_the_whole_span():
    L, D = 40, 8
    q, k, v, _ = _rand(L, D, 2)
    spans = [(5, 12), (20, 33)]
    o, lse = S.span_attention_fwd_seq(q, k, v, spans)
    for i in list(range(0, 5)) + list(range(12, 20)) + list(range(33, L)):
        o_i, lse_i = A.attention_row(q[i], k, v, i)
        assert np.allclose(o[i], o_i, atol=1e-13) and abs(lse[i] - lse_i) < 1e-13
    for a, b in spans:
        for i in range(a, b):                      # a row of a span = the causal row of the span's last position
            o_i, lse_i = A.attention_row(q[i], k, v, b - 1)
            assert np.allclose(o[i], o_i, atol=1e-13) and abs(lse[i] - lse_i) < 1e-13


@pytest.mark.parametrize("spans", [[], [(0, 7)], [(2, 5)], [(0, 3), (4, 7)], [(1, 2), (3, 6)]])
def test_brute_force_over_the_predicate(spans):
    L, D = 7, 3
    q, k, v, do = _rand(L, D, 3)
    bo, blse, bdq, bdk, bdv = S.brute_force_span_seq(q.tolist(), k.tolist(), v.tolist(), do.tolist(), spans)
    o, lse = S.span_attention_fwd_seq(q, k, v, spans)
    dq, dk, dv = S.span_attention_bwd_seq(q, k, v, do, spans)
    for got, ref in ((o, bo), (lse, blse), (dq, bdq), (dk, bdk), (dv, bdv)):
        assert np.allclose(got, ref, atol=1e-12)


def test_gradients_against_central_finite_differences():
    L, D = 11, 4
    q, k, v, do = _rand(L, D, 4)
    spans = [(2, 6), (7, 10)]
    dq, dk, dv = S.span_attention_bwd_seq(q, k, v, do, spans)

    def loss(q_, k_, v_):
        return float((S.span_attention_fwd_seq(q_, k_, v_, spans)[0] * do).sum())

    eps = 1e-6
    for which, grad in ((0, dq), (1, dk), (2, dv)):
        num = np.zeros_like(grad)
        for i in range(L):
            for c in range(D):
                args_p, args_m = [q.copy(), k.copy(), v.copy()], [q.copy(), k.copy(), v.copy()]
                args_p[which][i, c] += eps
                args_m[which][i, c] -= eps
                num[i, c] = (loss(*args_p) - loss(*args_m)) / (2 * eps)
        assert np.linalg.norm(num - grad) <= 1e-6 * np.linalg.norm(grad)


def test_limits_first_queries_and_predicate_agree():
    L = 23
    spans = [(0, 4), (9, 10), (15, 23)]
    lim, first = S.row_limits(L, spans), S.first_queries(L, spans)
    for i in range(L):
        for j in range(L):
            assert S.visible(i, j, spans) == (j < lim[i]) == (i >= first[j])
    assert np.all(np.diff(lim) >= 0) and np.all(np.diff(first) >= 0)     # both non-decreasing
    assert lim.tolist()[:5] == [4, 4, 4, 4, 5] and first.tolist()[15:] == [15] * 8


def test_mask_efficiency_closed_forms():
    assert S.mask_efficiency(100, []) == 0.0
    L = 64
    assert math.isclose(S.mask_efficiency(L, [(0, L)]), (L - 1) / (L + 1))          # full attention: L^2 pairs
    m, a = 10, 17
    assert math.isclose(S.mask_efficiency(L, [(a, a + m)]), m * (m - 1) / (L * (L + 1)))
    assert math.isclose(S.mask_efficiency(L, [(0, 8), (20, 36)]), (8 * 7 + 16 * 15) / (L * (L + 1)))


def test_packed_batch_keeps_sequences_and_heads_apart():
    rng = np.random.default_rng(5)
    lens, hq, hkv, D = [9, 14], 4, 2, 4
    T = sum(lens)
    q, do = rng.standard_normal((T, hq, D)), rng.standard_normal((T, hq, D))
    k, v = rng.standard_normal((T, hkv, D)), rng.standard_normal((T, hkv, D))
    spans = [[(2, 7)], [(0, 5), (8, 14)]]
    cu = np.array([0, 9, 23])
    o, lse = S.span_attention_fwd_packed(q, k, v, cu, spans)
    dq, dk, dv = S.span_attention_bwd_packed(q, k, v, do, cu, spans)
    for b, (t0, t1) in enumerate([(0, 9), (9, 23)]):
        dk_sum, dv_sum = np.zeros((t1 - t0, hkv, D)), np.zeros((t1 - t0, hkv, D))
        for h in range(hq):
            o_s, lse_s = S.span_attention_fwd_seq(q[t0:t1, h], k[t0:t1, h // 2], v[t0:t1, h // 2], spans[b])
            assert np.array_equal(o[t0:t1, h], o_s) and np.array_equal(lse[t0:t1, h], lse_s)
            a, bk, bv = S.span_attention_bwd_seq(q[t0:t1, h], k[t0:t1, h // 2], v[t0:t1, h // 2], do[t0:t1, h], spans[b])
            assert np.array_equal(dq[t0:t1, h], a)
            dk_sum[:, h // 2] += bk
            dv_sum[:, h // 2] += bv
        assert np.allclose(dk[t0:t1], dk_sum, atol=1e-13) and np.allclose(dv[t0:t1], dv_sum, atol=1e-13)


def test_span_tables_cover_the_visibility_predicate_exactly():
    """Token pairs implied by the causal block pairs plus the span pairs (each restricted by row_limit) ==
    the visibility predicate, and a span pair exists only where a span reaches across the two chunks."""
    from oracle import plan_ref as P
    lens, degs = [37, 50], [3, 2]
    spans = [[(4, 9), (11, 30)], [(0, 2), (20, 45)]]
    tab = P.span_tables(lens, degs, spans)
    pl = P.plan_blocks(lens, degs)
    cb, co = pl["chunk_bounds"], pl["chunk_offset"]
    T = sum(lens)
    cover = np.zeros((T, T), dtype=np.int32)
    lim = np.array(tab["row_limit"])
    for (b, r, s, qc, kc, kind) in pl["pairs"]:
        for i in range(cb[co[b] + qc], cb[co[b] + qc + 1]):
            for j in range(cb[co[b] + kc], cb[co[b] + kc + 1]):
                if j < lim[i]:                       # DIAG blocks widen inside a span, FULL blocks are unchanged
                    cover[i, j] += 1
    for (b, r, s, qc, kc) in tab["span_pairs"]:
        d = degs[b]
        assert kc > qc and r == (qc if qc < d else 2 * d - 1 - qc)
        assert s == (r - (kc if kc < d else 2 * d - 1 - kc)) % d
        n = 0
        for i in range(cb[co[b] + qc], cb[co[b] + qc + 1]):
            for j in range(cb[co[b] + kc], cb[co[b] + kc + 1]):
                if j < lim[i]:
                    cover[i, j] += 1
                    n += 1
        assert n > 0                                  # no idle span pair
    want = np.zeros((T, T), dtype=np.int32)
    t0 = 0
    for b, L in enumerate(lens):
        for i in range(L):
            for j in range(L):
                want[t0 + i, t0 + j] = S.visible(i, j, spans[b])
        t0 += L
    assert np.array_equal(cover, want)
    fq = np.array(tab["first_query"])
    ii, jj = np.nonzero(want)
    assert np.all(ii >= fq[jj]) and np.all(jj < lim[ii])
