"""Pins for oracle/attention_ref.py: invariants, closed forms, library routines, finite
differences, brute force.  Each is chosen so that a dropped term, wrong sign/index or transposed
operand in the oracle fails at least one of them."""
import math

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import attention_ref as A


def _rand(L, D, seed, n=4):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((L, D)) for _ in range(n)]


@pytest.mark.parametrize("L,D", [(1, 4), (7, 8), (33, 16), (130, 64)])
def test_probability_rows_sum_to_one_and_are_causal(L, D):
    q, k, v, _ = _rand(L, D, 1)
    p, lse = A._probabilities(q, k, (0, L))
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.triu(p, 1) == 0.0)
    assert np.all(p >= 0)


def test_constant_v_gives_o_equal_v():
    q, k, _, _ = _rand(50, 16, 2)
    c = np.random.default_rng(3).standard_normal(16)
    v = np.tile(c, (50, 1))
    o, _ = A.attention_fwd_seq(q, k, v)
    assert np.allclose(o, v, atol=1e-12)


def test_first_token_attends_only_to_itself():
    q, k, v, _ = _rand(20, 8, 4)
    o, lse = A.attention_fwd_seq(q, k, v)
    assert np.allclose(o[0], v[0], atol=1e-14)
    assert math.isclose(lse[0], float(q[0] @ k[0]) / math.sqrt(8), rel_tol=1e-13)


def test_zero_q_is_running_mean_and_log_count():
    _, k, v, _ = _rand(40, 8, 5)
    q = np.zeros((40, 8))
    o, lse = A.attention_fwd_seq(q, k, v)
    want = np.cumsum(v, axis=0) / np.arange(1, 41)[:, None]
    assert np.allclose(o, want, atol=1e-13)
    assert np.allclose(lse, np.log(np.arange(1, 41)), atol=1e-13)


def test_last_row_equals_library_softmax():
    """The last query sees every key: plain (unmasked) softmax attention from scipy."""
    L, D = 64, 32
    q, k, v, _ = _rand(L, D, 6)
    o, lse = A.attention_fwd_seq(q, k, v)
    s = (k @ q[-1]) / math.sqrt(D)
    assert np.allclose(o[-1], softmax(s) @ v, atol=1e-13)
    assert math.isclose(lse[-1], logsumexp(s), rel_tol=1e-13)
    # and every row i equals the unmasked library softmax over the prefix 0..i
    for i in (0, 1, 17, 40):
        s = (k[: i + 1] @ q[i]) / math.sqrt(D)
        assert np.allclose(o[i], softmax(s) @ v[: i + 1], atol=1e-13)
        assert math.isclose(lse[i], logsumexp(s), rel_tol=1e-12, abs_tol=1e-13)


def test_scale_is_inverse_sqrt_head_dim():
    """With q = k = unit vectors e_0 * a, scores are a^2/sqrt(D): two-token closed form."""
    D, a = 16, 3.0
    q = np.zeros((2, D)); k = np.zeros((2, D)); v = np.zeros((2, D))
    q[:, 0] = a; k[1, 0] = a; v[0, 0] = 1.0; v[1, 1] = 1.0
    o, lse = A.attention_fwd_seq(q, k, v)
    s1 = a * a / math.sqrt(D)
    w1 = math.exp(s1) / (1.0 + math.exp(s1))
    assert np.allclose(o[1, :2], [1 - w1, w1], atol=1e-14)
    assert math.isclose(lse[1], math.log(1.0 + math.exp(s1)), rel_tol=1e-14)


@pytest.mark.parametrize("L,D", [(1, 2), (5, 3), (12, 4)])
def test_matches_triple_loop_brute_force(L, D):
    q, k, v, do = _rand(L, D, 7)
    o, lse = A.attention_fwd_seq(q, k, v)
    dq, dk, dv = A.attention_bwd_seq(q, k, v, do)
    bo, bl, bdq, bdk, bdv = A.brute_force_seq(q.tolist(), k.tolist(), v.tolist(), do.tolist())
    for x, y in ((o, bo), (lse, bl), (dq, bdq), (dk, bdk), (dv, bdv)):
        assert np.allclose(x, y, atol=1e-12)


@pytest.mark.parametrize("L,D", [(6, 4), (16, 8)])
def test_gradients_match_central_finite_differences(L, D):
    q, k, v, do = _rand(L, D, 8)
    dq, dk, dv = A.attention_bwd_seq(q, k, v, do)

    def loss(q_, k_, v_):
        o, _ = A.attention_fwd_seq(q_, k_, v_)
        return float((o * do).sum())

    eps = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            xp = x.copy(); xm = x.copy()
            xp[idx] += eps; xm[idx] -= eps
            args_p = dict(q=q, k=k, v=v); args_m = dict(q=q, k=k, v=v)
            args_p[name] = xp; args_m[name] = xm
            num[idx] = (loss(args_p["q"], args_p["k"], args_p["v"]) - loss(args_m["q"], args_m["k"], args_m["v"])) / (2 * eps)
        rel = np.linalg.norm(num - g) / np.linalg.norm(num)
        assert rel < 1e-6, (name, rel)


def test_softmax_gradient_rows_sum_to_zero():
    """sum_j ds_ij = 0 for every row (softmax Jacobian annihilates constants): dq of a sequence
    whose keys are all equal must vanish."""
    L, D = 24, 8
    q, _, v, do = _rand(L, D, 9)
    k = np.tile(np.random.default_rng(10).standard_normal(D), (L, 1))
    dq, _, _ = A.attention_bwd_seq(q, k, v, do)
    assert np.allclose(dq, 0.0, atol=1e-12)


def test_row_slabs_and_row_form_agree_with_full_form():
    L, D = 150, 16
    q, k, v, do = _rand(L, D, 11)
    o, lse = A.attention_fwd_seq(q, k, v)
    dq, dk, dv = A.attention_bwd_seq(q, k, v, do)
    o2 = np.zeros_like(o); l2 = np.zeros_like(lse)
    dq2 = np.zeros_like(dq); dk2 = np.zeros_like(dk); dv2 = np.zeros_like(dv)
    for rows in [(0, 37), (37, 101), (101, 150)]:
        ob, lb = A.attention_fwd_seq(q, k, v, rows)
        o2[rows[0]:rows[1]] = ob; l2[rows[0]:rows[1]] = lb
        a, b, c = A.attention_bwd_seq(q, k, v, do, rows)
        dq2[rows[0]:rows[1]] = a; dk2 += b; dv2 += c
    for x, y in ((o, o2), (lse, l2), (dq, dq2), (dk, dk2), (dv, dv2)):
        assert np.allclose(x, y, atol=1e-12)
    for i in (0, 5, 149):
        oi, li = A.attention_row(q[i], k, v, i)
        assert np.allclose(oi, o[i], atol=1e-13) and math.isclose(li, lse[i], rel_tol=1e-13)


def test_row_gradient_form_sums_to_full_gradients():
    L, D = 40, 8
    q, k, v, do = _rand(L, D, 14)
    dq, dk, dv = A.attention_bwd_seq(q, k, v, do)
    dk2 = np.zeros_like(dk); dv2 = np.zeros_like(dv)
    for i in range(L):
        dqi, p, ds = A.attention_row_grad(q[i], k, v, do[i], i)
        assert np.allclose(dqi, dq[i], atol=1e-13)
        dv2[: i + 1] += p[:, None] * do[i][None, :]
        dk2[: i + 1] += ds[:, None] * q[i][None, :] / math.sqrt(D)
    assert np.allclose(dk2, dk, atol=1e-12) and np.allclose(dv2, dv, atol=1e-12)


def test_packed_gqa_matches_per_sequence_and_sums_kv_heads():
    rng = np.random.default_rng(12)
    lens = [5, 1, 19]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T, hq, hkv, D = cu[-1], 4, 2, 8
    q = rng.standard_normal((T, hq, D)); k = rng.standard_normal((T, hkv, D))
    v = rng.standard_normal((T, hkv, D)); do = rng.standard_normal((T, hq, D))
    o, lse = A.attention_fwd_packed(q, k, v, cu, slab=7)
    dq, dk, dv = A.attention_bwd_packed(q, k, v, do, cu, slab=7)
    dk_ref = np.zeros_like(dk); dv_ref = np.zeros_like(dv)
    for b in range(3):
        s = slice(cu[b], cu[b + 1])
        for h in range(hq):
            ob, lb = A.attention_fwd_seq(q[s, h], k[s, h // 2], v[s, h // 2])
            assert np.allclose(o[s, h], ob, atol=1e-13) and np.allclose(lse[s, h], lb, atol=1e-13)
            a, bb, c = A.attention_bwd_seq(q[s, h], k[s, h // 2], v[s, h // 2], do[s, h])
            assert np.allclose(dq[s, h], a, atol=1e-13)
            dk_ref[s, h // 2] += bb; dv_ref[s, h // 2] += c
    assert np.allclose(dk, dk_ref, atol=1e-12) and np.allclose(dv, dv_ref, atol=1e-12)
    # no leakage across sequences: changing sequence 0 leaves sequence 2's output unchanged
    q2 = q.copy(); q2[: cu[1]] += 1.0
    o2, _ = A.attention_fwd_packed(q2, k, v, cu, slab=7)
    assert np.array_equal(o2[cu[1]:], o[cu[1]:])
    assert not np.allclose(o2[: cu[1]], o[: cu[1]])


def test_merge_of_disjoint_key_ranges_is_exact():
    L, D = 90, 16
    q, k, v, _ = _rand(L, D, 13)
    o, lse = A.attention_fwd_seq(q, k, v)
    rows = (60, 90)
    parts = [A.partial_attention(q, k, v, rows, [(0, 13)]),
             A.partial_attention(q, k, v, rows, [(13, 40), (55, 60)]),
             A.partial_attention(q, k, v, rows, [(40, 55)]),
             A.partial_attention(q, k, v, rows, [(60, 90)])]
    om, lm = A.merge_partials([p[0] for p in parts], [p[1] for p in parts])
    assert np.allclose(om, o[60:90], atol=1e-12) and np.allclose(lm, lse[60:90], atol=1e-12)
    # a single partial merges to itself
    o1, l1 = A.merge_partials([parts[0][0]], [parts[0][1]])
    assert np.allclose(o1, parts[0][0], atol=1e-15) and np.allclose(l1, parts[0][1], atol=1e-15)


def test_merge_two_slot_closed_form():
    """Two slots with lse a, b: weights are the logistic of (a-b)."""
    a, b = 0.3, -1.1
    o, l = A.merge_partials(np.array([[1.0, 0.0], [0.0, 1.0]]), np.array([a, b]))
    w = 1.0 / (1.0 + math.exp(b - a))
    assert np.allclose(o, [w, 1 - w], atol=1e-15)
    assert math.isclose(float(l), math.log(math.exp(a) + math.exp(b)), rel_tol=1e-15)
