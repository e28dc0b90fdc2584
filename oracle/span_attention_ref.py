"""fp64 CPU oracle for attention with bidirectional spans inside an otherwise causal sequence.

TEST INFRASTRUCTURE ONLY: the slow, plain definition the CUDA kernels are checked against.  It
shares no code with the CUDA path and must never be imported by it.

What it computes.  The paper's cost model carries a mask efficiency factor eta_k because
multimodal models let some tokens (an image's or a video frame's tokens) attend to each other in
both directions while text stays causal (Sec. 4.3, "Time Estimation", Eq. 4: eta_k = 0 for a causal
mask, eta_k > 0 when part of the sequence uses full attention).  The paper gives no mask layout;
the reading used here: a sequence carries a sorted list of disjoint spans [a, b) (positions relative
to the sequence start); query i sees key j iff

    j <= i                      (causal), or
    a <= i < b and a <= j < b   for one of the spans (both inside the same span).

Equivalently row i sees exactly the keys j < lim(i) with lim(i) = b inside a span [a, b) and i + 1
elsewhere, and key j is seen by exactly the queries i >= first(j) with first(j) = a inside a span
and j elsewhere.  With that mask the attention function and its gradients are Eq. 1 (Sec. 3.1) and
its derivative as in `attention_ref.py`:

    s_ij = q_i . k_j / sqrt(D),  p_ij = softmax over the visible j,  o_i = sum_j p_ij v_j,
    dv_j = sum_i p_ij dO_i, dp_ij = dO_i . v_j, delta_i = dO_i . o_i, ds_ij = p_ij (dp_ij - delta_i),
    dq_i = sum_j ds_ij k_j / sqrt(D), dk_j = sum_i ds_ij q_i / sqrt(D).

`mask_efficiency` is the eta_k this mask implies: visible pairs relative to the causal count, minus 1.

Pins: tests/test_oracle_spans.py (no spans == the causal oracle; one span over the whole sequence ==
scipy's unmasked softmax / logsumexp; triple-loop brute force over the visibility predicate; central
finite differences; closed forms of lim, first and eta).
"""
from __future__ import annotations

import math

import numpy as np

__all__ = ["visible", "row_limits", "first_queries", "mask_efficiency", "span_attention_fwd_seq",
           "span_attention_bwd_seq", "span_attention_fwd_packed", "span_attention_bwd_packed", "brute_force_span_seq"]


def visible(i: int, j: int, spans) -> bool:
    """The visibility predicate, straight from the definition."""
    if j <= i:
        return True
    return any(a <= i < b and a <= j < b for a, b in spans)


def row_limits(L: int, spans) -> np.ndarray:
    """lim[i] = first key position row i does not see."""
    lim = np.arange(1, L + 1, dtype=np.int64)
    for a, b in spans:
        lim[a:b] = b
    return lim


def first_queries(L: int, spans) -> np.ndarray:
    """first[j] = first query position that sees key j."""
    first = np.arange(L, dtype=np.int64)
    for a, b in spans:
        first[a:b] = a
    return first


def mask_efficiency(L: int, spans) -> float:
    """eta of Eq. 4 for this mask: (visible pairs) / (causal pairs) - 1."""
    causal = L * (L + 1) // 2
    return float(int(row_limits(L, spans).sum()) - causal) / causal


def _mask(L, spans):
    return np.arange(L)[None, :] < row_limits(L, spans)[:, None]


def _probabilities(q, k, spans):
    L, D = q.shape
    s = (q @ k.T) / math.sqrt(D)
    s = np.where(_mask(L, spans), s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return e / z, (m + np.log(z))[:, 0]


def span_attention_fwd_seq(q, k, v, spans):
    """One (sequence, head): q, k, v [L, D] fp64, spans list of (a, b) -> (o [L, D], lse [L])."""
    p, lse = _probabilities(q, k, spans)
    return p @ v, lse


def span_attention_bwd_seq(q, k, v, do, spans):
    """One (sequence, head): (dq, dk, dv), each [L, D]."""
    D = q.shape[1]
    p, _ = _probabilities(q, k, spans)
    o = p @ v
    dv = p.T @ do
    dp = do @ v.T
    delta = (do * o).sum(axis=1, keepdims=True)
    ds = p * (dp - delta)
    return (ds @ k) / math.sqrt(D), (ds.T @ q) / math.sqrt(D), dv


def span_attention_fwd_packed(q, k, v, cu_seqlens, spans_per_seq):
    """Packed batch: q [T, hq, D], k/v [T, hkv, D]; spans_per_seq[b] = list of (a, b) of sequence b."""
    T, hq, D = q.shape
    g = hq // k.shape[1]
    o, lse = np.zeros((T, hq, D)), np.zeros((T, hq))
    for b in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(hq):
            o[t0:t1, h], lse[t0:t1, h] = span_attention_fwd_seq(q[t0:t1, h], k[t0:t1, h // g], v[t0:t1, h // g],
                                                                 spans_per_seq[b])
    return o, lse


def span_attention_bwd_packed(q, k, v, do, cu_seqlens, spans_per_seq):
    """Packed batch gradients; dk, dv summed over the query heads of a KV head."""
    T, hq, D = q.shape
    hkv = k.shape[1]
    g = hq // hkv
    dq, dk, dv = np.zeros((T, hq, D)), np.zeros((T, hkv, D)), np.zeros((T, hkv, D))
    for b in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(hq):
            a, bk, bv = span_attention_bwd_seq(q[t0:t1, h], k[t0:t1, h // g], v[t0:t1, h // g], do[t0:t1, h],
                                               spans_per_seq[b])
            dq[t0:t1, h] = a
            dk[t0:t1, h // g] += bk
            dv[t0:t1, h // g] += bv
    return dq, dk, dv


def brute_force_span_seq(q, k, v, do, spans):
    """Triple loops over the visibility predicate with Python floats (tiny inputs only)."""
    L, D = len(q), len(q[0])
    sc = 1.0 / math.sqrt(D)
    o = [[0.0] * D for _ in range(L)]
    lse = [0.0] * L
    P = [[0.0] * L for _ in range(L)]
    for i in range(L):
        js = [j for j in range(L) if visible(i, j, spans)]
        s = {j: sc * sum(q[i][c] * k[j][c] for c in range(D)) for j in js}
        z = sum(math.exp(x) for x in s.values())
        lse[i] = math.log(z)
        for j in js:
            P[i][j] = math.exp(s[j]) / z
            for c in range(D):
                o[i][c] += P[i][j] * v[j][c]
    dq = [[0.0] * D for _ in range(L)]
    dk = [[0.0] * D for _ in range(L)]
    dv = [[0.0] * D for _ in range(L)]
    for i in range(L):
        delta = sum(do[i][c] * o[i][c] for c in range(D))
        for j in range(L):
            if P[i][j] == 0.0:
                continue
            dp = sum(do[i][c] * v[j][c] for c in range(D))
            ds = P[i][j] * (dp - delta)
            for c in range(D):
                dv[j][c] += P[i][j] * do[i][c]
                dq[i][c] += sc * ds * k[j][c]
                dk[j][c] += sc * ds * q[i][c]
    return np.array(o), np.array(lse), np.array(dq), np.array(dk), np.array(dv)
