"""fp64 CPU oracle for packed varlen causal attention, its gradients, and the partial/LSE merge.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA kernels are checked
against.  It shares no code with the CUDA path and must never be imported by it; only the tests,
the smoke check and the benchmark's CPU-baseline leg use it.

What it computes (paper Sec. 3.1, Eq. 1, with the causal mask of Sec. 4.3 "Time Estimation",
eta_k = 0):  for one sequence of length L, one query head and its KV head, inputs widened to fp64,

    s_ij  = (q_i . k_j) / sqrt(D)            for j <= i
    LSE_i = log sum_{j<=i} exp(s_ij)
    p_ij  = exp(s_ij - LSE_i)
    o_i   = sum_{j<=i} p_ij v_j

and, given dO (the paper states no backward; this is the derivative of the definition above):

    dv_j  = sum_{i>=j} p_ij dO_i
    dp_ij = dO_i . v_j
    delta_i = dO_i . o_i
    ds_ij = p_ij (dp_ij - delta_i)
    dq_i  = sum_{j<=i} ds_ij k_j / sqrt(D)
    dk_j  = sum_{i>=j} ds_ij q_i / sqrt(D)

Grouped-query attention: query head h reads KV head floor(h / (hq/hkv)); dk, dv are summed over the
query heads that share a KV head.

The functions take a *row range* of queries so that long sequences can be evaluated a slab of rows
at a time (each row is still the definition above, the sums over i are just taken slab by slab);
`rows=None` means all rows at once.

Chunked evaluation (a context-parallel plan cuts the key range of a query chunk into several KV
ranges, each giving a normalised partial output and its log-sum-exp) and the exact merge

    LSE = m + log sum_s exp(lse_s - m),    o = sum_s exp(lse_s - LSE) o_s

are also here; the paper (built on ring-style CP, Sec. 3.2) does not print the merge formula, it is
the re-association of the softmax sum and is pinned by "chunk-then-merge == unchunked".

Pins: tests/test_oracle_attention.py (row sums, constant V, first token, Q = 0 closed form,
finite differences, chunk-then-merge, per-row form vs full form, triple-loop brute force).
"""
from __future__ import annotations

import math

import numpy as np

__all__ = [
    "attention_fwd_seq", "attention_bwd_seq", "attention_fwd_packed", "attention_bwd_packed",
    "attention_row", "attention_row_grad", "partial_attention", "merge_partials", "brute_force_seq",
]


def _probabilities(q, k, rows):
    """Scaled scores, LSE and probabilities for query rows [i0, i1) against keys [0, i1)."""
    i0, i1 = rows
    D = q.shape[-1]
    s = (q[i0:i1] @ k[:i1].T) / math.sqrt(D)                      # [i1-i0, i1]
    ii = np.arange(i0, i1)[:, None]
    jj = np.arange(i1)[None, :]
    allowed = jj <= ii
    s = np.where(allowed, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)                                             # masked entries -> exp(-inf) = 0
    z = e.sum(axis=1, keepdims=True)
    lse = (m + np.log(z))[:, 0]
    p = e / z
    return p, lse


def attention_fwd_seq(q, k, v, rows=None):
    """One (sequence, head): q[L,D], k[L,D], v[L,D] fp64 -> (o[rows,D], lse[rows])."""
    L = q.shape[0]
    rows = (0, L) if rows is None else rows
    p, lse = _probabilities(q, k, rows)
    o = p @ v[: rows[1]]
    return o, lse


def attention_bwd_seq(q, k, v, do, rows=None):
    """One (sequence, head).  Returns (dq[rows,D], dk[L,D], dv[L,D]); dk/dv hold the contribution
    of the query rows in `rows` only (all of it when rows is None)."""
    L, D = q.shape
    rows = (0, L) if rows is None else rows
    i0, i1 = rows
    p, _ = _probabilities(q, k, rows)
    o = p @ v[:i1]
    dO = do[i0:i1]
    dv = np.zeros_like(v)
    dk = np.zeros_like(k)
    dv[:i1] = p.T @ dO
    dp = dO @ v[:i1].T
    delta = (dO * o).sum(axis=1, keepdims=True)
    ds = p * (dp - delta)
    dq = (ds @ k[:i1]) / math.sqrt(D)
    dk[:i1] = (ds.T @ q[i0:i1]) / math.sqrt(D)
    return dq, dk, dv


def _slabs(L, slab):
    return [(a, min(L, a + slab)) for a in range(0, L, slab)]


def attention_fwd_packed(q, k, v, cu_seqlens, slab=2048):
    """Packed batch.  q[T,hq,D], k/v[T,hkv,D] fp64, cu_seqlens[B+1] -> o[T,hq,D], lse[T,hq]."""
    T, hq, D = q.shape
    hkv = k.shape[1]
    g = hq // hkv
    o = np.zeros((T, hq, D))
    lse = np.zeros((T, hq))
    for b in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(hq):
            qs, ks, vs = q[t0:t1, h], k[t0:t1, h // g], v[t0:t1, h // g]
            for rows in _slabs(t1 - t0, slab):
                ob, lb = attention_fwd_seq(qs, ks, vs, rows)
                o[t0 + rows[0]: t0 + rows[1], h] = ob
                lse[t0 + rows[0]: t0 + rows[1], h] = lb
    return o, lse


def attention_bwd_packed(q, k, v, do, cu_seqlens, slab=2048):
    """Packed batch gradients: dq[T,hq,D], dk[T,hkv,D], dv[T,hkv,D] (fp64)."""
    T, hq, D = q.shape
    hkv = k.shape[1]
    g = hq // hkv
    dq = np.zeros((T, hq, D))
    dk = np.zeros((T, hkv, D))
    dv = np.zeros((T, hkv, D))
    for b in range(len(cu_seqlens) - 1):
        t0, t1 = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(hq):
            qs, ks, vs, dos = q[t0:t1, h], k[t0:t1, h // g], v[t0:t1, h // g], do[t0:t1, h]
            for rows in _slabs(t1 - t0, slab):
                dqb, dkb, dvb = attention_bwd_seq(qs, ks, vs, dos, rows)
                dq[t0 + rows[0]: t0 + rows[1], h] = dqb
                dk[t0:t1, h // g] += dkb
                dv[t0:t1, h // g] += dvb
    return dq, dk, dv


def attention_row(q_i, k, v, i):
    """Single query row i of one (sequence, head): the definition restricted to one row.
    k, v are the sequence's keys/values [L,D]; only rows 0..i are read.  Returns (o_i[D], lse_i)."""
    D = q_i.shape[-1]
    s = (k[: i + 1] @ q_i) / math.sqrt(D)
    m = s.max()
    e = np.exp(s - m)
    z = e.sum()
    return (e / z) @ v[: i + 1], m + math.log(z)


def attention_row_grad(q_i, k, v, do_i, i):
    """Gradient terms of a single query row i of one (sequence, head): returns (dq_i[D], p[i+1],
    ds[i+1]); row i adds p_j * dO_i to dv_j and ds_j * q_i / sqrt(D) to dk_j for every j <= i."""
    D = q_i.shape[-1]
    s = (k[: i + 1] @ q_i) / math.sqrt(D)
    m = s.max()
    e = np.exp(s - m)
    p = e / e.sum()
    o_i = p @ v[: i + 1]
    dp = v[: i + 1] @ do_i
    delta = float(do_i @ o_i)
    ds = p * (dp - delta)
    return (ds @ k[: i + 1]) / math.sqrt(D), p, ds


def partial_attention(q, k, v, q_rows, kv_ranges):
    """Normalised partial output and its LSE for query rows [q0,q1) of one (sequence, head),
    attending only to keys in the union of `kv_ranges` (list of (j0,j1)), causally masked (j <= i).
    Every row must see at least one key.  Positions are sequence-relative."""
    q0, q1 = q_rows
    D = q.shape[-1]
    cols = np.concatenate([np.arange(a, b) for a, b in kv_ranges])
    s = (q[q0:q1] @ k[cols].T) / math.sqrt(D)
    allowed = cols[None, :] <= np.arange(q0, q1)[:, None]
    s = np.where(allowed, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    z = e.sum(axis=1, keepdims=True)
    return (e / z) @ v[cols], (m + np.log(z))[:, 0]


def merge_partials(o_parts, lse_parts):
    """Exact combination of S normalised partials.  o_parts[S,...,D], lse_parts[S,...]."""
    lse_parts = np.asarray(lse_parts, dtype=np.float64)
    o_parts = np.asarray(o_parts, dtype=np.float64)
    m = lse_parts.max(axis=0)
    lse = m + np.log(np.exp(lse_parts - m).sum(axis=0))
    w = np.exp(lse_parts - lse)
    return (w[..., None] * o_parts).sum(axis=0), lse


def brute_force_seq(q, k, v, do=None):
    """Triple-loop evaluation of the definition with Python floats (tiny inputs only)."""
    L, D = len(q), len(q[0])
    sc = 1.0 / math.sqrt(D)
    o = [[0.0] * D for _ in range(L)]
    lse = [0.0] * L
    P = [[0.0] * L for _ in range(L)]
    for i in range(L):
        s = [sc * sum(q[i][c] * k[j][c] for c in range(D)) for j in range(i + 1)]
        z = sum(math.exp(x) for x in s)
        lse[i] = math.log(z)
        for j in range(i + 1):
            P[i][j] = math.exp(s[j]) / z
            for c in range(D):
                o[i][c] += P[i][j] * v[j][c]
    if do is None:
        return np.array(o), np.array(lse)
    dq = [[0.0] * D for _ in range(L)]
    dk = [[0.0] * D for _ in range(L)]
    dv = [[0.0] * D for _ in range(L)]
    for i in range(L):
        delta = sum(do[i][c] * o[i][c] for c in range(D))
        for j in range(i + 1):
            dp = sum(do[i][c] * v[j][c] for c in range(D))
            ds = P[i][j] * (dp - delta)
            for c in range(D):
                dv[j][c] += P[i][j] * do[i][c]
                dq[i][c] += sc * ds * k[j][c]
                dk[j][c] += sc * ds * q[i][c]
    return np.array(o), np.array(lse), np.array(dq), np.array(dk), np.array(dv)
