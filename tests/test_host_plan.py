"""Host-only tests of libfcp: exported symbols, the block plan bit-exact against the oracle's integer
plan, the strategy planner against the oracle (Algorithm 1 and exhaustive search), error paths."""
import ctypes
import math
import os
import re

import numpy as np
import pytest

from oracle import plan_ref as P
from paper_2602_21788_b200 import build, fcp, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "fcp.h")).read()
    declared = set(re.findall(r"\b(fcp_[a-z_]+)\s*\(", hdr)) - {"fcp_plan"}
    assert set(fcp.EXPORTS) == declared
    L = ctypes.CDLL(fcp.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name
    assert fcp.status_string(0) == "FCP_OK" and fcp.status_string(-6) == "FCP_ERR_TIMEOUT"


def _compare(plan, ref):
    assert plan.table("chunk_bounds").tolist() == ref["chunk_bounds"]
    assert plan.table("chunk_offset").tolist() == ref["chunk_offset"]
    assert plan.table("pairs").tolist() == [list(p) for p in ref["pairs"]]
    assert plan.table("items").tolist() == [list(i) for i in ref["items"]]
    so = plan.table("slot_offset"); sr = plan.table("slot_rows")
    got = [(int(so[c + 1] - so[c]), sr[so[c]:so[c + 1]].tolist()) for c in range(len(so) - 1)]
    assert got == [(n, list(r)) for n, r in ref["chunk_slots"]]
    assert plan.info("R") == ref["n_partial_rows"]


@pytest.mark.parametrize("lens,degs", [
    ([1], [1]), ([1], [3]), ([5, 2, 1], [3, 2, 4]), ([64, 599, 609], [1, 3, 2]), ([1000], [8]),
    ([131072], [7]), ([393216, 843, 142], [7, 1, 1]), ([97, 3, 4096, 17], [5, 2, 6, 64]),
])
def test_block_plan_bit_exact_vs_oracle(lens, degs):
    plan = fcp.fcp_plan_blocks(lens, degs, 8, 2, 128)
    _compare(plan, P.plan_blocks(lens, degs))


@pytest.mark.parametrize("name", list(synth.WORKLOADS))
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_block_plan_bit_exact_on_workloads(name, seed):
    w = synth.make_workload(name, seed)
    plan = fcp.fcp_plan_blocks(w.seqlens, w.cp_degrees, w.hq, w.hkv, w.head_dim)
    _compare(plan, P.plan_blocks(w.seqlens.tolist(), w.cp_degrees.tolist()))
    assert plan.info("T") == w.total_tokens


def _cover_fwd(units, T, row_limit=None):
    """Token-pair coverage implied by a table of forward work units (per-item or fused); `row_limit`:
    the plan's row limits when it has bidirectional spans (a DIAG range then ends at the row's limit)."""
    fwd = np.zeros((T, T), dtype=np.int32)
    for u in units:
        q0, rows, prow, nr = u[0], u[1], u[2], u[3]
        nts = [u[10], u[11]]
        nr0 = u[12]
        for s in range(2):
            for j in range(nts[s]):
                r = 0 if j < nr0 else 1
                kb, ke, kd = (u[4], u[5], u[6]) if r == 0 else (u[7], u[8], u[9])
                ks = kb + 128 * j if r == 0 else kb + 128 * (j - nr0)
                for row in range(min(128, rows - 128 * s)):
                    qp = q0 + 128 * s + row
                    limit = ke - ks
                    if kd:
                        limit = min(limit, (qp + 1 if row_limit is None else row_limit[qp]) - ks)
                    limit = min(limit, 128)
                    assert limit >= 1 or row_limit is not None
                    if limit > 0:
                        fwd[qp, ks:ks + limit] += 1
    return fwd


def _cover_bwd(plan, T, first_query=None):
    """Token-pair coverage implied by the backward units: a DIAG range runs from Q tile T_FIRST on, and the
    tiles before T_MASK_END drop the queries before each key's first query (the key itself, or its span's begin)."""
    bwd = np.zeros((T, T), dtype=np.int32)
    qr = plan.table("bwd_qranges")
    for u in plan.table("bwd_units"):
        k0, krows, first, nq, t_first, cost, t_mask_end = u[0], u[1], u[2], u[3], u[4], u[5], u[7]
        n = 0
        for r in range(nq):
            qb, qe, diag = qr[first + r][:3]
            t = t_first if diag else 0
            while qb + 128 * t < qe:
                n += 1
                q_row = qb + 128 * t
                qv = min(128, qe - q_row)
                for row in range(krows):
                    fq = k0 + row if first_query is None else first_query[k0 + row]
                    lo = max(0, fq - q_row) if (diag and t < t_mask_end) else 0
                    if lo < qv:
                        bwd[q_row + lo:q_row + qv, k0 + row] += 1
                t += 1
        assert n == cost
    return bwd


def _cover(plan, lens):
    """Token-pair coverage implied by the derived forward and backward work lists."""
    cu = np.concatenate([[0], np.cumsum(lens)])
    T = int(cu[-1])
    fwd = _cover_fwd(plan.table("fwd_units"), T)
    bwd = _cover_bwd(plan, T)
    want = np.zeros((T, T), dtype=np.int32)
    for b in range(len(lens)):
        L = lens[b]
        want[cu[b]:cu[b + 1], cu[b]:cu[b + 1]] = np.tril(np.ones((L, L), dtype=np.int32))
    return fwd, bwd, want


def _pairs_cover(plan, lens):
    """Token-pair coverage of the canonical block pairs themselves (FULL: whole block, DIAG: its triangle)."""
    T = int(sum(lens))
    cb, co = plan.table("chunk_bounds"), plan.table("chunk_offset")
    out = np.zeros((T, T), dtype=np.int32)
    for (b, r, s, qc, kc, kind) in plan.table("pairs"):
        q0, q1, k0, k1 = cb[co[b] + qc], cb[co[b] + qc + 1], cb[co[b] + kc], cb[co[b] + kc + 1]
        blk = np.ones((q1 - q0, k1 - k0), dtype=np.int32)
        out[q0:q1, k0:k1] += np.tril(blk) if kind else blk
    return out


@pytest.mark.parametrize("lens,degs", [([300, 5, 129], [1, 3, 2]), ([700], [2]), ([1030], [3]), ([257, 256, 255], [1, 1, 1]),
                                       ([3, 1000, 2], [4, 7, 1]), ([513], [64])])
def test_work_lists_cover_the_causal_triangle_exactly_once(lens, degs):
    plan = fcp.fcp_plan_blocks(lens, degs, 4, 4, 64)
    fwd, bwd, want = _cover(plan, lens)
    assert np.array_equal(fwd, want)
    assert np.array_equal(bwd, want)
    # the fused forward units (all items of a Q chunk on one CTA) execute the same token pairs as the
    # plan's block pairs, each exactly once, and every query row belongs to exactly one unit
    pairs = _pairs_cover(plan, lens)
    assert np.array_equal(pairs, want)
    fused_units = plan.table("fused_units")
    assert np.array_equal(_cover_fwd(fused_units, int(sum(lens))), pairs)
    rows = np.zeros(sum(lens), dtype=np.int32)
    for u in fused_units:
        rows[u[0]:u[0] + u[1]] += 1
    assert np.all(rows == 1) and plan.info("n_fused_units") == len(fused_units)
    # backward execution order: a permutation of the units
    assert sorted(plan.table("bwd_work").tolist()) == list(range(plan.info("n_bwd_units")))
    # every partial row is written by exactly one forward unit
    R = plan.info("R")
    hit = np.zeros(R, dtype=np.int32)
    for u in plan.table("fwd_units"):
        hit[u[2]:u[2] + u[1]] += 1
    assert np.all(hit == 1)
    # merge units tile the tokens exactly once
    tok = np.zeros(sum(lens), dtype=np.int32)
    for m in plan.table("merge_units"):
        tok[m[0]:m[0] + m[1]] += 1
    assert np.all(tok == 1)


COEFFS = [dict(alpha1=1.0, alpha2=0.0, alpha3=0.0, beta1=0.0, beta2=0.0, v=1.0),
          dict(alpha1=1e-3, alpha2=0.7, alpha3=40.0, beta1=5.0, beta2=11.0, v=2.0)]


@pytest.mark.parametrize("coeffs", COEFFS)
def test_strategy_matches_oracle_and_exhaustive_search(coeffs):
    rng = np.random.default_rng(17)
    n_ok = 0
    for trial in range(80):
        B = int(rng.integers(1, 9))
        N = int(rng.integers(1, 11))
        lens = [int(x) for x in rng.integers(16, 3000, size=B)]
        E = float(rng.integers(800, 6000))
        eta = [float(x) for x in rng.random(B)] if trial % 2 else None
        ref = P.plan_strategy(lens, N, E, 1.0, 100.0, coeffs, eta)
        if ref is None:
            with pytest.raises(fcp.FcpError) as ei:
                fcp.fcp_plan_strategy(lens, N, E, 1.0, 100.0, coeffs, eta)
            assert ei.value.status == fcp.FCP_ERR_INFEASIBLE
            continue
        got = fcp.fcp_plan_strategy(lens, N, E, 1.0, 100.0, coeffs, eta)
        assert got["group_of"].tolist() == ref["group_of"]
        assert got["cp_degree"].tolist() == ref["cp_degree"]
        assert got["n_groups"] == len(ref["d_group"])
        assert got["makespan"] == ref["makespan"]
        assert sum(ref["d_group"]) == N
        if len(ref["d_group"]) <= 5:
            assert got["makespan"] == P.brute_force_allocate(ref["times"], ref["d_min"], N)
        n_ok += 1
    assert n_ok > 20


def test_strategy_plan_is_stable_under_small_coefficient_noise():
    """Sec. 5.4 reports identical plans up to 20 % coefficient noise on the paper's data; on a
    synthetic skewed batch only assert that the makespan under the noisy plan stays within a few %."""
    rng = np.random.default_rng(0)
    lens = [int(x) for x in np.clip(rng.lognormal(8.0, 1.2, size=24), 128, 131072)]
    base = dict(alpha1=1e-6, alpha2=1e-3, alpha3=1e-4, beta1=0.5, beta2=0.2, v=1.0)
    ref = fcp.fcp_plan_strategy(lens, 32, 30000.0, 1.0, 0.0, base)
    for trial in range(5):
        noisy = {k: v * (1.0 + 0.2 * (2 * rng.random() - 1)) if k != "v" else v for k, v in base.items()}
        got = fcp.fcp_plan_strategy(lens, 32, 30000.0, 1.0, 0.0, noisy)
        # evaluate the noisy plan under the true coefficients
        groups = {}
        for i, g in enumerate(got["group_of"]):
            groups.setdefault(int(g), []).append(i)
        true_mk = max(P.group_time([lens[i] for i in m], [0.0] * len(m), int(got["cp_degree"][m[0]]), base)
                      for m in groups.values())
        assert true_mk <= ref["makespan"] * 1.10


def test_error_paths():
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_blocks([10], [1], 8, 2, 96)
    assert e.value.status == fcp.FCP_ERR_UNSUPPORTED
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_blocks([10], [1], 8, 3, 128)
    assert e.value.status == fcp.FCP_ERR_UNSUPPORTED
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_blocks([10], [65], 8, 2, 128)
    assert e.value.status == fcp.FCP_ERR_UNSUPPORTED
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_blocks([10, 0], [1, 1], 8, 2, 128)
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_blocks([10], [0], 8, 2, 128)
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    with pytest.raises(fcp.FcpError) as e:                             # an empty batch is refused, not planned
        fcp.fcp_plan_blocks([], [], 8, 2, 128)
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_strategy([10], 4, 1.0, 1.0, 2.0, COEFFS[0])      # E <= M_ms
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_plan_strategy([10], 65, 100.0, 1.0, 0.0, COEFFS[0])
    assert e.value.status == fcp.FCP_ERR_UNSUPPORTED
    plan = fcp.fcp_plan_blocks([10], [1], 8, 2, 128)
    with pytest.raises(fcp.FcpError) as e:                             # compute call before upload
        fcp.fcp_attn_fwd(plan, 16, 16, 16, 16, 16)
    assert e.value.status == fcp.FCP_ERR_NOT_UPLOADED
    a, b, c = plan.workspace_bytes(8)
    assert a == plan.info("R") * 8 * 128 * 4 and b == plan.info("R") * 8 * 4 and c > 10 * 8 * 128 * 4


# ----------------------------------------------------------------------------------------------
# bidirectional spans
# ----------------------------------------------------------------------------------------------
SPAN_CASES = [
    ([300], [1], [[(100, 140)]]),                                   # inside one tile boundary region
    ([300], [1], [[(120, 135), (250, 300)]]),                       # across a tile edge; up to the sequence end
    ([700, 50], [3, 2], [[(0, 130), (230, 236), (400, 699)], []]),  # across chunk edges (bounds 116, 233, 350, ...)
    ([1030], [6], [[(80, 95), (500, 860)]]),                        # a span over several chunks
    ([257, 129], [1, 1], [[(0, 257)], [(1, 2)]]),                   # whole sequence; a one-token span (no effect)
]


@pytest.mark.parametrize("lens,degs,spans", SPAN_CASES)
def test_span_plan_tables_bit_exact_and_units_cover_the_mask(lens, degs, spans):
    from oracle import span_attention_ref as S
    plan = fcp.fcp_plan_blocks_spans(lens, degs, spans, 4, 2, 128)
    ref = P.span_tables(lens, degs, spans)
    assert plan.table("row_limit").tolist() == ref["row_limit"]
    assert plan.table("first_query").tolist() == ref["first_query"]
    assert plan.table("span_pairs").tolist() == [list(x) for x in ref["span_pairs"]]
    _compare(plan, P.plan_blocks(lens, degs))                       # the causal tables are unchanged
    T = sum(lens)
    want = np.zeros((T, T), dtype=np.int32)
    t0 = 0
    for b, L in enumerate(lens):
        lim = S.row_limits(L, spans[b])
        for i in range(L):
            want[t0 + i, t0:t0 + lim[i]] = 1
        t0 += L
    assert np.array_equal(_cover_fwd(plan.table("fused_units"), T, plan.table("row_limit")), want)
    assert np.array_equal(_cover_bwd(plan, T, plan.table("first_query")), want)
    for b, L in enumerate(lens):
        assert math.isclose(fcp.fcp_span_mask_efficiency(L, spans[b]), S.mask_efficiency(L, spans[b]), rel_tol=1e-12)


def test_span_plan_without_spans_is_the_causal_plan_and_bad_spans_are_refused():
    a = fcp.fcp_plan_blocks([500, 77], [2, 1], 4, 4, 64)
    b = fcp.fcp_plan_blocks_spans([500, 77], [2, 1], [[], []], 4, 4, 64)
    for name in ("pairs", "items", "fwd_units", "fused_units", "bwd_units", "bwd_qranges", "bwd_work", "merge_units"):
        assert np.array_equal(a.table(name), b.table(name)), name
    assert b.table("row_limit").size == 0 and b.table("span_pairs").size == 0
    for bad in ([[(5, 5)], []], [[(10, 600)], []], [[(20, 30), (25, 40)], []], [[(30, 40), (10, 20)], []], [[(-1, 4)], []]):
        with pytest.raises(fcp.FcpError) as e:
            fcp.fcp_plan_blocks_spans([500, 77], [2, 1], bad, 4, 4, 64)
        assert e.value.status == fcp.FCP_ERR_INVALID_ARG
    with pytest.raises(fcp.FcpError) as e:
        fcp.fcp_span_mask_efficiency(10, [(3, 30)])
    assert e.value.status == fcp.FCP_ERR_INVALID_ARG
