"""Pins for oracle/plan_ref.py: closed-form counts, exact-once coverage of the causal triangle,
plan-driven chunked attention == unchunked attention, and the planner against exhaustive search."""
import itertools
import math

import numpy as np
import pytest

from oracle import attention_ref as A
from oracle import plan_ref as P


@pytest.mark.parametrize("d", range(1, 9))
def test_pairs_cover_causal_chunk_triangle_exactly_once(d):
    seen = {}
    per_rank = {r: 0 for r in range(d)}
    for r in range(d):
        for s in range(d):
            for qc, kc, kind in P.rank_step_pairs(d, r, s):
                assert (qc, kc) not in seen
                seen[(qc, kc)] = kind
                per_rank[r] += 1
                assert qc in (r, 2 * d - 1 - r)                       # a rank only owns its two Q chunks
                j = (r - s) % d
                assert kc in (j, 2 * d - 1 - j)                       # and only sees the visiting rank's KV
    want = {(qc, kc) for qc in range(2 * d) for kc in range(qc + 1)}
    assert set(seen) == want
    assert len(seen) == d * (2 * d + 1)
    assert all(n == 2 * d + 1 for n in per_rank.values())             # load balance across ranks
    assert all((kind == P.DIAG) == (qc == kc) for (qc, kc), kind in seen.items())


@pytest.mark.parametrize("L,d", [(1, 1), (1, 3), (5, 3), (6, 3), (7, 3), (13, 7), (16, 8), (1000, 7),
                                  (131072, 7), (393216, 7), (97, 5)])
def test_chunk_bounds_partition_the_sequence(L, d):
    b = P.chunk_bounds(L, d)
    assert b[0] == 0 and b[-1] == L and len(b) == 2 * d + 1
    lens = np.diff(b)
    assert lens.min() >= 0 and lens.sum() == L
    assert lens.max() - lens.min() <= 1                               # "evenly"
    assert lens.max() == math.ceil(L / (2 * d)) or lens.max() == L // (2 * d)


@pytest.mark.parametrize("d", range(1, 9))
def test_item_and_slot_counts_closed_form(d):
    L = 64 * d + 3
    pl = P.plan_blocks([L], [d])
    assert len(pl["pairs"]) == d * (2 * d + 1)
    assert len(pl["items"]) == d * (d + 1) // 2 + d * d
    n_slots = [cs[0] for cs in pl["chunk_slots"]]
    assert n_slots == [c + 1 if c < d else d for c in range(2 * d)]
    b = P.chunk_bounds(L, d)
    assert pl["n_partial_rows"] == sum(n_slots[c] * (b[c + 1] - b[c]) for c in range(2 * d))
    # items: consecutive, non-overlapping partial row ranges in item order
    row = 0
    for it in pl["items"]:
        assert it[5] == row
        row += b[it[3] + 1] - b[it[3]]
    assert pl["pairs"] == sorted(pl["pairs"]) and [i[:4] for i in pl["items"]] == sorted(i[:4] for i in pl["items"])


def test_short_sequences_drop_empty_chunks():
    pl = P.plan_blocks([1, 2, 5], [3, 2, 4])
    cb, co = pl["chunk_bounds"], pl["chunk_offset"]
    for (b, r, s, qc, kc, kind) in pl["pairs"]:
        assert cb[co[b] + qc + 1] > cb[co[b] + qc] and cb[co[b] + kc + 1] > cb[co[b] + kc]
    # token-pair coverage must still be the full causal triangle of each sequence
    for b, L in enumerate([1, 2, 5]):
        cover = np.zeros((L, L), dtype=int)
        t0 = cb[co[b]]
        for (bb, r, s, qc, kc, kind) in pl["pairs"]:
            if bb != b:
                continue
            q0, q1 = cb[co[b] + qc] - t0, cb[co[b] + qc + 1] - t0
            k0, k1 = cb[co[b] + kc] - t0, cb[co[b] + kc + 1] - t0
            for i in range(q0, q1):
                for j in range(k0, k1):
                    if j <= i:
                        cover[i, j] += 1
                    else:
                        assert kind == P.DIAG
        assert np.array_equal(cover, np.tril(np.ones((L, L), dtype=int)))
    # slots are numbered 0..n-1 without holes per chunk
    for n, rows in pl["chunk_slots"]:
        assert len(rows) == n


@pytest.mark.parametrize("lens,degs", [([37], [1]), ([64, 5, 130], [2, 3, 1]), ([29], [8]), ([97, 3], [5, 2])])
def test_plan_driven_chunked_attention_equals_unchunked(lens, degs):
    """Evaluate every item of the plan as a partial over its KV ranges, merge per Q chunk through the
    slot table, and compare with plain causal attention (pins plan + merge + slot numbering)."""
    rng = np.random.default_rng(21)
    D = 8
    pl = P.plan_blocks(lens, degs)
    cb, co = pl["chunk_bounds"], pl["chunk_offset"]
    T = sum(lens)
    q = rng.standard_normal((T, D)); k = rng.standard_normal((T, D)); v = rng.standard_normal((T, D))
    R = pl["n_partial_rows"]
    o_part = np.full((R, D), np.nan); l_part = np.full(R, np.nan)
    for (b, r, s, qc, slot, row0, n, first) in pl["items"]:
        t0 = cb[co[b]]
        qr = (cb[co[b] + qc] - t0, cb[co[b] + qc + 1] - t0)
        ranges = []
        for (_, _, _, _, kc, kind) in pl["pairs"][first:first + n]:
            ranges.append((cb[co[b] + kc] - t0, cb[co[b] + kc + 1] - t0))
        sl = slice(t0, t0 + lens[b])
        op, lp = A.partial_attention(q[sl], k[sl], v[sl], qr, ranges)
        o_part[row0:row0 + qr[1] - qr[0]] = op
        l_part[row0:row0 + qr[1] - qr[0]] = lp
    assert not np.isnan(o_part).any()
    ci = 0
    for b, d in enumerate(degs):
        t0 = cb[co[b]]
        sl = slice(t0, t0 + lens[b])
        o_ref, l_ref = A.attention_fwd_seq(q[sl], k[sl], v[sl])
        for c in range(2 * d):
            n, rows = pl["chunk_slots"][ci]; ci += 1
            a, e = cb[co[b] + c] - t0, cb[co[b] + c + 1] - t0
            if e == a:
                assert n == 0
                continue
            om, lm = A.merge_partials([o_part[r0:r0 + e - a] for r0 in rows], [l_part[r0:r0 + e - a] for r0 in rows])
            assert np.allclose(om, o_ref[a:e], atol=1e-12) and np.allclose(lm, l_ref[a:e], atol=1e-12)


# ------------------------------------------------------------------------------- strategy planner
COEFFS = [dict(alpha1=1.0, alpha2=0.0, alpha3=0.0, beta1=0.0, beta2=0.0, v=1.0),
          dict(alpha1=1e-3, alpha2=0.7, alpha3=40.0, beta1=5.0, beta2=11.0, v=2.0)]


def test_group_time_closed_forms():
    c = COEFFS[0]
    assert P.group_time([10], [0.0], 1, c) == 100.0
    assert P.group_time([10, 20], [0.0, 1.0], 5, c) == (100.0 + 2 * 400.0) / 5
    c = COEFFS[1]
    # d = 1: no communication; compute = a1 L^2 + a2 L + b1
    assert math.isclose(P.group_time([100], [0.0], 1, c), 1e-3 * 1e4 + 70.0 + 5.0)
    # d = 2: comm = a3 L / v + b2 = 2011, attention compute = 5 -> overlap hides the smaller (5)
    assert math.isclose(P.group_time([100], [0.0], 2, c), (10.0 + 70.0) / 2 + 5.0 + 2011.0 - 5.0)


@pytest.mark.parametrize("coeffs", COEFFS)
def test_dp_matches_exhaustive_search(coeffs):
    rng = np.random.default_rng(5)
    checked = 0
    for trial in range(60):
        K = int(rng.integers(1, 6))
        N = int(rng.integers(K, 11))
        lens = [[int(x) for x in rng.integers(1, 200, size=rng.integers(1, 4))] for _ in range(K)]
        dmin = [int(x) for x in rng.integers(1, 3, size=K)]
        times = [[math.inf] + [P.group_time(l, [0.0] * len(l), d, coeffs) for d in range(1, N + 1)] for l in lens]
        res = P.dp_allocate(times, dmin, N)
        if sum(dmin) > N:
            assert res is None
            continue
        deg, mk = res
        assert sum(deg) == N and all(d >= m for d, m in zip(deg, dmin))
        assert mk == max(times[i][deg[i]] for i in range(K))
        assert mk == P.brute_force_allocate(times, dmin, N)
        checked += 1
    assert checked > 30


def test_single_group_takes_all_ranks_and_equal_groups_split_evenly():
    c = COEFFS[0]
    r = P.plan_strategy([1000], N=7, E=1e9, M_token=1.0, M_ms=0.0, coeffs=c)
    assert r["d_group"] == [7] and r["cp_degree"] == [7]
    # four equal groups that cannot share a bin (budget = one sequence), 12 ranks -> 3 each
    r = P.plan_strategy([500] * 4, N=12, E=500.0, M_token=1.0, M_ms=0.0, coeffs=c)
    assert r["d_group"] == [3, 3, 3, 3] and math.isclose(r["makespan"], 500.0 ** 2 / 3)


def test_bfd_grouping_rules():
    """Hand trace, budget 100 tokens per rank, order 250, 60, 45, 40, 10:
    250 -> opens bin 0 with ceil(2.5) = 3 ranks (headroom 50); 60 does not fit 50 -> opens bin 1
    (headroom 40); 45 fits only bin 0 (-> 5); 40 fits only bin 1 (-> 0); 10 fits nowhere -> bin 2."""
    g, dmin = P.bfd_groups([60, 250, 45, 40, 10], E=100.0, M_token=1.0, M_ms=0.0)
    assert dmin == [3, 1, 1]
    assert g == [1, 0, 0, 1, 2]
    # best fit: 30 fits bins with headroom 50 and 40 -> goes to the tighter one (bin 1)
    g, dmin = P.bfd_groups([250, 60, 30], E=100.0, M_token=1.0, M_ms=0.0)
    assert g == [0, 1, 1] and dmin == [3, 1]
    # model-state memory shrinks the budget: E' = 100 - 50 = 50 -> 250 needs 5 ranks
    g, dmin = P.bfd_groups([250], E=100.0, M_token=1.0, M_ms=50.0)
    assert dmin == [5]


def _golden(name):
    import os
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", name)


def test_case_study_degree_mixes_use_the_whole_rank_budget():
    """Table 6 prints the CP-group mixes of two batches on 32 ranks (tests/golden/case_study_degree_mixes.txt):
    every system spends exactly N ranks, and only FCP mixes degrees, non-powers-of-two among them.  The
    allocator reproduces the invariant on a skewed synthetic batch."""
    rows = [l.split() for l in open(_golden("case_study_degree_mixes.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for system, case, *mix in rows:
        degs = [(int(a), int(b)) for a, b in (m.split("x") for m in mix)]
        assert sum(d * n for d, n in degs) == 32, (system, case)
        assert (len(degs) > 1) == (system == "FCP")
    assert any(d & (d - 1) for s, c, *mix in rows if s == "FCP" for d in (int(m.split("x")[0]) for m in mix))
    rng = np.random.default_rng(3)
    lens = [int(x) for x in np.clip(rng.lognormal(8.0, 1.0, size=20), 256, 131072)]
    r = P.plan_strategy(lens, N=32, E=20000.0, M_token=1.0, M_ms=0.0, coeffs=COEFFS[0])
    assert r is not None and sum(r["d_group"]) == 32
    assert all(d >= m for d, m in zip(r["d_group"], r["d_min"]))
    assert len(set(r["d_group"])) > 1                   # heterogeneous, incl. non-powers-of-two allowed
    assert P.plan_strategy([100000] * 5, N=4, E=1000.0, M_token=1.0, M_ms=0.0, coeffs=COEFFS[0]) is None


def test_stored_plan_tables_match_the_oracle():
    """tests/golden/plan_tables_small.json was written by tests/golden/make_plan_tables.py from this oracle: a
    change in the reading of the plan (bounds, ring steps, slots, row order) shows up here."""
    import json
    for case in json.load(open(_golden("plan_tables_small.json"))):
        ref = P.plan_blocks(case["lens"], case["degs"])
        assert [int(x) for x in ref["chunk_bounds"]] == case["chunk_bounds"]
        assert [[int(v) for v in p] for p in ref["pairs"]] == case["pairs"]
        assert [[int(v) for v in i] for i in ref["items"]] == case["items"]
        assert [[int(n), [int(v) for v in r]] for n, r in ref["chunk_slots"]] == case["chunk_slots"]
        assert int(ref["n_partial_rows"]) == case["n_partial_rows"]
        # closed forms that do not come from the oracle: d(2d+1) pairs for L >= 2d, chunk lengths sum to L
        for b, (L, d) in enumerate(zip(case["lens"], case["degs"])):
            if L >= 2 * d:
                assert sum(1 for p in case["pairs"] if p[0] == b) == d * (2 * d + 1)
