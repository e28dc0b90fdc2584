"""Integer oracle for the context-parallel block plan and the strategy planner.

TEST INFRASTRUCTURE ONLY: never imported by the CUDA/C++ path; the two share no code.

Block plan.  The paper fixes only that a sequence handled with CP degree d is cut evenly along the
sequence dimension (Sec. 4.3, "Memory Estimation") and that d may be any positive integer
(Sec. 4.2).  The construction used here is the load-balanced ring layout of the prior work the
paper builds on (Sec. 3.2): 2d chunks with bounds floor(c*L/(2d)); virtual rank r owns chunks r and
2d-1-r; at ring step s the rank holds the keys/values of rank j = (r - s) mod d and computes every
causally-needed (Q chunk, KV chunk) pair between its own two Q chunks and the two visiting KV
chunks.  One partial output ("slot") is produced per (Q chunk, rank, step).

Strategy planner (Sec. 4.4, Eq. 7, Algorithm 1): best-fit-decreasing grouping under the per-rank
memory budget, then the 2-D dynamic programme over (groups, ranks), written here both as the
algorithm's loops and as an exhaustive search over all degree vectors (tiny inputs) so that the
two can be compared.

Pins: tests/test_oracle_plan.py (exact-once coverage of the causal triangle, pair/item/slot counts
in closed form, brute-force makespan equality, degree sums such as the case-study mixes of
Table 6).
"""
from __future__ import annotations

import itertools
import math

FULL, DIAG = 0, 1


def chunk_bounds(L: int, d: int):
    """b_c = floor(c*L/(2d)), c = 0..2d (sequence-relative)."""
    return [(c * L) // (2 * d) for c in range(2 * d + 1)]


def rank_step_pairs(d: int, r: int, s: int):
    """(q_chunk, kv_chunk, kind) triples virtual rank r computes at ring step s."""
    last = 2 * d - 1
    j = (r - s) % d
    if s == 0:
        return [(r, r, DIAG), (last - r, r, FULL), (last - r, last - r, DIAG)]
    if j < r:
        return [(r, j, FULL), (last - r, j, FULL)]
    return [(last - r, j, FULL), (last - r, last - j, FULL)]


def plan_blocks(seqlens, cp_degrees):
    """Returns a dict of integer tables (lists of tuples) in the canonical row order.

    chunk_bounds : per sequence, packed-token indices of the 2d+1 chunk bounds, concatenated
    chunk_offset : B+1 offsets into chunk_bounds
    pairs        : (seq, rank, step, q_chunk, kv_chunk, kind), sorted lexicographically;
                   pairs with an empty Q or KV chunk are dropped
    items        : (seq, rank, step, q_chunk, slot, part_row0, n_pairs, first_pair); one per
                   (seq, rank, step, q_chunk) that kept at least one pair, same sort order;
                   slot = rank of this step among the steps that touch the q_chunk (ascending
                   step); part_row0 = running sum of the Q-chunk lengths in item order
    chunk_slots  : per (seq, chunk) in order: (n_slots, [part_row0 of slot 0, 1, ...])
    n_partial_rows : total rows of the partial buffers
    """
    cb, coff, pairs, items, chunk_slots = [], [0], [], [], []
    t0 = 0
    for b, (L, d) in enumerate(zip(seqlens, cp_degrees)):
        L, d = int(L), int(d)
        bounds = chunk_bounds(L, d)
        cb.extend(t0 + x for x in bounds)
        coff.append(len(cb))
        seq_pairs = []
        for r in range(d):
            for s in range(d):
                for (qc, kc, kind) in rank_step_pairs(d, r, s):
                    if bounds[qc + 1] > bounds[qc] and bounds[kc + 1] > bounds[kc]:
                        seq_pairs.append((b, r, s, qc, kc, kind))
        seq_pairs.sort()
        pairs.extend(seq_pairs)
        t0 += L
    # items
    row = 0
    per_chunk_steps = {}
    i = 0
    while i < len(pairs):
        b, r, s, qc = pairs[i][:4]
        n = 1
        while i + n < len(pairs) and pairs[i + n][:4] == (b, r, s, qc):
            n += 1
        per_chunk_steps.setdefault((b, qc), []).append(s)
        items.append([b, r, s, qc, None, None, n, i])
        i += n
    for it in items:
        b, r, s, qc = it[:4]
        it[4] = sorted(per_chunk_steps[(b, qc)]).index(s)
        it[5] = row
        lo = cb[coff[b] + qc]
        hi = cb[coff[b] + qc + 1]
        row += hi - lo
    items = [tuple(it) for it in items]
    by_chunk = {}
    for it in items:
        by_chunk.setdefault((it[0], it[3]), {})[it[4]] = it[5]
    for b, d in enumerate(cp_degrees):
        for c in range(2 * int(d)):
            slots = by_chunk.get((b, c), {})
            chunk_slots.append((len(slots), [slots[k] for k in range(len(slots))]))
    return dict(chunk_bounds=cb, chunk_offset=coff, pairs=pairs, items=items,
                chunk_slots=chunk_slots, n_partial_rows=row)


def span_tables(seqlens, cp_degrees, spans_per_seq):
    """Integer tables of a plan whose sequences carry bidirectional spans (a query inside a span
    [a, b) also sees the later keys of its span; Sec. 4.3 motivates the mask efficiency factor eta
    with such tokens).  Positions in `spans_per_seq` are sequence-relative; the tables are packed.

    row_limit[t]   : first key (packed index) that query t does not see: t + 1, or its span's end
    first_query[t] : first query (packed index) that sees key t: t, or its span's begin
    span_pairs     : (seq, rank, step, q_chunk, kv_chunk) with kv_chunk > q_chunk, sorted: the block
                     pairs above the chunk diagonal in which some query sees some key.  The ring
                     hands every rank every KV chunk within its d steps: the rank that owns q_chunk
                     computes such a pair at the step at which the owner of kv_chunk visits.
    """
    row_limit, first_query, span_pairs = [], [], []
    t0 = 0
    for b, (L, d) in enumerate(zip(seqlens, cp_degrees)):
        L, d = int(L), int(d)
        lim = [t0 + i + 1 for i in range(L)]
        fq = [t0 + i for i in range(L)]
        for (a, e) in spans_per_seq[b]:
            for i in range(a, e):
                lim[i] = t0 + e
                fq[i] = t0 + a
        row_limit.extend(lim)
        first_query.extend(fq)
        bounds = chunk_bounds(L, d)
        owner = lambda c: c if c < d else 2 * d - 1 - c
        for qc in range(2 * d):
            for kc in range(qc + 1, 2 * d):
                # some row of q_chunk sees some key of kv_chunk: a span reaches from one into the other
                if any(max(a, bounds[qc]) < min(e, bounds[qc + 1]) and max(a, bounds[kc]) < min(e, bounds[kc + 1])
                       for (a, e) in spans_per_seq[b]):
                    r = owner(qc)
                    span_pairs.append((b, r, (r - owner(kc)) % d, qc, kc))
        t0 += L
    span_pairs.sort()
    return dict(row_limit=row_limit, first_query=first_query, span_pairs=span_pairs)


# ---------------------------------------------------------------------------------------------
# strategy planner
# ---------------------------------------------------------------------------------------------
def group_time(lens, etas, d, coeffs):
    """T(G, d) of Eq. 6 with the per-rank reading of Eqs. 4-5: the compute terms of a group are
    shared by its d ranks; ring communication exists only when d > 1."""
    a1, a2, a3, b1, b2, v = (coeffs[k] for k in ("alpha1", "alpha2", "alpha3", "beta1", "beta2", "v"))
    quad = 0.0
    lin = 0.0
    tot = 0.0
    for L, eta in zip(lens, etas):
        quad += a1 * (1.0 + eta) * float(L) * float(L)
        lin += a2 * float(L)
        tot += float(L)
    t_cpa = quad / d
    t_cp = (quad + lin) / d + b1
    t_cm = (a3 * tot) / v + b2 if d > 1 else 0.0
    t_cma = t_cm
    return t_cp + t_cm - min(t_cpa, t_cma)


def bfd_groups(seqlens, E, M_token, M_ms):
    """Stage 1: best-fit-decreasing.  Returns (group_of[B], d_min[K'])."""
    cap1 = E - M_ms
    order = sorted(range(len(seqlens)), key=lambda i: (-int(seqlens[i]), i))
    head, dmin = [], []
    group_of = [0] * len(seqlens)
    for i in order:
        need = float(seqlens[i]) * M_token
        best = -1
        for gidx, room in enumerate(head):
            if room >= need and (best < 0 or room < head[best]):
                best = gidx
        if best < 0:
            dm = max(1, int(math.ceil(need / cap1)))
            head.append(dm * cap1 - need)
            dmin.append(dm)
            best = len(head) - 1
        else:
            head[best] -= need
        group_of[i] = best
    return group_of, dmin


def dp_allocate(times, dmin, N):
    """Stage 2 (Algorithm 1).  times[k][d] = T(G_k, d) for d in 0..N (index 0 unused).
    Returns (degrees, makespan) or None if sum(dmin) > N."""
    K = len(dmin)
    if sum(dmin) > N:
        return None
    INF = math.inf
    DP = [[INF] * (N + 1) for _ in range(K + 1)]
    path = [[0] * (N + 1) for _ in range(K + 1)]
    DP[0][0] = 0.0
    for k in range(1, K + 1):
        before = sum(dmin[: k - 1])
        remain = sum(dmin[k:])
        for j in range(before + dmin[k - 1], N - remain + 1):
            for d in range(dmin[k - 1], j - before + 1):
                cost = max(DP[k - 1][j - d], times[k - 1][d])
                if cost < DP[k][j]:
                    DP[k][j] = cost
                    path[k][j] = d
    deg = [0] * K
    p, qq = K, N
    while p > 0:
        deg[p - 1] = path[p][qq]
        qq -= deg[p - 1]
        p -= 1
    return deg, DP[K][N]


def brute_force_allocate(times, dmin, N):
    """Exhaustive minimum makespan over all degree vectors with d_k >= dmin_k and sum d_k = N."""
    K = len(dmin)
    best = math.inf
    for deg in itertools.product(*[range(dmin[k], N + 1) for k in range(K)]):
        if sum(deg) != N:
            continue
        best = min(best, max(times[k][deg[k]] for k in range(K)))
    return best


def plan_strategy(seqlens, N, E, M_token, M_ms, coeffs, etas=None):
    """Both stages.  Returns dict(group_of, d_group, cp_degree, makespan) or None if infeasible."""
    etas = [0.0] * len(seqlens) if etas is None else list(etas)
    group_of, dmin = bfd_groups(seqlens, E, M_token, M_ms)
    K = len(dmin)
    members = [[i for i in range(len(seqlens)) if group_of[i] == g] for g in range(K)]
    times = [[math.inf] + [group_time([seqlens[i] for i in m], [etas[i] for i in m], d, coeffs)
                           for d in range(1, N + 1)] for m in members]
    res = dp_allocate(times, dmin, N)
    if res is None:
        return None
    deg, makespan = res
    return dict(group_of=group_of, d_group=deg, d_min=dmin, cp_degree=[deg[g] for g in group_of],
                makespan=makespan, times=times)
