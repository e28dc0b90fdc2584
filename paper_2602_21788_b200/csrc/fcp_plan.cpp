// Host side of libfcp: the strategy planner (Sec. 4.4, Eq. 7, Algorithm 1) and the block plan that
// the kernels consume.  Plain C++, integers and doubles only; nothing here touches the GPU.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <limits>
#include <numeric>
#include <vector>

#include "fcp_plan.hpp"

namespace {
thread_local char g_err[512] = "";
}

void fcp_set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
}

extern "C" const char* fcp_last_error_message(void) { return g_err; }

extern "C" const char* fcp_status_string(int status) {
  switch (status) {
    case FCP_OK: return "FCP_OK";
    case FCP_ERR_INVALID_ARG: return "FCP_ERR_INVALID_ARG";
    case FCP_ERR_INFEASIBLE: return "FCP_ERR_INFEASIBLE";
    case FCP_ERR_UNSUPPORTED: return "FCP_ERR_UNSUPPORTED";
    case FCP_ERR_WORKSPACE: return "FCP_ERR_WORKSPACE";
    case FCP_ERR_CUDA: return "FCP_ERR_CUDA";
    case FCP_ERR_TIMEOUT: return "FCP_ERR_TIMEOUT";
    case FCP_ERR_NOT_UPLOADED: return "FCP_ERR_NOT_UPLOADED";
    default: return "FCP_ERR_UNKNOWN";
  }
}

// ---------------------------------------------------------------------------------------------
// Strategy planner
// ---------------------------------------------------------------------------------------------
namespace {

struct GroupSums {  // sums over the sequences of one atomic group
  double quad = 0.0, lin = 0.0, tot = 0.0;
};

// T(G, d), Eq. 6: T_cp + T_cm - min(T_cpa, T_cma).  Eqs. 4-5 are written per group; the d ranks of
// a group share the compute terms, and ring communication only exists for d > 1.
double group_time(const GroupSums& g, int d, const fcp_cost_coeffs& c) {
  const double t_cpa = g.quad / d;
  const double t_cp = (g.quad + g.lin) / d + c.beta1;
  const double t_cm = d > 1 ? (c.alpha3 * g.tot) / c.v + c.beta2 : 0.0;
  const double t_cma = t_cm;
  return t_cp + t_cm - std::min(t_cpa, t_cma);
}

}  // namespace

extern "C" int fcp_plan_strategy(const int32_t* seqlens, int32_t B, int32_t N, double E,
                                 double M_token, double M_ms, const fcp_cost_coeffs* coeffs,
                                 int32_t* group_of, int32_t* cp_degree, int32_t* n_groups,
                                 double* makespan) {
  if (!seqlens || !coeffs || B <= 0 || N <= 0 || !(E > M_ms) || !(M_token > 0.0) || !(coeffs->v > 0.0)) {
    fcp_set_error("fcp_plan_strategy: invalid argument");
    return FCP_ERR_INVALID_ARG;
  }
  if (N > FCP_MAX_DEGREE) {
    fcp_set_error("fcp_plan_strategy: N=%d exceeds FCP_MAX_DEGREE=%d", N, FCP_MAX_DEGREE);
    return FCP_ERR_UNSUPPORTED;
  }
  for (int i = 0; i < B; ++i)
    if (seqlens[i] <= 0) {
      fcp_set_error("fcp_plan_strategy: seqlens[%d]=%d", i, seqlens[i]);
      return FCP_ERR_INVALID_ARG;
    }

  // Stage 1: best-fit-decreasing.  Longest first (ties: lower index); a sequence goes to the open
  // group with the least remaining headroom that still holds it (ties: lowest group), otherwise it
  // opens a group of d_min = ceil(need / budget) ranks.
  const double budget = E - M_ms;
  std::vector<int> order(B);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return seqlens[a] > seqlens[b]; });
  std::vector<double> headroom;
  std::vector<int> dmin;
  std::vector<int> gof(B, 0);
  for (int i : order) {
    const double need = double(seqlens[i]) * M_token;
    int best = -1;
    for (int g = 0; g < (int)headroom.size(); ++g)
      if (headroom[g] >= need && (best < 0 || headroom[g] < headroom[best])) best = g;
    if (best < 0) {
      const int dm = std::max(1, (int)std::ceil(need / budget));
      headroom.push_back(dm * budget - need);
      dmin.push_back(dm);
      best = (int)headroom.size() - 1;
    } else {
      headroom[best] -= need;
    }
    gof[i] = best;
  }
  const int K = (int)dmin.size();
  long long need_ranks = 0;
  for (int d : dmin) need_ranks += d;
  if (need_ranks > N) {
    fcp_set_error("fcp_plan_strategy: minimum degrees need %lld ranks, only %d available", need_ranks, N);
    return FCP_ERR_INFEASIBLE;
  }

  // Per-group sums in sequence-index order.
  std::vector<GroupSums> sums(K);
  for (int i = 0; i < B; ++i) {
    const double L = double(seqlens[i]);
    const double eta = coeffs->eta ? coeffs->eta[i] : 0.0;
    GroupSums& g = sums[gof[i]];
    g.quad += coeffs->alpha1 * (1.0 + eta) * L * L;
    g.lin += coeffs->alpha2 * L;
    g.tot += L;
  }

  // Stage 2: the recurrence of Eq. 7, best[k][j] = min over d of max(best[k-1][j-d], T(G_k, d)), kept as two
  // rolling rows over j plus the arg-min of every (group, j) cell for the walk back.  A cell (k, j) is
  // reachable when the first k groups can have their minimum degrees (j >= lo[k]) and the remaining ones
  // still get theirs (j <= N - (need - lo[k])); d ranges over [d_min, j - lo[k-1]].  Ties keep the smallest
  // d (strict comparison, d ascending).  The answer is read at j = N: the strategy hands out every rank, as
  // the paper's text does ("backtrack from DP[K'][N]"; its case-study mixes add up to the rank count).
  // Because T(G, d) is not monotone in d once the ring term appears at d = 2, a plan that leaves ranks
  // idle could have a smaller makespan; that variant (min over j <= N) is not what the paper runs.
  const double INF = std::numeric_limits<double>::infinity();
  std::vector<int> lo(K + 1, 0);                 // lo[k] = sum of d_min over the first k groups
  for (int k = 0; k < K; ++k) lo[k + 1] = lo[k] + dmin[k];
  std::vector<double> prev(N + 1, INF), cur(N + 1, INF);
  std::vector<int> choice((size_t)K * (N + 1), 0);
  std::vector<double> tg(N + 1, 0.0);            // T(G_k, d) for the group at hand
  prev[0] = 0.0;
  for (int k = 0; k < K; ++k) {
    const int j_hi = N - ((int)need_ranks - lo[k + 1]);
    for (int d = dmin[k]; d <= j_hi - lo[k]; ++d) tg[d] = group_time(sums[k], d, *coeffs);
    std::fill(cur.begin(), cur.end(), INF);
    for (int j = lo[k + 1]; j <= j_hi; ++j) {
      double best = INF;
      int arg = 0;
      for (int d = dmin[k]; d <= j - lo[k]; ++d) {
        const double cand = std::max(prev[j - d], tg[d]);
        if (cand < best) {
          best = cand;
          arg = d;
        }
      }
      cur[j] = best;
      choice[(size_t)k * (N + 1) + j] = arg;
    }
    prev.swap(cur);
  }
  const double best_makespan = prev[N];
  std::vector<int> deg(K, 0);
  for (int k = K - 1, j = N; k >= 0; --k) {
    deg[k] = choice[(size_t)k * (N + 1) + j];
    j -= deg[k];
  }
  for (int i = 0; i < B; ++i) {
    if (group_of) group_of[i] = gof[i];
    if (cp_degree) cp_degree[i] = deg[gof[i]];
  }
  if (n_groups) *n_groups = K;
  if (makespan) *makespan = best_makespan;
  return FCP_OK;
}

// ---------------------------------------------------------------------------------------------
// Block plan
// ---------------------------------------------------------------------------------------------
namespace {

struct Pair {
  int32_t seq, rank, step, qc, kc, kind;
  bool operator<(const Pair& o) const {
    if (rank != o.rank) return rank < o.rank;
    if (step != o.step) return step < o.step;
    if (qc != o.qc) return qc < o.qc;
    return kc < o.kc;
  }
};

inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }

}  // namespace

extern "C" int fcp_plan_blocks(const int32_t* seqlens, const int32_t* cp_degrees, int32_t B,
                               const fcp_params* params, fcp_plan** out) {
  return fcp_plan_blocks_spans(seqlens, cp_degrees, B, nullptr, nullptr, params, out);
}

extern "C" int fcp_plan_blocks_spans(const int32_t* seqlens, const int32_t* cp_degrees, int32_t B,
                                     const int32_t* span_offset, const int32_t* spans,
                                     const fcp_params* params, fcp_plan** out) {
  if (!seqlens || !cp_degrees || !params || !out || B <= 0 || (span_offset && !spans && span_offset[B] > 0)) {
    fcp_set_error("fcp_plan_blocks: invalid argument");
    return FCP_ERR_INVALID_ARG;
  }
  *out = nullptr;
  if ((params->head_dim != 64 && params->head_dim != 128) || params->hq <= 0 || params->hkv <= 0 ||
      params->hq % params->hkv != 0) {
    fcp_set_error("fcp_plan_blocks: unsupported shape hq=%d hkv=%d head_dim=%d", params->hq, params->hkv,
                  params->head_dim);
    return FCP_ERR_UNSUPPORTED;
  }
  int64_t T = 0;
  int32_t max_len = 0;
  for (int b = 0; b < B; ++b) {
    if (seqlens[b] <= 0 || cp_degrees[b] <= 0) {
      fcp_set_error("fcp_plan_blocks: sequence %d has length %d, degree %d", b, seqlens[b], cp_degrees[b]);
      return FCP_ERR_INVALID_ARG;
    }
    if (cp_degrees[b] > FCP_MAX_DEGREE) {
      fcp_set_error("fcp_plan_blocks: degree %d > FCP_MAX_DEGREE", cp_degrees[b]);
      return FCP_ERR_UNSUPPORTED;
    }
    T += seqlens[b];
    max_len = std::max(max_len, seqlens[b]);
  }
  if (T >= (int64_t(1) << 31) - 2 * FCP_FWD_UNIT_ROWS) {
    fcp_set_error("fcp_plan_blocks: %lld tokens exceed the 2^31 limit", (long long)T);
    return FCP_ERR_INVALID_ARG;
  }

  fcp_plan* p = new fcp_plan();
  p->params = *params;
  if (!(p->params.scale > 0.f)) p->params.scale = 1.0f / std::sqrt((float)params->head_dim);
  p->B = B;
  p->T = T;
  p->max_seqlen = max_len;
  p->cu_seqlens.assign(B + 1, 0);
  for (int b = 0; b < B; ++b) p->cu_seqlens[b + 1] = p->cu_seqlens[b] + seqlens[b];

  // Bidirectional spans: query t sees the keys before row_limit[t]; key t is seen from query
  // first_query[t] on (both in packed-token indices, both non-decreasing within a sequence).
  const bool has_spans = span_offset != nullptr && span_offset[B] > span_offset[0];
  if (has_spans) {
    p->span_offset.assign(span_offset, span_offset + B + 1);
    p->spans.assign(spans, spans + 2 * (size_t)span_offset[B]);
    p->row_limit.resize(T);
    p->first_query.resize(T);
    for (int64_t t = 0; t < T; ++t) {
      p->row_limit[t] = (int32_t)t + 1;
      p->first_query[t] = (int32_t)t;
    }
    for (int b = 0; b < B; ++b) {
      int32_t prev_end = 0;
      if (span_offset[b + 1] < span_offset[b]) {
        delete p;
        fcp_set_error("fcp_plan_blocks_spans: span_offset decreases at sequence %d", b);
        return FCP_ERR_INVALID_ARG;
      }
      for (int32_t i = span_offset[b]; i < span_offset[b + 1]; ++i) {
        const int32_t a = spans[2 * i], e = spans[2 * i + 1];
        if (a < prev_end || e <= a || e > seqlens[b]) {
          delete p;
          fcp_set_error("fcp_plan_blocks_spans: span [%d, %d) of sequence %d (length %d) is empty, out of range, "
                        "unsorted or overlaps the one before", a, e, b, seqlens[b]);
          return FCP_ERR_INVALID_ARG;
        }
        prev_end = e;
        const int32_t t0 = p->cu_seqlens[b];
        for (int32_t t = a; t < e; ++t) {
          p->row_limit[t0 + t] = t0 + e;
          p->first_query[t0 + t] = t0 + a;
        }
      }
    }
  }

  // Chunk bounds and pairs.
  p->chunk_offset.push_back(0);
  std::vector<Pair> pairs;
  for (int b = 0; b < B; ++b) {
    const int64_t L = seqlens[b];
    const int d = cp_degrees[b];
    const int32_t t0 = p->cu_seqlens[b];
    const size_t base = p->chunk_bounds.size();
    for (int c = 0; c <= 2 * d; ++c) p->chunk_bounds.push_back(t0 + (int32_t)((int64_t)c * L / (2 * d)));
    p->chunk_offset.push_back((int32_t)p->chunk_bounds.size());
    auto nonempty = [&](int c) { return p->chunk_bounds[base + c + 1] > p->chunk_bounds[base + c]; };
    std::vector<Pair> sp;
    auto add = [&](int r, int s, int qc, int kc) {
      if (nonempty(qc) && nonempty(kc)) sp.push_back(Pair{b, r, s, qc, kc, qc == kc ? 1 : 0});
    };
    const int last = 2 * d - 1;
    for (int r = 0; r < d; ++r)
      for (int s = 0; s < d; ++s) {
        const int j = ((r - s) % d + d) % d;   // rank whose K/V visits at this ring step
        if (s == 0) {
          add(r, s, r, r);
          add(r, s, last - r, r);
          add(r, s, last - r, last - r);
        } else if (j < r) {
          add(r, s, r, j);
          add(r, s, last - r, j);
        } else {
          add(r, s, last - r, j);
          add(r, s, last - r, last - j);
        }
      }
    std::sort(sp.begin(), sp.end());
    pairs.insert(pairs.end(), sp.begin(), sp.end());
  }
  for (const Pair& x : pairs) {
    const int32_t row[6] = {x.seq, x.rank, x.step, x.qc, x.kc, x.kind};
    p->pairs.insert(p->pairs.end(), row, row + 6);
  }
  // Block pairs above the chunk diagonal that a span makes necessary: (q_chunk, kv_chunk > q_chunk) such that
  // a span reaches into both.  The rank that owns q_chunk computes it when the owner of kv_chunk visits.
  if (has_spans) {
    for (int b = 0; b < B; ++b) {
      const int d = cp_degrees[b];
      const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
      const int32_t t0 = cbp[0];
      std::vector<Pair> sp;
      auto owner = [&](int c) { return c < d ? c : 2 * d - 1 - c; };
      for (int qc = 0; qc < 2 * d; ++qc)
        for (int kc = qc + 1; kc < 2 * d; ++kc) {
          bool hit = false;
          for (int32_t i = span_offset[b]; i < span_offset[b + 1] && !hit; ++i) {
            const int32_t a = t0 + spans[2 * i], e = t0 + spans[2 * i + 1];
            hit = std::max(a, cbp[qc]) < std::min(e, cbp[qc + 1]) && std::max(a, cbp[kc]) < std::min(e, cbp[kc + 1]);
          }
          if (hit) {
            const int r = owner(qc);
            sp.push_back(Pair{b, r, ((r - owner(kc)) % d + d) % d, qc, kc, 2});
          }
        }
      std::sort(sp.begin(), sp.end());
      for (const Pair& x : sp) {
        const int32_t row[5] = {x.seq, x.rank, x.step, x.qc, x.kc};
        p->span_pairs.insert(p->span_pairs.end(), row, row + 5);
      }
    }
  }

  // Items: one per (seq, rank, step, q_chunk); slot = order of the step among the steps touching
  // that Q chunk; partial rows are laid out in item order.
  const int n_chunks_total = p->chunk_offset[B] - B;  // sum of 2d
  std::vector<int32_t> chunk_index0(B + 1, 0);        // global chunk index of chunk 0 of each sequence
  for (int b = 0; b < B; ++b) chunk_index0[b + 1] = chunk_index0[b] + 2 * cp_degrees[b];
  std::vector<std::vector<std::pair<int, int>>> chunk_items(n_chunks_total);  // (step, item index)
  int64_t row = 0;
  for (size_t i = 0; i < pairs.size();) {
    size_t n = 1;
    while (i + n < pairs.size() && pairs[i + n].seq == pairs[i].seq && pairs[i + n].rank == pairs[i].rank &&
           pairs[i + n].step == pairs[i].step && pairs[i + n].qc == pairs[i].qc)
      ++n;
    const Pair& x = pairs[i];
    const int item = (int)(p->items.size() / 8);
    const int32_t cb = p->chunk_offset[x.seq] + x.qc;
    const int32_t len = p->chunk_bounds[cb + 1] - p->chunk_bounds[cb];
    const int32_t rowv[8] = {x.seq, x.rank, x.step, x.qc, 0, (int32_t)row, (int32_t)n, (int32_t)i};
    p->items.insert(p->items.end(), rowv, rowv + 8);
    chunk_items[chunk_index0[x.seq] + x.qc].push_back({x.step, item});
    row += len;
    if (row >= (int64_t(1) << 31) - 2 * FCP_FWD_UNIT_ROWS) {
      delete p;
      fcp_set_error("fcp_plan_blocks: partial rows exceed the 2^31 limit");
      return FCP_ERR_INVALID_ARG;
    }
    i += n;
  }
  p->R = row;
  p->slot_offset.push_back(0);
  for (int c = 0; c < n_chunks_total; ++c) {
    auto& v = chunk_items[c];
    std::sort(v.begin(), v.end());
    for (size_t k = 0; k < v.size(); ++k) {
      p->items[(size_t)v[k].second * 8 + 4] = (int32_t)k;
      p->slot_rows.push_back(p->items[(size_t)v[k].second * 8 + 5]);
    }
    p->slot_offset.push_back((int32_t)p->slot_rows.size());
  }

  // ---- derived work lists (execution order; not part of the canonical tables) ----
  // Forward: an item's Q chunk is cut into units of two adjacent 128-row tiles.  KV ranges of an
  // item are its pairs in kv_chunk order, so a DIAG range (kv_chunk == q_chunk) is always last.
  struct FU { int32_t f[FCP_FWD_UNIT_W]; };
  std::vector<FU> fus;
  const int n_items = (int)(p->items.size() / 8);
  for (int it = 0; it < n_items; ++it) {
    const int32_t* I = &p->items[(size_t)it * 8];
    const int b = I[0], qc = I[3], np = I[6], fp = I[7];
    const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
    const int32_t q0 = cbp[qc], q1 = cbp[qc + 1];
    int32_t kb[2] = {0, 0}, ke[2] = {0, 0}, kd[2] = {0, 0};
    for (int r = 0; r < np; ++r) {
      const Pair& x = pairs[fp + r];
      kb[r] = cbp[x.kc];
      ke[r] = cbp[x.kc + 1];
      kd[r] = x.kind;
    }
    const int last = np - 1;
    const int nt_first = np == 2 ? ceil_div(ke[0] - kb[0], FCP_TILE) : 0;
    for (int32_t off = 0; off < q1 - q0; off += FCP_FWD_UNIT_ROWS) {
      FU u{};
      const int32_t rows = std::min<int32_t>(FCP_FWD_UNIT_ROWS, q1 - q0 - off);
      u.f[FU_Q_ROW0] = q0 + off;
      u.f[FU_Q_ROWS] = rows;
      u.f[FU_PART_ROW0] = I[5] + off;
      u.f[FU_N_RANGES] = np;
      u.f[FU_KV0_BEGIN] = kb[0]; u.f[FU_KV0_END] = ke[0]; u.f[FU_KV0_DIAG] = kd[0];
      u.f[FU_KV1_BEGIN] = kb[1]; u.f[FU_KV1_END] = ke[1]; u.f[FU_KV1_DIAG] = kd[1];
      for (int s = 0; s < 2; ++s) {
        const int32_t rs = std::min<int32_t>(FCP_TILE, rows - s * FCP_TILE);
        int nt = 0;
        if (rs > 0) {
          if (kd[last]) nt = ceil_div((int64_t)off + s * FCP_TILE + rs, FCP_TILE);  // keys up to the last row
          else nt = ceil_div(ke[last] - kb[last], FCP_TILE);
          nt += nt_first;
        }
        u.f[FU_NT_STAGE0 + s] = nt;
      }
      u.f[FU_NT_RANGE0] = np == 2 ? nt_first : 0x7fffffff;
      u.f[FU_ITEM] = it;
      {
        const int ci = chunk_index0[b] + qc;   // a Q chunk with one slot needs no merge
        u.f[FU_SINGLE_SLOT] = p->slot_offset[ci + 1] - p->slot_offset[ci] == 1;
      }
      fus.push_back(u);
    }
  }
  std::stable_sort(fus.begin(), fus.end(), [](const FU& a, const FU& b) {
    return a.f[FU_NT_STAGE0] + a.f[FU_NT_STAGE1] > b.f[FU_NT_STAGE0] + b.f[FU_NT_STAGE1];
  });
  p->fwd_units.reserve(fus.size() * FCP_FWD_UNIT_W);
  for (const FU& u : fus) p->fwd_units.insert(p->fwd_units.end(), u.f, u.f + FCP_FWD_UNIT_W);

  // Fused forward (merge on the fly): all items of a Q chunk run on one CTA, so the KV ranges of the
  // chunk's block pairs are swept in one online softmax and no partial leaves the SM.  The ranges of
  // a Q chunk are its pairs in kv_chunk order with adjacent FULL ranges joined.  In a causal plan
  // that is the prefix [sequence start, chunk start) plus the DIAG range of the chunk itself, which
  // one DIAG range starting at the sequence start describes exactly (every key before the chunk
  // precedes every row of it); consecutive Q chunks of that form are joined into one run of rows,
  // tiled in units of two Q tiles from the start of the run, so no tile is cut at a chunk edge.
  struct Range { int32_t b, e, diag; };
  std::vector<std::vector<Range>> q_cover(n_chunks_total);   // per Q chunk: joined KV ranges of its pairs
  {
    std::vector<std::vector<std::pair<int, int>>> by_q(n_chunks_total);   // (kv_chunk, kind)
    for (const Pair& x : pairs) by_q[chunk_index0[x.seq] + x.qc].push_back({x.kc, x.kind});
    for (int b = 0; b < B; ++b) {
      const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
      for (int c = 0; c < 2 * cp_degrees[b]; ++c) {
        auto& v = by_q[chunk_index0[b] + c];
        std::sort(v.begin(), v.end());
        auto& out_r = q_cover[chunk_index0[b] + c];
        for (auto& kk : v) {
          const Range r{cbp[kk.first], cbp[kk.first + 1], kk.second};
          if (!out_r.empty() && !out_r.back().diag && !r.diag && out_r.back().e == r.b) out_r.back().e = r.e;
          else out_r.push_back(r);
        }
      }
    }
  }
  {
    std::vector<FU> gus;
    // rows [r0, r1) of the sequence [t0, t1) attend to [t0, row] (and, inside a span, on to the span's end)
    auto emit_run = [&](int32_t t0, int32_t t1, int32_t r0, int32_t r1) {
      for (int32_t off = 0; off < r1 - r0; off += FCP_FWD_UNIT_ROWS) {
        FU u{};
        const int32_t rows = std::min<int32_t>(FCP_FWD_UNIT_ROWS, r1 - r0 - off);
        u.f[FU_Q_ROW0] = r0 + off;
        u.f[FU_Q_ROWS] = rows;
        u.f[FU_N_RANGES] = 1;
        u.f[FU_KV0_BEGIN] = t0; u.f[FU_KV0_END] = has_spans ? t1 : r1; u.f[FU_KV0_DIAG] = 1;
        for (int s = 0; s < 2; ++s) {
          const int32_t rs = std::min<int32_t>(FCP_TILE, rows - s * FCP_TILE);
          // key tiles up to the last key the stage's last row sees (row limits do not decrease along a sequence)
          const int32_t last_row = r0 + off + s * FCP_TILE + rs - 1;
          const int32_t key_end = rs > 0 ? (has_spans ? p->row_limit[last_row] : last_row + 1) : t0;
          u.f[FU_NT_STAGE0 + s] = rs > 0 ? ceil_div(key_end - t0, FCP_TILE) : 0;
        }
        u.f[FU_NT_RANGE0] = 0x7fffffff;
        u.f[FU_ITEM] = -1;
        u.f[FU_SINGLE_SLOT] = 1;
        gus.push_back(u);
      }
    };
    for (int b = 0; b < B; ++b) {
      const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
      const int32_t t0 = cbp[0], t1 = cbp[2 * cp_degrees[b]];
      int32_t run0 = -1, run1 = -1;
      for (int c = 0; c < 2 * cp_degrees[b]; ++c) {
        const int32_t q0 = cbp[c], q1 = cbp[c + 1];
        if (q1 == q0) continue;
        const auto& rg = q_cover[chunk_index0[b] + c];
        const bool prefix = (rg.size() == 1 && rg[0].diag && rg[0].b == q0 && q0 == t0) ||
                            (rg.size() == 2 && !rg[0].diag && rg[0].b == t0 && rg[0].e == q0 && rg[1].diag && rg[1].b == q0);
        if (prefix) {
          if (run0 < 0) run0 = q0;
          else if (run1 != q0) { emit_run(t0, t1, run0, run1); run0 = q0; }
          run1 = q1;
          continue;
        }
        if (run0 >= 0) { emit_run(t0, t1, run0, run1); run0 = -1; }
        // a chunk whose ranges are not a causal prefix keeps them as they are (at most two per unit)
        if (rg.empty() || rg.size() > 2 || has_spans) {
          delete p;
          fcp_set_error("fcp_plan_blocks: Q chunk %d of sequence %d has %d disjoint KV ranges", c, b, (int)rg.size());
          return FCP_ERR_UNSUPPORTED;
        }
        const int lastr = (int)rg.size() - 1;
        const int nt_first = rg.size() == 2 ? ceil_div(rg[0].e - rg[0].b, FCP_TILE) : 0;
        for (int32_t off = 0; off < q1 - q0; off += FCP_FWD_UNIT_ROWS) {
          FU u{};
          const int32_t rows = std::min<int32_t>(FCP_FWD_UNIT_ROWS, q1 - q0 - off);
          u.f[FU_Q_ROW0] = q0 + off;
          u.f[FU_Q_ROWS] = rows;
          u.f[FU_N_RANGES] = (int32_t)rg.size();
          u.f[FU_KV0_BEGIN] = rg[0].b; u.f[FU_KV0_END] = rg[0].e; u.f[FU_KV0_DIAG] = rg[0].diag;
          if (rg.size() == 2) { u.f[FU_KV1_BEGIN] = rg[1].b; u.f[FU_KV1_END] = rg[1].e; u.f[FU_KV1_DIAG] = rg[1].diag; }
          for (int s = 0; s < 2; ++s) {
            const int32_t rs = std::min<int32_t>(FCP_TILE, rows - s * FCP_TILE);
            int nt = 0;
            if (rs > 0)
              nt = nt_first + (rg[lastr].diag ? ceil_div((int64_t)(q0 + off - rg[lastr].b) + s * FCP_TILE + rs, FCP_TILE)
                                              : ceil_div(rg[lastr].e - rg[lastr].b, FCP_TILE));
            u.f[FU_NT_STAGE0 + s] = nt;
          }
          u.f[FU_NT_RANGE0] = rg.size() == 2 ? nt_first : 0x7fffffff;
          u.f[FU_ITEM] = -1;
          u.f[FU_SINGLE_SLOT] = 1;
          gus.push_back(u);
        }
      }
      if (run0 >= 0) emit_run(t0, t1, run0, run1);
    }
    std::stable_sort(gus.begin(), gus.end(), [](const FU& a, const FU& b) {
      return a.f[FU_NT_STAGE0] + a.f[FU_NT_STAGE1] > b.f[FU_NT_STAGE0] + b.f[FU_NT_STAGE1];
    });
    p->fused_units.reserve(gus.size() * FCP_FWD_UNIT_W);
    for (const FU& u : gus) p->fused_units.insert(p->fused_units.end(), u.f, u.f + FCP_FWD_UNIT_W);
  }

  // Backward: one unit per 128-key tile; it visits the Q rows of all block pairs whose kv_chunk holds
  // its keys (q_chunk >= kv_chunk), the DIAG pair from its own tile on.  The Q ranges of a KV chunk
  // are its pairs in q_chunk order with adjacent ranges joined (a DIAG range followed by the FULL
  // ranges of the later chunks is one DIAG range up to their end).  When every KV chunk of a sequence
  // ends up with the single range [chunk start, sequence end) DIAG -- the causal plan -- the key
  // tiles are cut from the start of the sequence instead of from each chunk start (a key tile may
  // then span two KV chunks; the causal mask only depends on token positions), so that neither key
  // tiles nor query tiles are cut at chunk edges.
  struct BU { int32_t f[FCP_BWD_UNIT_W]; };
  std::vector<BU> bus;
  {
    std::vector<std::vector<std::pair<int, int>>> by_kv(n_chunks_total);  // (q_chunk, kind)
    for (const Pair& x : pairs) by_kv[chunk_index0[x.seq] + x.kc].push_back({x.qc, x.kind});
    for (int b = 0; b < B; ++b) {
      const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
      const int nc = 2 * cp_degrees[b];
      const int32_t t0 = cbp[0], t1 = cbp[nc];
      std::vector<std::vector<Range>> kv_cover(nc);
      bool causal_seq = true;
      for (int c = 0; c < nc; ++c) {
        auto& v = by_kv[chunk_index0[b] + c];
        std::sort(v.begin(), v.end());
        auto& out_r = kv_cover[c];
        for (auto& qk : v) {
          const Range r{cbp[qk.first], cbp[qk.first + 1], qk.second};
          if (!out_r.empty() && !r.diag && out_r.back().e == r.b) out_r.back().e = r.e;   // keeps the first range's kind
          else out_r.push_back(r);
        }
        if (cbp[c + 1] > cbp[c])
          causal_seq = causal_seq && out_r.size() == 1 && out_r[0].diag && out_r[0].b == cbp[c] && out_r[0].e == t1;
      }
      // `spans`: the tiles are cut from the sequence start and a DIAG range starts where the first key of the
      // tile is first seen (earlier than the tile's own position when that key lies inside a span)
      auto emit_tiles = [&](int32_t k0, int32_t k1, int32_t first, const std::vector<Range>& rg, bool spans_on) {
        for (int32_t off = 0, t = 0; off < k1 - k0; off += FCP_TILE, ++t) {
          BU u{};
          const int32_t rows = std::min<int32_t>(FCP_TILE, k1 - k0 - off);
          u.f[BU_KV_ROW0] = k0 + off;
          u.f[BU_KV_ROWS] = rows;
          u.f[BU_FIRST_QRANGE] = first;
          u.f[BU_N_QRANGES] = (int32_t)rg.size();
          // Q tiles of a DIAG range run from T_FIRST on; those before T_MASK_END hold (query, key) pairs the
          // mask removes.  Causal: the tile on the diagonal only.
          int32_t t_first = t, t_mask_end = t + 1;
          if (spans_on) {
            t_first = (p->first_query[k0 + off] - k0) / FCP_TILE;
            t_mask_end = ceil_div(p->first_query[k0 + off + rows - 1] - k0, FCP_TILE);
          }
          u.f[BU_T_FIRST] = t_first;
          u.f[BU_T_MASK_END] = t_mask_end;
          int cost = 0;
          for (const Range& r : rg) {
            const int nt = ceil_div(r.e - r.b, FCP_TILE);
            cost += r.diag ? std::max(0, nt - t_first) : nt;
          }
          u.f[BU_COST] = cost;
          u.f[BU_SEQ] = b;
          bus.push_back(u);
        }
      };
      auto push_ranges = [&](const std::vector<Range>& rg) {
        const int32_t first = (int32_t)(p->bwd_qranges.size() / FCP_BWD_QRANGE_W);
        for (const Range& r : rg) {
          const int32_t rowq[4] = {r.b, r.e, r.diag, 0};
          p->bwd_qranges.insert(p->bwd_qranges.end(), rowq, rowq + 4);
        }
        return first;
      };
      if (causal_seq) {
        const std::vector<Range> whole{Range{t0, t1, 1}};
        emit_tiles(t0, t1, push_ranges(whole), whole, has_spans);
      } else {
        if (has_spans) {
          delete p;
          fcp_set_error("fcp_plan_blocks_spans: sequence %d has spans but its block pairs are not the causal set", b);
          return FCP_ERR_UNSUPPORTED;
        }
        for (int c = 0; c < nc; ++c)
          if (!kv_cover[c].empty()) emit_tiles(cbp[c], cbp[c + 1], push_ranges(kv_cover[c]), kv_cover[c], false);
      }
    }
  }
  for (const BU& u : bus) p->bwd_units.insert(p->bwd_units.end(), u.f, u.f + FCP_BWD_UNIT_W);
  // Execution order of the backward units within one KV head (the kernel runs the KV heads one after
  // the other, each over this list).  dQ is accumulated with fp32 reductions in global memory, which
  // only run at L2 speed while the rows they touch stay resident: so all CTAs work on one
  // (sequence, KV head) panel at a time, key tiles in ascending position (descending cost), and
  // sweep the query tiles roughly in step.  Sequences go longest first.
  {
    std::vector<int> seq_order(B);
    std::iota(seq_order.begin(), seq_order.end(), 0);
    std::stable_sort(seq_order.begin(), seq_order.end(), [&](int a, int b) { return seqlens[a] > seqlens[b]; });
    std::vector<std::vector<int32_t>> units_of(B);
    for (size_t i = 0; i < bus.size(); ++i) units_of[bus[i].f[BU_SEQ]].push_back((int32_t)i);   // ascending key position
    for (int b : seq_order)
      for (int32_t u : units_of[b]) p->bwd_work.push_back(u);
  }

  // Merge: runs of up to FCP_MERGE_TOKENS tokens inside one chunk.  Chunks with two or more slots
  // come first: a forward pass that writes the single-slot chunks straight to the output only needs
  // the first n_merge_multi units merged.
  for (int pass = 0; pass < 2; ++pass) {
    for (int b = 0; b < B; ++b) {
      const int32_t* cbp = &p->chunk_bounds[p->chunk_offset[b]];
      for (int c = 0; c < 2 * cp_degrees[b]; ++c) {
        const int ci = chunk_index0[b] + c;
        const bool single = p->slot_offset[ci + 1] - p->slot_offset[ci] <= 1;
        if (single != (pass == 1)) continue;
        for (int32_t t = cbp[c]; t < cbp[c + 1]; t += FCP_MERGE_TOKENS) {
          const int32_t rowm[4] = {t, std::min<int32_t>(FCP_MERGE_TOKENS, cbp[c + 1] - t), ci, cbp[c]};
          p->merge_units.insert(p->merge_units.end(), rowm, rowm + 4);
        }
      }
    }
    if (pass == 0) p->n_merge_multi = (int32_t)(p->merge_units.size() / FCP_MERGE_UNIT_W);
  }
  *out = p;
  return FCP_OK;
}

extern "C" int fcp_span_mask_efficiency(int32_t length, const int32_t* spans, int32_t n_spans, double* eta) {
  if (length <= 0 || !eta || n_spans < 0 || (n_spans > 0 && !spans)) {
    fcp_set_error("fcp_span_mask_efficiency: invalid argument");
    return FCP_ERR_INVALID_ARG;
  }
  // a span of m tokens adds the m(m-1)/2 pairs above its diagonal to the L(L+1)/2 causal ones
  double extra = 0.0;
  int32_t prev_end = 0;
  for (int i = 0; i < n_spans; ++i) {
    const int32_t a = spans[2 * i], e = spans[2 * i + 1];
    if (a < prev_end || e <= a || e > length) {
      fcp_set_error("fcp_span_mask_efficiency: span [%d, %d) is empty, out of range, unsorted or overlapping", a, e);
      return FCP_ERR_INVALID_ARG;
    }
    prev_end = e;
    const double m = double(e - a);
    extra += m * (m - 1.0) / 2.0;
  }
  *eta = extra / (double(length) * (double(length) + 1.0) / 2.0);
  return FCP_OK;
}

extern "C" int fcp_plan_get(const fcp_plan* plan, int32_t which, const int32_t** host_ptr, int64_t* count) {
  if (!plan || !host_ptr || !count) return FCP_ERR_INVALID_ARG;
  const std::vector<int32_t>* v = nullptr;
  switch (which) {
    case FCP_TABLE_CU_SEQLENS: v = &plan->cu_seqlens; break;
    case FCP_TABLE_CHUNK_OFFSET: v = &plan->chunk_offset; break;
    case FCP_TABLE_CHUNK_BOUNDS: v = &plan->chunk_bounds; break;
    case FCP_TABLE_PAIRS: v = &plan->pairs; break;
    case FCP_TABLE_ITEMS: v = &plan->items; break;
    case FCP_TABLE_SLOT_OFFSET: v = &plan->slot_offset; break;
    case FCP_TABLE_SLOT_ROWS: v = &plan->slot_rows; break;
    case FCP_TABLE_FWD_UNITS: v = &plan->fwd_units; break;
    case FCP_TABLE_BWD_UNITS: v = &plan->bwd_units; break;
    case FCP_TABLE_BWD_QRANGES: v = &plan->bwd_qranges; break;
    case FCP_TABLE_MERGE_UNITS: v = &plan->merge_units; break;
    case FCP_TABLE_BWD_WORK: v = &plan->bwd_work; break;
    case FCP_TABLE_FUSED_UNITS: v = &plan->fused_units; break;
    case FCP_TABLE_ROW_LIMIT: v = &plan->row_limit; break;
    case FCP_TABLE_FIRST_QUERY: v = &plan->first_query; break;
    case FCP_TABLE_SPAN_PAIRS: v = &plan->span_pairs; break;
    default: fcp_set_error("fcp_plan_get: unknown table %d", which); return FCP_ERR_INVALID_ARG;
  }
  *host_ptr = v->data();
  *count = (int64_t)v->size();
  return FCP_OK;
}

extern "C" int fcp_plan_info(const fcp_plan* plan, int32_t which, int64_t* value) {
  if (!plan || !value) return FCP_ERR_INVALID_ARG;
  switch (which) {
    case 0: *value = plan->T; break;
    case 1: *value = plan->R; break;
    case 2: *value = (int64_t)plan->pairs.size() / 6; break;
    case 3: *value = (int64_t)plan->items.size() / 8; break;
    case 4: *value = (int64_t)plan->fwd_units.size() / FCP_FWD_UNIT_W; break;
    case 5: *value = (int64_t)plan->bwd_units.size() / FCP_BWD_UNIT_W; break;
    case 6: *value = (int64_t)plan->merge_units.size() / FCP_MERGE_UNIT_W; break;
    case 7: *value = plan->B; break;
    case 8: *value = plan->n_merge_multi; break;
    case 9: *value = (int64_t)plan->fused_units.size() / FCP_FWD_UNIT_W; break;
    default: return FCP_ERR_INVALID_ARG;
  }
  return FCP_OK;
}
