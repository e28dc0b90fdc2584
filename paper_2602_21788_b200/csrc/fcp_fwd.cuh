// Forward attention over the block plan (Eq. 1 of the paper restricted to an item's KV ranges,
// causal mask k_pos <= q_pos), one persistent grid for all virtual ranks of all sequences.
//
// Work unit = (two adjacent 128-row Q tiles of one plan item, one query head).  Roles per CTA:
//   warp 0        work scheduler (global counter -> shared-memory ring) and TMA producer: Q tiles and the K/V tile
//                 ring (128-byte swizzled boxes)
//   warps 1, 2    UMMA issuers, one per Q tile: S = Q K^T into TMEM, O += P V with P read from TMEM
//   warps 4..7    softmax for Q tile 0: one thread per query row, the whole 128-column row in registers
//   warps 8..11   softmax for Q tile 1
//   warps 12..15  epilogue for both tiles: normalise O, store the partial output and its log-sum-exp
// TMEM (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each (D = 128); bf16 P overwrites the
// first 64 columns of its S.  While one tile's softmax runs on the CUDA cores the tensor core works
// on the other tile, so the two Q tiles share every K/V tile that is staged.
//
// Registers are moved between the warp groups at start-up: a softmax thread holds a full row of S
// (128 values), reads it from TMEM once, and needs no exchange with another thread for the row
// maximum or the row sum; the producer/issuer and epilogue groups give up what they do not need.
#pragma once
#include "fcp_plan.hpp"
#include "sm100_ptx.cuh"

namespace fcp {

constexpr int FWD_THREADS = 512;          // 4 control warps + 2 x 4 softmax warps + 4 epilogue warps
constexpr int FWD_KV_SLOTS = 4;
constexpr int FWD_WORK_SLOTS = 4;         // ring of work items handed from the producer to the other roles
// register budgets per thread of the three roles: 128 * 64 + 256 * 184 + 128 * 80 = 512 * 128
#define FCP_FWD_REGS_CTRL "64"
#define FCP_FWD_REGS_SOFTMAX "184"
#define FCP_FWD_REGS_EPI "80"

template <int D>
struct FwdSmem {
  static constexpr int Q_TILE_BYTES = 128 * D * 2;
  static constexpr int KV_TILE_BYTES = 128 * D * 2;
  static constexpr int Q_OFF = 0;
  static constexpr int KV_OFF = 2 * Q_TILE_BYTES;
  static constexpr int BAR_OFF = KV_OFF + FWD_KV_SLOTS * KV_TILE_BYTES;
  // barriers: q_full[2] q_empty[2] kv_full[S] kv_empty[S] s_full[2] p_full[2] o_final[2] o_empty[2] turn[2]
  //           stat_full[2] stat_empty[2]
  //           w_full[W] w_empty[W]
  static constexpr int N_BARS = 4 + 2 * FWD_KV_SLOTS + 14 + 2 * FWD_WORK_SLOTS;
  static constexpr int MISC_OFF = BAR_OFF + N_BARS * 8;   // tmem base (4 B), abort flag (4 B), work ring [W][unit, head]
  static constexpr int STAT_OFF = MISC_OFF + 16 + 8 * FWD_WORK_SLOTS;   // [2 tiles][row sum, reference maximum][128 rows] fp32
  static constexpr int TOTAL = STAT_OFF + 2 * 2 * 128 * 4;
  static constexpr int DYN_BYTES = TOTAL + 1024;          // slack to align the base to 1024 B
};

struct FwdArgs {
  const int32_t* units;   // [n_units][16]
  int32_t n_units;
  int32_t head_begin, head_count, hq, hkv;
  int32_t head_group;     // heads that are adjacent in the work order: hq/hkv when the head range is made of whole
                          // KV-head groups, else 1; head_count % head_group == 0
  int32_t* work_counter;  // zero before the launch: the grid's next work item
  float scale_log2;       // softmax scale * log2(e)
  float* o_partial;       // [R][head_count][D]
  float* lse_partial;     // [R][head_count]
  __nv_bfloat16* o_direct;   // [T][hq][D] or nullptr: final output of Q chunks that have a single slot
  float* lse_direct;         // [T][hq]
  float* o_f32_direct;       // [T][hq][D] or nullptr: the rows written to o_direct before their rounding to bf16
  const int32_t* row_limit;  // [T] or nullptr (causal): first key (packed index) that query t does not see
  int32_t* status;        // [4]
};

template <int D>
__global__ void __launch_bounds__(FWD_THREADS, 1)
fcp_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const FwdArgs a) {
  using SM = FwdSmem<D>;
  constexpr int KBLK = D / 64;                 // 64-element (128-byte) column blocks per row
  constexpr uint32_t BLK_BYTES = 128 * 128;    // one [128 rows][64] swizzled block
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t S_COL0 = 0, O_COL0 = 256; // S stage s at 128*s, O stage s at 256 + 128*s

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + SM::BAR_OFF;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  const int B_QFULL = 0, B_QEMPTY = 2, B_KVFULL = 4, B_KVEMPTY = 4 + FWD_KV_SLOTS,
            B_SFULL = 4 + 2 * FWD_KV_SLOTS, B_PFULL = B_SFULL + 2, B_OFINAL = B_SFULL + 4, B_OEMPTY = B_SFULL + 6,
            B_TURN = B_SFULL + 8, B_STATFULL = B_SFULL + 10, B_STATEMPTY = B_SFULL + 12, B_WFULL = B_SFULL + 14,
            B_WEMPTY = B_WFULL + FWD_WORK_SLOTS;
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(smem + SM::MISC_OFF);
  volatile int* abort_flag = (volatile int*)(smem + SM::MISC_OFF + 4);
  volatile int* work_ring = (volatile int*)(smem + SM::MISC_OFF + 16);   // [FWD_WORK_SLOTS][unit, head]
  const WaitCtx wctx{abort_flag, a.status, (uint32_t)FCP_WAIT_NS};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(B_QFULL + i), 1);
      mbar_init(BAR(B_QEMPTY + i), 1);
      mbar_init(BAR(B_SFULL + i), 1);
      mbar_init(BAR(B_PFULL + i), 4);          // one elected lane per softmax warp
      mbar_init(BAR(B_OFINAL + i), 1);
      mbar_init(BAR(B_OEMPTY + i), 4);         // one elected lane per epilogue warp
      mbar_init(BAR(B_TURN + i), 4);
      mbar_init(BAR(B_STATFULL + i), 4);
      mbar_init(BAR(B_STATEMPTY + i), 4);
    }
    for (int i = 0; i < FWD_WORK_SLOTS; ++i) {
      mbar_init(BAR(B_WFULL + i), 1);
      mbar_init(BAR(B_WEMPTY + i), 2 + 8 + 4);   // two issuing threads, one lane of each softmax and epilogue warp
    }
    for (int i = 0; i < FWD_KV_SLOTS; ++i) {
      mbar_init(BAR(B_KVFULL + i), 1);
      mbar_init(BAR(B_KVEMPTY + i), 2);        // one commit from each issuer
    }
    fence_mbar_init();
    prefetch_tmap(&tm_q);
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const int64_t n_work = (int64_t)a.n_units * a.head_count;
  const int g = a.hq / a.hkv;
  // Work order.  Item w = (head within a group of gi heads, unit, group), innermost first; gi = the query heads of
  // one KV head when the head range is made of whole KV-head groups, else 1.  Units are sorted by cost, so the CTAs
  // that run at the same time work on adjacent units of the same KV head and stream the same K/V tiles: one copy in
  // L2 serves them all.  Items are handed out dynamically: the producer thread takes item numbers from a global
  // counter and passes (unit, head) through a small ring in shared memory to the issuing threads and the softmax
  // and epilogue warps, which all consume every item in order; -1 ends the list.
  const int gi = a.head_group;
  // returns 1 with (U, h) of the next item, 0 at the end of the list, -1 if the CTA is aborting
  auto take_item = [&](uint32_t& n, const int32_t*& U, int& h, bool whole_warp) -> int {
    const uint32_t slot = n % FWD_WORK_SLOTS, par = (n / FWD_WORK_SLOTS) & 1;
    const bool got = whole_warp ? mbar_wait_warp(BAR(B_WFULL + slot), par, wctx, 40) : mbar_wait(BAR(B_WFULL + slot), par, wctx, 40);
    if (!got) return -1;
    const int unit = work_ring[2 * slot];
    h = work_ring[2 * slot + 1];
    if (whole_warp) {
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_WEMPTY + slot));
    } else {
      mbar_arrive(BAR(B_WEMPTY + slot));
    }
    ++n;
    if (unit < 0) return 0;
    U = a.units + (size_t)unit * FCP_FWD_UNIT_W;
    return 1;
  };

  if (warp < 4) asm volatile("setmaxnreg.dec.sync.aligned.u32 " FCP_FWD_REGS_CTRL ";");
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t kv_it = 0, qcnt[2] = {0, 0}, nw = 0;
      bool ok = true;
#pragma unroll 1
      while (ok) {
        const int64_t w = atomicAdd(a.work_counter, 1);
        const uint32_t slot = nw % FWD_WORK_SLOTS;
        ok = mbar_wait(BAR(B_WEMPTY + slot), ((nw / FWD_WORK_SLOTS) & 1) ^ 1, wctx, 41);
        if (!ok) break;
        const bool last = w >= n_work;
        int unit = -1, h = 0;
        if (!last) {
          const int64_t t = w / gi;
          unit = (int)(t % a.n_units);
          h = a.head_begin + (int)(t / a.n_units) * gi + (int)(w % gi);
        }
        work_ring[2 * slot] = unit;
        work_ring[2 * slot + 1] = h;
        mbar_arrive(BAR(B_WFULL + slot));      // release: the two stores above are visible to the waiters
        ++nw;
        if (last) break;
        const int32_t* U = a.units + (size_t)unit * FCP_FWD_UNIT_W;
        const int hk = h / g;
        const int nt[2] = {__ldg(U + FU_NT_STAGE0), __ldg(U + FU_NT_STAGE1)};
        const int q_row0 = __ldg(U + FU_Q_ROW0);
#pragma unroll 1
        for (int s = 0; s < 2 && ok; ++s) {
          if (nt[s] == 0) continue;
          ok = mbar_wait(BAR(B_QEMPTY + s), (qcnt[s] & 1) ^ 1, wctx, 10 + s);
          if (!ok) break;
          mbar_expect_tx(BAR(B_QFULL + s), SM::Q_TILE_BYTES);
#pragma unroll 1
          for (int kb = 0; kb < KBLK; ++kb)
            tma_load_3d(sbase + SM::Q_OFF + s * SM::Q_TILE_BYTES + kb * BLK_BYTES, &tm_q, BAR(B_QFULL + s), kb * 64, h,
                        q_row0 + s * 128);
          ++qcnt[s];
        }
        const int n_max = max(nt[0], nt[1]);
        const int nr0 = __ldg(U + FU_NT_RANGE0);
        const int kv0 = __ldg(U + FU_KV0_BEGIN), kv1 = __ldg(U + FU_KV1_BEGIN);
#pragma unroll 1
        for (int j = 0; j < n_max && ok; ++j) {
          const int row = j < nr0 ? kv0 + j * 128 : kv1 + (j - nr0) * 128;
#pragma unroll 1
          for (int t = 0; t < 2; ++t) {   // t = 0: K tile, t = 1: V tile
            const uint32_t slot = kv_it % FWD_KV_SLOTS;
            ok = mbar_wait(BAR(B_KVEMPTY + slot), ((kv_it / FWD_KV_SLOTS) & 1) ^ 1, wctx, 12);
            if (!ok) break;
            mbar_expect_tx(BAR(B_KVFULL + slot), SM::KV_TILE_BYTES);
#pragma unroll 1
            for (int kb = 0; kb < KBLK; ++kb)
              tma_load_3d(sbase + SM::KV_OFF + slot * SM::KV_TILE_BYTES + kb * BLK_BYTES, t == 0 ? &tm_k : &tm_v,
                          BAR(B_KVFULL + slot), kb * 64, hk, row);
            ++kv_it;
          }
        }
      }
    }
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------------ UMMA issuers, one per Q tile
    // A single thread cannot issue the 32 UMMAs of one K/V tile (two Q tiles) plus its waits and
    // commits in the 2048 clocks they take to execute, so each Q tile has its own issuing thread;
    // their products touch disjoint TMEM columns and only read the shared K/V tiles.
    if (lane == 0) {
      // one issuing thread per Q tile (measured faster than a warp in uniform flow with a leader lane)
      const bool leader = true;
      constexpr uint32_t IDESC_QK = make_idesc(128, 128, 0, 0);
      constexpr uint32_t IDESC_PV = make_idesc(128, D, 0, 1);
      const int s = warp - 1;
      const uint32_t t_s = tmem + S_COL0 + s * 128, t_o = tmem + O_COL0 + s * 128;
      const uint32_t q_addr = sbase + SM::Q_OFF + s * SM::Q_TILE_BYTES;
      uint32_t kv_it = 0, qcnt = 0, pcnt = 0, ocnt = 0, nw = 0;
      bool ok = true;
#pragma unroll 1
      while (ok) {
        const int32_t* U;
        int h;
        const int r = take_item(nw, U, h, false);
        if (r <= 0) { ok = r == 0; break; }
        const int nts = __ldg(U + FU_NT_STAGE0 + s);
        const int n_max = max(__ldg(U + FU_NT_STAGE0), __ldg(U + FU_NT_STAGE1));
        if (nts > 0) {
          ok = mbar_wait(BAR(B_QFULL + s), qcnt & 1, wctx, 20 + s);
          ++qcnt;
        }
#pragma unroll 1
        for (int j = 0; j <= n_max && ok; ++j) {
          // ring positions: K_j at kv_it + 2j, V_{j-1} at kv_it + 2j - 1
          const uint32_t itK = kv_it + 2 * j, itV = kv_it + 2 * j - 1;
          const uint32_t slotK = itK % FWD_KV_SLOTS, slotV = itV % FWD_KV_SLOTS;
          // Every slot is awaited and released by both issuers, whether or not their tile uses it:
          // a release may only be counted in the phase of the load it answers.
          if (j >= 1) ok = mbar_wait(BAR(B_KVFULL + slotV), (itV / FWD_KV_SLOTS) & 1, wctx, 22);
          if (ok && j < n_max) ok = mbar_wait(BAR(B_KVFULL + slotK), (itK / FWD_KV_SLOTS) & 1, wctx, 23);
          if (!ok) break;
          if (j >= 1 && j - 1 < nts) {
            // O_s (+)= P_s(j-1) V_{j-1}
            if (j == 1) {
              ok = mbar_wait(BAR(B_OEMPTY + s), (ocnt & 1) ^ 1, wctx, 24 + s);
              ++ocnt;
            }
            if (ok) ok = mbar_wait(BAR(B_PFULL + s), pcnt & 1, wctx, 26 + s);
            ++pcnt;
            if (!ok) break;
            tc_fence_after();
            umma_loop_ts(leader, t_o, t_s, false, sbase + SM::KV_OFF + slotV * SM::KV_TILE_BYTES, IDESC_PV, j > 1 ? 1u : 0u);
            if (j == nts) tc_commit_if(leader, BAR(B_OFINAL + s));
          }
          if (j < nts) {
            // S_s = Q_s K_j^T
            tc_fence_after();
            umma_loop_kk<D / 16>(leader, t_s, q_addr, sbase + SM::KV_OFF + slotK * SM::KV_TILE_BYTES, IDESC_QK);
            tc_commit_if(leader, BAR(B_SFULL + s));
            if (j == nts - 1) tc_commit_if(leader, BAR(B_QEMPTY + s));
          }
          if (j >= 1) tc_commit_if(leader, BAR(B_KVEMPTY + slotV));
          if (j < n_max) tc_commit_if(leader, BAR(B_KVEMPTY + slotK));
        }
        kv_it += 2 * n_max;
      }
    }
  } else if (warp >= 4 && warp < 12) {
    // ------------------------------------------------------------------ softmax
    // Four warps per Q tile, one per TMEM lane quarter; a thread owns one query row and reads all 128
    // scores of the current K/V tile into registers with one round of TMEM loads.
    asm volatile("setmaxnreg.inc.sync.aligned.u32 " FCP_FWD_REGS_SOFTMAX ";");
    const int s = (warp - 4) >> 2;            // Q tile handled by this warp group
    const int rb = warp & 3;                  // TMEM lane quarter this warp may access
    const int row = rb * 32 + lane;
    const uint32_t t_s = tmem_addr(tmem, rb * 32, S_COL0 + s * 128);   // P goes over the first 64 columns
    const uint32_t t_o = tmem_addr(tmem, rb * 32, O_COL0 + s * 128);
    float* stat = (float*)(smem + SM::STAT_OFF) + s * 256;
    const float c2 = a.scale_log2;
    uint32_t scnt = 0, ucnt = 0, tcnt = 0, nw = 0;
    bool ok = true;
#pragma unroll 1
    while (ok) {
      const int32_t* U;
      int h;
      const int r = take_item(nw, U, h, true);
      if (r <= 0) { ok = r == 0; break; }
      const int nts = __ldg(U + FU_NT_STAGE0 + s);
      const int n_max = max(__ldg(U + FU_NT_STAGE0), __ldg(U + FU_NT_STAGE1));
      const int q_pos = __ldg(U + FU_Q_ROW0) + s * 128 + row;
      // first key this row does not see in a DIAG range: the one after itself, or the end of its span
      const int row_lim = (a.row_limit != nullptr && s * 128 + row < __ldg(U + FU_Q_ROWS)) ? __ldg(a.row_limit + q_pos) : q_pos + 1;
      const int nr0 = __ldg(U + FU_NT_RANGE0);
      const int kvb0 = __ldg(U + FU_KV0_BEGIN), kvb1 = __ldg(U + FU_KV1_BEGIN);
      const int kve0 = __ldg(U + FU_KV0_END), kve1 = __ldg(U + FU_KV1_END);
      const int kvd0 = __ldg(U + FU_KV0_DIAG), kvd1 = __ldg(U + FU_KV1_DIAG);
      float m_ref = -INFINITY, l = 0.f;
#pragma unroll 1
      for (int j = 0; j < n_max && ok; ++j) {
        // The two softmax groups take turns at the exponentials (the MUFU pipe cannot serve both at
        // full speed): tile 0 of K/V tile j, tile 1 of j, tile 0 of j+1, ...  While one group is in
        // its exponentials the tensor core runs the other tile's products.  A group without work
        // for this j only passes the turn on.
        if (j >= nts) {
          ok = mbar_wait_warp(BAR(B_TURN + s), (tcnt & 1) ^ (s ^ 1), wctx, 34 + s);
          ++tcnt;
          __syncwarp();
          if (lane == 0) mbar_arrive(BAR(B_TURN + (s ^ 1)));
          continue;
        }
        const bool r1 = j >= nr0;
        const int ks = r1 ? kvb1 + (j - nr0) * 128 : kvb0 + j * 128;
        int limit = (r1 ? kve1 : kve0) - ks;                  // valid columns of this tile for this row
        if (r1 ? kvd1 : kvd0) limit = min(limit, row_lim - ks);
        const bool masked = __any_sync(0xffffffffu, limit < 128);
        ok = mbar_wait_warp(BAR(B_SFULL + s), scnt & 1, wctx, 30 + s);
        ++scnt;
        if (!ok) break;
        tc_fence_after();
        uint32_t sv[4][32];
#pragma unroll
        for (int b = 0; b < 4; ++b) tmem_ld32(t_s + 32 * b, sv[b]);
        tc_wait_ld();
        if (masked) {
#pragma unroll
          for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (b * 32 + i >= limit) sv[b][i] = 0xff800000u;         // -inf
        }
        float mx;
        {
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
          for (int b = 0; b < 4; ++b)
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              mx0 = fmaxf(mx0, fmaxf(__uint_as_float(sv[b][i]), __uint_as_float(sv[b][i + 1])));
              mx1 = fmaxf(mx1, fmaxf(__uint_as_float(sv[b][i + 2]), __uint_as_float(sv[b][i + 3])));
              mx2 = fmaxf(mx2, fmaxf(__uint_as_float(sv[b][i + 4]), __uint_as_float(sv[b][i + 5])));
              mx3 = fmaxf(mx3, fmaxf(__uint_as_float(sv[b][i + 6]), __uint_as_float(sv[b][i + 7])));
            }
          mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c2;
        }
        // Lazy reference maximum: O and l are only rescaled when the row maximum grew by more than
        // 2^8, so p <= 256 always and the result is exact up to rounding.  The products issued so far
        // have completed (S of this tile was committed after them), so O is at rest here.
        const bool grow = mx > m_ref + 8.f;
        if (__any_sync(0xffffffffu, grow)) {
          const float m_new = grow ? mx : m_ref;
          const float f = grow ? ex2(m_ref - m_new) : 1.f;    // m_ref = -inf -> 0
          l *= f;
          if (j > 0) {
#pragma unroll 1
            for (int c = 0; c < D / 16; ++c) {
              uint32_t ov[16];
              tmem_ld16(t_o + c * 16, ov);
              tc_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * f);
              tmem_st16(t_o + c * 16, ov);
            }
          }
          m_ref = m_new;
        }
        ok = mbar_wait_warp(BAR(B_TURN + s), (tcnt & 1) ^ (s ^ 1), wctx, 34 + s);
        ++tcnt;
        if (!ok) break;
        // exponentials, row sum, bf16 P over the first 64 columns of S (masked scores are -inf -> 0)
        float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          uint32_t pk[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float p0 = ex2(fmaf(__uint_as_float(sv[b][2 * i]), c2, -m_ref));
            const float p1 = ex2(fmaf(__uint_as_float(sv[b][2 * i + 1]), c2, -m_ref));
            if ((i & 3) == 0) sum0 += p0 + p1;
            else if ((i & 3) == 1) sum1 += p0 + p1;
            else if ((i & 3) == 2) sum2 += p0 + p1;
            else sum3 += p0 + p1;
            pk[i] = pack_bf16(p0, p1);
          }
          tmem_st16(t_s + b * 16, pk);
        }
        l += (sum0 + sum1) + (sum2 + sum3);
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_TURN + (s ^ 1)));
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_PFULL + s));
      }
      if (!ok) break;
      if (nts == 0) continue;
      // hand the row sum and the reference maximum to the epilogue warps
      ok = mbar_wait_warp(BAR(B_STATEMPTY + s), (ucnt & 1) ^ 1, wctx, 36 + s);
      ++ucnt;
      if (!ok) break;
      stat[row] = l;
      stat[128 + row] = m_ref;
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_STATFULL + s));
    }
  } else if (warp >= 12) {
    // ------------------------------------------------------------------ epilogue
    // Normalised partial output + log-sum-exp of both Q tiles, while the softmax warps and the
    // issuers already work on the next unit.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 " FCP_FWD_REGS_EPI ";");
    const int rb = warp & 3;
    const int row = rb * 32 + lane;
    uint32_t ecnt0 = 0, ecnt1 = 0, nw = 0;     // phases seen per Q tile; work items taken
    bool ok = true;
#pragma unroll 1
    while (ok) {
      const int32_t* U;
      int h;
      const int r = take_item(nw, U, h, true);
      if (r <= 0) { ok = r == 0; break; }
      const int hl = h - a.head_begin;
      const int q_rows = __ldg(U + FU_Q_ROWS);
      const int64_t prow0 = (int64_t)__ldg(U + FU_PART_ROW0);
      // A Q chunk with one slot has nothing to merge: its partial is the result, and goes straight to
      // the output (rounded to bf16 exactly as the merge would round it) when the caller asks for that.
      const bool direct = a.o_direct != nullptr && __ldg(U + FU_SINGLE_SLOT) != 0;
      const int64_t trow0 = (int64_t)__ldg(U + FU_Q_ROW0);
#pragma unroll 1
      for (int s = 0; s < 2 && ok; ++s) {
        if (__ldg(U + FU_NT_STAGE0 + s) == 0) continue;
        const float* stat = (const float*)(smem + SM::STAT_OFF) + s * 256;
        const uint32_t ph = (s ? ecnt1 : ecnt0) & 1;
        if (s) ++ecnt1; else ++ecnt0;
        ok = mbar_wait_warp(BAR(B_STATFULL + s), ph, wctx, 38 + s);
        if (!ok) break;
        const float l = stat[row], m_ref = stat[128 + row];
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_STATEMPTY + s));
        ok = mbar_wait_warp(BAR(B_OFINAL + s), ph, wctx, 32 + s);
        if (!ok) break;
        tc_fence_after();
        const uint32_t t_o = tmem_addr(tmem, rb * 32, O_COL0 + s * 128);
        const int rows_s = min(128, q_rows - s * 128);
        const float inv_l = 1.f / l;
        const float lse_row = (m_ref + log2f(l)) * 0.6931471805599453f;
        if (direct) {
          const int64_t orow = (trow0 + s * 128 + row) * a.hq + a.head_begin + hl;
          __nv_bfloat16* op = a.o_direct + orow * D;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t ov[32];
            tmem_ld32(t_o + c * 32, ov);
            tc_wait_ld();
            if (row < rows_s) {
#pragma unroll
              for (int i = 0; i < 32; i += 8)
                *reinterpret_cast<uint4*>(op + c * 32 + i) =
                    make_uint4(pack_bf16(__uint_as_float(ov[i]) * inv_l, __uint_as_float(ov[i + 1]) * inv_l),
                               pack_bf16(__uint_as_float(ov[i + 2]) * inv_l, __uint_as_float(ov[i + 3]) * inv_l),
                               pack_bf16(__uint_as_float(ov[i + 4]) * inv_l, __uint_as_float(ov[i + 5]) * inv_l),
                               pack_bf16(__uint_as_float(ov[i + 6]) * inv_l, __uint_as_float(ov[i + 7]) * inv_l));
            }
          }
          if (row < rows_s) a.lse_direct[orow] = lse_row;
          if (a.o_f32_direct != nullptr) {
            float* fp = a.o_f32_direct + orow * D;
#pragma unroll 1
            for (int c = 0; c < D / 32; ++c) {
              uint32_t ov[32];
              tmem_ld32(t_o + c * 32, ov);
              tc_wait_ld();
              if (row < rows_s) {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                  *reinterpret_cast<float4*>(fp + c * 32 + i) =
                      make_float4(__uint_as_float(ov[i]) * inv_l, __uint_as_float(ov[i + 1]) * inv_l,
                                  __uint_as_float(ov[i + 2]) * inv_l, __uint_as_float(ov[i + 3]) * inv_l);
              }
            }
          }
        } else {
          const int64_t prow = prow0 + s * 128 + row;
          float* op = a.o_partial + (prow * a.head_count + hl) * D;
#pragma unroll 1
          for (int c = 0; c < D / 32; ++c) {
            uint32_t ov[32];
            tmem_ld32(t_o + c * 32, ov);
            tc_wait_ld();
            if (row < rows_s) {
#pragma unroll
              for (int i = 0; i < 32; i += 4)
                *reinterpret_cast<float4*>(op + c * 32 + i) =
                    make_float4(__uint_as_float(ov[i]) * inv_l, __uint_as_float(ov[i + 1]) * inv_l,
                                __uint_as_float(ov[i + 2]) * inv_l, __uint_as_float(ov[i + 3]) * inv_l);
            }
          }
          if (row < rows_s) a.lse_partial[prow * a.head_count + hl] = lse_row;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_OEMPTY + s));
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  wait_teardown(wctx);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace fcp
