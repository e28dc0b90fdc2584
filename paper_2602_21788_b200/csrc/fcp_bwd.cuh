// Backward attention over the block plan, grouped by KV chunk: the derivative of Eq. 1 of the paper
// with the causal mask.  One persistent grid; a work unit = (128-key tile of a KV chunk, KV head).
// The unit keeps its K and V tiles in shared memory and dK, dV in tensor memory while it walks over
// every (Q tile, query head of the group) of every block pair that attends to the chunk:
//
//   T1  S^T  = K Q^T                   (UMMA, smem x smem)      TMEM cols [  0,128)
//   T2  dP^T = V dO^T                  (UMMA, smem x smem)      TMEM cols [128,256)
//   C1  P^T  = exp2(S^T*c - lse2[q])   (CUDA cores, thread = key row x half of the queries), bf16 over S^T
//   T3  dV  += P^T dO                  (UMMA, TMEM x smem)      TMEM cols [256,384)
//   C2  dS^T = P^T o (dP^T*scale - delta[q]*scale)               bf16 to smem
//   T5  dQ^T = K^T dS^T  (D = 128; rows = head-dim index)  or  dQ = dS K  (D = 64; rows = queries)
//                                      (UMMA, smem x smem)      over dP^T
//   T4  dK  += dS^T Q                  (UMMA, smem x smem)      TMEM cols [384,512); issued after T5 so
//                                      that it runs while the drain warps read the dQ tile
//   C3  dQ accumulator += tile         fp32 reductions to global memory (coalesced for D = 128)
//
// 16 warps: warp 0 TMA producer and work scheduler, warp 1 UMMA issuer (warps 2-3 idle), warps 4..11
// the element-wise math C1/C2 (two warps per TMEM lane quarter, each half of the query columns),
// warps 12..15 the dQ drain C3 and the dK/dV epilogue.  The issuer runs T1 of the next tile as soon
// as C1 has read S^T, and T2 of the next tile as soon as C3 has drained dQ, so the tensor core, the
// math warps and the drain warps work on different tiles at the same time.
//
// Work items are handed out through a global counter: KV heads one after the other, within a head
// the units in plan order (one sequence after the other, keys ascending), so that the dQ rows being
// reduced into stay in L2.
#pragma once
#include "fcp_plan.hpp"
#include "sm100_ptx.cuh"

namespace fcp {

constexpr int BWD_THREADS = 512;
constexpr int BWD_QDO_STAGES = 2;
constexpr int BWD_MATH_WARPS = 8;
constexpr int BWD_DRAIN_WARPS = 4;

template <int D>
struct BwdSmem {
  static constexpr int TILE_BYTES = 128 * D * 2;
  static constexpr int K_OFF = 0;
  static constexpr int V_OFF = TILE_BYTES;
  static constexpr int DS_OFF = 2 * TILE_BYTES;                         // [2][128 keys][64 q] bf16, swizzled
  static constexpr int Q_OFF = DS_OFF + 128 * 128 * 2;
  static constexpr int DO_OFF = Q_OFF + BWD_QDO_STAGES * TILE_BYTES;
  static constexpr int ROWS_OFF = DO_OFF + BWD_QDO_STAGES * TILE_BYTES;  // [2 buffers][lse2[128], delta[128]] fp32
  static constexpr int BAR_OFF = ROWS_OFF + 2048;
  static constexpr int N_BARS = 2 + 2 * BWD_QDO_STAGES + 9 + 4;
  static constexpr int MISC_OFF = BAR_OFF + N_BARS * 8;                  // tmem base, abort flag, work ring [2][2]
  static constexpr int TOTAL = MISC_OFF + 32;
  // The tiles need 1024-byte alignment.  The dynamic shared window of a kernel without static shared
  // memory starts 1024-byte aligned; the kernel checks this and reports an error instead of running
  // if it ever does not hold (there is no room for alignment slack at D = 128).
  static constexpr int DYN_BYTES = TOTAL;
};

struct BwdArgs {
  const int32_t* units;     // [n_units][8]
  const int32_t* qranges;   // [n][4]
  const int32_t* work;      // [n_units]: units in execution order; work item w = (work[w % n_units], hk_begin + w / n_units)
  int32_t n_work, n_units, hq, hkv;
  int32_t hk_begin;         // first KV head of this pass
  int32_t hq_acc;           // query heads held by dq_acc / delta_t / lse2_t: those of the pass, numbered from 0
  int32_t* counter;         // work counter, zero before the launch
  int64_t T, t_stride;
  float scale, scale_log2;
  const float* delta_t;     // [hq_acc][t_stride], already multiplied by the softmax scale
  const float* lse2_t;      // [hq_acc][t_stride], log2 units
  const int32_t* first_query;   // [T] or nullptr (causal): first query (packed index) that sees key t
  float* dq_acc;            // [T][hq_acc][D] fp32, zero-initialised
  __nv_bfloat16* dk;        // [T][hkv][D]
  __nv_bfloat16* dv;
  int32_t* status;
};

// The (head-of-group, Q range, Q tile) iterations of one unit, in the order every role walks them.
// The head is the outer loop: all CTAs of a (sequence, KV head) panel then sweep the query tiles of
// one query head at a time, which keeps the dQ rows they reduce into (and the Q/dO tiles they
// share) to one head's worth of L2.
struct BwdIter {
  const int32_t* qr;     // Q ranges of the unit
  int nq, t_first, t_mask_end, g;   // a DIAG range starts at Q tile t_first; tiles before t_mask_end need the mask
  int r, t, hh;          // range, tile within range, head within group
  int qb, qe, diag;
  bool valid;
  int q_row, q_valid;
  bool causal;

  __device__ __forceinline__ void load_range() {
    const int32_t* Q = qr + (size_t)r * FCP_BWD_QRANGE_W;
    qb = __ldg(Q + BQ_BEGIN);
    qe = __ldg(Q + BQ_END);
    diag = __ldg(Q + BQ_DIAG);
    t = diag ? t_first : 0;
  }
  __device__ __forceinline__ void settle() {           // make (hh, r, t) point at an existing tile
    while (valid && qb + t * 128 >= qe) {
      if (++r >= nq) {
        r = 0;
        if (++hh >= g) { valid = false; break; }
      }
      load_range();
    }
    if (valid) {
      q_row = qb + t * 128;
      q_valid = min(128, qe - q_row);
      causal = diag && t < t_mask_end;
    }
  }
  __device__ __forceinline__ void init(const int32_t* U, const int32_t* qranges, int g_) {
    qr = qranges + (size_t)__ldg(U + BU_FIRST_QRANGE) * FCP_BWD_QRANGE_W;
    nq = __ldg(U + BU_N_QRANGES);
    t_first = __ldg(U + BU_T_FIRST);
    t_mask_end = __ldg(U + BU_T_MASK_END);
    g = g_;
    r = 0; hh = 0;
    valid = nq > 0;
    if (valid) load_range();
    settle();
  }
  __device__ __forceinline__ void advance() {
    ++t;
    settle();
  }
};

__device__ __forceinline__ void red_add_f32(float* p, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}
__device__ __forceinline__ void red_add_v4_f32(float* p, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int D>
__global__ void __launch_bounds__(BWD_THREADS, 1)
fcp_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const BwdArgs a) {
  using SM = BwdSmem<D>;
  constexpr int KBLK = D / 64;
  constexpr uint32_t BLK_BYTES = 128 * 128;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t C_S = 0, C_DP = 128, C_DV = 256, C_DK = 384;
  constexpr bool DQ_T = (D == 128);            // dQ tile kept transposed in TMEM (rows = head-dim index)

  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  if ((sbase & 1023u) != 0) {                  // uniform across the grid: nobody touches a barrier
    if (threadIdx.x == 0 && blockIdx.x == 0) {
      a.status[0] = -5;
      a.status[1] = 199;
    }
    return;
  }
  const uint32_t bar0 = sbase + SM::BAR_OFF;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  const int B_KVFULL = 0, B_KVFREE = 1, B_QDOFULL = 2, B_QDOFREE = 2 + BWD_QDO_STAGES, B0 = 2 + 2 * BWD_QDO_STAGES;
  const int B_SFULL = B0, B_DPFULL = B0 + 1, B_PFULL = B0 + 2, B_DSFULL = B0 + 3, B_DQFULL = B0 + 4,
            B_DQEMPTY = B0 + 5, B_ACCFULL = B0 + 6, B_ACCEMPTY = B0 + 7, B_ROWS = B0 + 8, B_WFULL = B0 + 9,
            B_WEMPTY = B0 + 11;
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(smem + SM::MISC_OFF);
  volatile int* abort_flag = (volatile int*)(smem + SM::MISC_OFF + 4);
  volatile int* work_ring = (volatile int*)(smem + SM::MISC_OFF + 8);    // [2 slots][unit, kv head]
  const WaitCtx wctx{abort_flag, a.status, (uint32_t)FCP_WAIT_NS};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    *abort_flag = 0;
    mbar_init(BAR(B_KVFULL), 1);
    mbar_init(BAR(B_KVFREE), 1);
    for (int i = 0; i < BWD_QDO_STAGES; ++i) {
      mbar_init(BAR(B_QDOFULL + i), 1);
      mbar_init(BAR(B_QDOFREE + i), 1);
    }
    mbar_init(BAR(B_SFULL), 1);
    mbar_init(BAR(B_DPFULL), 1);
    mbar_init(BAR(B_PFULL), BWD_MATH_WARPS);
    mbar_init(BAR(B_DSFULL), BWD_MATH_WARPS);
    mbar_init(BAR(B_DQFULL), 1);
    mbar_init(BAR(B_DQEMPTY), BWD_DRAIN_WARPS);
    mbar_init(BAR(B_ACCFULL), 1);
    mbar_init(BAR(B_ACCEMPTY), BWD_DRAIN_WARPS);
    mbar_init(BAR(B_ROWS), BWD_MATH_WARPS);
    for (int i = 0; i < 2; ++i) {
      mbar_init(BAR(B_WFULL + i), 1);
      mbar_init(BAR(B_WEMPTY + i), 1 + BWD_MATH_WARPS + BWD_DRAIN_WARPS);   // issuer + one lane per consumer warp
    }
    fence_mbar_init();
    prefetch_tmap(&tm_q);
    prefetch_tmap(&tm_k);
    prefetch_tmap(&tm_v);
    prefetch_tmap(&tm_do);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const int g = a.hq / a.hkv;

  // Consumers take the next work item from the ring the producer fills; returns the unit row or
  // nullptr at the end of the list (or when aborting).  `n` counts the items taken so far.
  auto next_work = [&](uint32_t n, int& hk, bool& ok) -> const int32_t* {
    const uint32_t slot = n & 1;
    ok = mbar_wait_warp(BAR(B_WFULL + slot), (n >> 1) & 1, wctx, 140);
    if (!ok) return nullptr;
    const int unit = work_ring[2 * slot];
    hk = work_ring[2 * slot + 1];
    __syncwarp();
    if (lane == 0) mbar_arrive(BAR(B_WEMPTY + slot));
    return unit >= 0 ? a.units + (size_t)unit * FCP_BWD_UNIT_W : nullptr;
  };

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
    if (warp == 0 && lane == 0) {
      // ------------------------------------------------------------------ TMA producer + scheduler
      uint32_t n = 0, it = 0;
      bool ok = true;
      while (ok) {
        const int w = atomicAdd(a.counter, 1);
        const uint32_t slot = n & 1;
        ok = mbar_wait(BAR(B_WEMPTY + slot), ((n >> 1) & 1) ^ 1, wctx, 112);
        if (!ok) break;
        const bool last = w >= a.n_work;
        const int unit = last ? -1 : __ldg(a.work + w % a.n_units);
        const int hk = last ? 0 : a.hk_begin + w / a.n_units;
        work_ring[2 * slot] = unit;
        work_ring[2 * slot + 1] = hk;
        mbar_arrive(BAR(B_WFULL + slot));     // release: the two stores above are visible to the waiters
        if (last) break;
        const int32_t* U = a.units + (size_t)unit * FCP_BWD_UNIT_W;
        const int kv_row0 = __ldg(U + BU_KV_ROW0);
        ok = mbar_wait(BAR(B_KVFREE), (n & 1) ^ 1, wctx, 110);
        ++n;
        if (!ok) break;
        mbar_expect_tx(BAR(B_KVFULL), 2 * SM::TILE_BYTES);
#pragma unroll 1
        for (int kb = 0; kb < KBLK; ++kb) {
          tma_load_3d(sbase + SM::K_OFF + kb * BLK_BYTES, &tm_k, BAR(B_KVFULL), kb * 64, hk, kv_row0);
          tma_load_3d(sbase + SM::V_OFF + kb * BLK_BYTES, &tm_v, BAR(B_KVFULL), kb * 64, hk, kv_row0);
        }
        BwdIter iter;
#pragma unroll 1
        for (iter.init(U, a.qranges, g); iter.valid; iter.advance(), ++it) {
          const uint32_t st = it % BWD_QDO_STAGES;
          ok = mbar_wait(BAR(B_QDOFREE + st), ((it / BWD_QDO_STAGES) & 1) ^ 1, wctx, 111);
          if (!ok) break;
          mbar_expect_tx(BAR(B_QDOFULL + st), 2 * SM::TILE_BYTES);
          const int h = hk * g + iter.hh;
#pragma unroll 1
          for (int kb = 0; kb < KBLK; ++kb) {
            tma_load_3d(sbase + SM::Q_OFF + st * SM::TILE_BYTES + kb * BLK_BYTES, &tm_q, BAR(B_QDOFULL + st), kb * 64, h, iter.q_row);
            tma_load_3d(sbase + SM::DO_OFF + st * SM::TILE_BYTES + kb * BLK_BYTES, &tm_do, BAR(B_QDOFULL + st), kb * 64, h, iter.q_row);
          }
        }
      }
    } else if (warp == 1 && lane == 0) {
      // ------------------------------------------------------------------ UMMA issuer
      constexpr uint32_t IDESC_ST = make_idesc(128, 128, 0, 0);   // K-major x K-major -> [keys][queries]
      constexpr uint32_t IDESC_ACC = make_idesc(128, D, 0, 1);    // TMEM A, MN-major B -> dV, dK
      constexpr uint32_t IDESC_DQ = DQ_T ? make_idesc(128, 128, 1, 1)   // K^T (MN-major) x dS^T (MN-major)
                                         : make_idesc(128, D, 1, 1);    // dS (MN-major) x K (MN-major)
      uint32_t n = 0, it = 0;
      bool ok = true;
      const uint32_t kbase = sbase + SM::K_OFF, vbase = sbase + SM::V_OFF, dsbase = sbase + SM::DS_OFF;
      while (ok) {
        const uint32_t slot = n & 1;
        ok = mbar_wait(BAR(B_WFULL + slot), (n >> 1) & 1, wctx, 141);
        if (!ok) break;
        const int unit = work_ring[2 * slot];
        mbar_arrive(BAR(B_WEMPTY + slot));
        if (unit < 0) break;
        const int32_t* U = a.units + (size_t)unit * FCP_BWD_UNIT_W;
        const int n_iter = __ldg(U + BU_COST) * g;
        ok = mbar_wait(BAR(B_KVFULL), n & 1, wctx, 120);
        if (!ok) break;
        // Software pipeline over the unit's tiles: trip i issues T3, T4, T5 of tile i and T1, T2 of tile
        // i + 1; trip -1 only starts the first tile.  `it` counts the tiles whose T1/T2 have been issued.
        // Each barrier is looked at (mbar_test) one UMMA batch before it is needed.
        bool p_ready = false;
#pragma unroll 1
        for (int i = -1; i < n_iter && ok; ++i) {
          const bool cur = i >= 0, next = i + 1 < n_iter;
          const uint32_t st = (it + 1) % BWD_QDO_STAGES, st_next = it % BWD_QDO_STAGES;   // tile i is tile it - 1
          const uint32_t qbase = sbase + SM::Q_OFF + st * SM::TILE_BYTES, dobase = sbase + SM::DO_OFF + st * SM::TILE_BYTES;
          bool q_ready = false, ds_ready = false;
          if (cur) {
            // T3: dV += P^T dO
            if (!p_ready) ok = mbar_wait(BAR(B_PFULL), (it - 1) & 1, wctx, 123);
            if (ok && i == 0) ok = mbar_wait(BAR(B_ACCEMPTY), (n & 1) ^ 1, wctx, 124);
            if (!ok) break;
            if (next) q_ready = mbar_test(BAR(B_QDOFULL + st_next), (it / BWD_QDO_STAGES) & 1);
            tc_fence_after();
            umma_loop_ts(true, tmem + C_DV, tmem + C_S, true, dobase, IDESC_ACC, i > 0 ? 1u : 0u);
          }
          // T1 of the next tile: S^T has been read by the math warps and P^T is consumed in order
          if (next) {
            if (!q_ready) ok = mbar_wait(BAR(B_QDOFULL + st_next), (it / BWD_QDO_STAGES) & 1, wctx, 126);
            if (!ok) break;
            if (cur) ds_ready = mbar_test(BAR(B_DSFULL), (it - 1) & 1);
            tc_fence_after();
            umma_loop_kk<D / 16>(true, tmem + C_S, kbase, sbase + SM::Q_OFF + st_next * SM::TILE_BYTES, IDESC_ST);
            tc_commit(BAR(B_SFULL));
          }
          if (cur) {
            // T5: dQ tile, handed to the drain warps at once; T4: dK += dS^T Q runs while they read it.
            // Both take dS^T from shared memory (K-major A for T4, MN-major B for T5).
            if (!ds_ready) ok = mbar_wait(BAR(B_DSFULL), (it - 1) & 1, wctx, 125);
            if (!ok) break;
            tc_fence_after();
            if (DQ_T) umma_loop_mm(true, tmem + C_DP, kbase, dsbase, IDESC_DQ);
            else umma_loop_mm(true, tmem + C_DP, dsbase, kbase, IDESC_DQ);
            tc_commit(BAR(B_DQFULL));
            umma_loop_km(true, tmem + C_DK, dsbase, qbase, IDESC_ACC, i > 0 ? 1u : 0u);
            tc_commit(BAR(B_QDOFREE + st));
          }
          // T2 of the next tile once the drain warps have emptied the dQ tile of the one before it
          p_ready = false;
          if (next) {
            ok = mbar_wait(BAR(B_DQEMPTY), (it & 1) ^ 1, wctx, 127);
            if (!ok) break;
            p_ready = mbar_test(BAR(B_PFULL), it & 1);
            tc_fence_after();
            umma_loop_kk<D / 16>(true, tmem + C_DP, vbase, sbase + SM::DO_OFF + st_next * SM::TILE_BYTES, IDESC_ST);
            tc_commit(BAR(B_DPFULL));
            ++it;
          }
        }
        if (!ok) break;
        tc_commit(BAR(B_ACCFULL));
        tc_commit(BAR(B_KVFREE));
        ++n;
      }
    }
  } else if (warp < 4 + BWD_MATH_WARPS) {
    // ------------------------------------------------------------------ math warps: C1, C2
    asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
    const int rb = warp & 3;                    // TMEM lane quarter
    const int half = (warp - 4) >> 2;           // which 64 of the 128 query columns
    const int row = rb * 32 + lane;             // key row of S^T / dP^T
    const int mtid = threadIdx.x - 128;         // 0..255 among the math threads
    const uint32_t t_s = tmem_addr(tmem, rb * 32, C_S + half * 64), t_dp = tmem_addr(tmem, rb * 32, C_DP + half * 64);
    uint8_t* ds_row = smem + SM::DS_OFF + half * BLK_BYTES + row * 128;
    // this thread's share of the per-query-row statistics: lse2 (threads 0..127) or delta (128..255)
    const float* my_rows = (mtid < 128 ? a.lse2_t : a.delta_t) + (mtid & 127);
    auto load_row = [&](const BwdIter& x, int hk) -> float {
      const int64_t t = (int64_t)x.q_row + (mtid & 127);
      return t < a.T ? __ldg(my_rows + (int64_t)((hk - a.hk_begin) * g + x.hh) * a.t_stride + x.q_row) : 0.f;
    };
    uint32_t n = 0, it = 0;
    bool ok = true;
    while (true) {
      int hk = 0;
      const int32_t* U = next_work(n++, hk, ok);
      if (!U) break;
      const int kv_row0 = __ldg(U + BU_KV_ROW0), kv_rows = __ldg(U + BU_KV_ROWS);
      // first query that sees this thread's key row: the key itself, or the begin of its span
      const int first_q = (a.first_query != nullptr && row < kv_rows) ? __ldg(a.first_query + kv_row0 + row) : kv_row0 + row;
      BwdIter iter;
      iter.init(U, a.qranges, g);
      float pre = load_row(iter, hk);
#pragma unroll 1
      for (; iter.valid; ++it) {
        const int q_row = iter.q_row, q_valid = iter.q_valid;
        const bool causal = iter.causal;
        // Per-query-row statistics of this tile -> shared memory, double buffered by tile parity: a
        // thread that gets here has passed the previous tile's barrier, so every thread has finished
        // the tile before that one, the last reader of this buffer.  The next tile's values are
        // fetched now and stay in flight while this tile is processed.
        float* s_rows = (float*)(smem + SM::ROWS_OFF) + (it & 1) * 256;      // lse2[128] | delta[128]
        s_rows[mtid] = pre;
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_ROWS));
        iter.advance();
        if (iter.valid) pre = load_row(iter, hk);
        ok = mbar_wait_warp(BAR(B_ROWS), it & 1, wctx, 134);
        if (!ok) break;
        const float* s_lse = s_rows + half * 64;
        const float* s_delta = s_rows + 128 + half * 64;
        const bool need_mask = causal || q_valid < 128 || kv_rows < 128;   // uniform across the CTA

        ok = mbar_wait_warp(BAR(B_SFULL), it & 1, wctx, 130);
        if (!ok) break;
        tc_fence_after();
        // P^T of this key row and column half as bf16 pairs: pa = query columns [0,32), pb = [32,64).
        // C1 and C2 run as two rolled trips of 32 columns; between the trips the pair arrays rotate
        // (register arrays cannot be indexed by the trip), which halves the code of this loop.
        uint32_t pa[16], pb[16] = {};
        unsigned long long keep = ~0ull;
        if (need_mask) {
          // valid query columns of this key row, relative to this warp's half: [lo, hi).  Bit j of
          // `keep` = column j survives; applied to the packed pairs.
          const int hi = min(64, max(0, (row < kv_rows ? q_valid : 0) - half * 64));
          const int lo = min(64, max(0, (causal ? first_q - q_row : 0) - half * 64));
          keep = (hi > lo) ? ((hi == 64 ? ~0ull : ((1ull << hi) - 1)) & ~((1ull << lo) - 1)) : 0ull;
        }
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          uint32_t sv[32];
          tmem_ld32(t_s + c * 32, sv);
#pragma unroll
          for (int j = 0; j < 16; ++j) pa[j] = pb[j];
          tc_wait_ld();
          const float* lse_c = s_lse + c * 32;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 l4 = *reinterpret_cast<const float4*>(lse_c + 4 * i);
            const float p0 = ex2(fmaf(__uint_as_float(sv[4 * i]), a.scale_log2, -l4.x));
            const float p1 = ex2(fmaf(__uint_as_float(sv[4 * i + 1]), a.scale_log2, -l4.y));
            const float p2 = ex2(fmaf(__uint_as_float(sv[4 * i + 2]), a.scale_log2, -l4.z));
            const float p3 = ex2(fmaf(__uint_as_float(sv[4 * i + 3]), a.scale_log2, -l4.w));
            pb[2 * i] = pack_bf16(p0, p1);
            pb[2 * i + 1] = pack_bf16(p2, p3);
          }
          if (need_mask) {
            const uint32_t k32 = (uint32_t)(keep >> (32 * c));
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const uint32_t b2 = (k32 >> (2 * j)) & 3u;
              pb[j] &= (b2 & 1u ? 0x0000ffffu : 0u) | (b2 & 2u ? 0xffff0000u : 0u);
            }
          }
          tmem_st16(t_s + c * 16, pb);            // over this warp's own, already loaded, columns
        }
        tc_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_PFULL));

        ok = mbar_wait_warp(BAR(B_DPFULL), it & 1, wctx, 131);
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 2; ++c) {
          uint32_t dv_[32];
          tmem_ld32(t_dp + c * 32, dv_);
          tc_wait_ld();
          const float* delta_c = s_delta + c * 32;
          uint32_t out[16];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float4 d4 = *reinterpret_cast<const float4*>(delta_c + 4 * i);
            const uint32_t pp = pa[2 * i], pq = pa[2 * i + 1];
            const float d0 = __uint_as_float(pp << 16) * fmaf(__uint_as_float(dv_[4 * i]), a.scale, -d4.x);
            const float d1 = __uint_as_float(pp & 0xffff0000u) * fmaf(__uint_as_float(dv_[4 * i + 1]), a.scale, -d4.y);
            const float d2 = __uint_as_float(pq << 16) * fmaf(__uint_as_float(dv_[4 * i + 2]), a.scale, -d4.z);
            const float d3 = __uint_as_float(pq & 0xffff0000u) * fmaf(__uint_as_float(dv_[4 * i + 3]), a.scale, -d4.w);
            out[2 * i] = pack_bf16(d0, d1);
            out[2 * i + 1] = pack_bf16(d2, d3);
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) pa[j] = pb[j];
          // 32 values -> shared memory, keys x queries with queries contiguous (the K-major A operand
          // of the dK product and the MN-major B operand of the dQ product): 4 x 16-byte chunks, 128-byte swizzle
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int cc = c * 4 + ch;                          // 16-byte chunk within this half's 128-byte row
            uint4 v4 = make_uint4(out[ch * 4], out[ch * 4 + 1], out[ch * 4 + 2], out[ch * 4 + 3]);
            *reinterpret_cast<uint4*>(ds_row + ((cc ^ (row & 7)) << 4)) = v4;
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(BAR(B_DSFULL));
      }
      if (!ok) break;
    }
  } else {
    // ------------------------------------------------------------------ drain warps: C3, dK/dV epilogue
    asm volatile("setmaxnreg.inc.sync.aligned.u32 176;");
    const int rb = warp & 3;
    const int row = rb * 32 + lane;             // TMEM lane: head-dim index of dQ^T (or query row), key row of dK/dV
    const uint32_t t_dq = tmem_addr(tmem, rb * 32, C_DP);
    const uint32_t t_dv = tmem_addr(tmem, rb * 32, C_DV), t_dk = tmem_addr(tmem, rb * 32, C_DK);
    uint32_t n = 0, it = 0;
    bool ok = true;
    while (true) {
      int hk = 0;
      const int32_t* U = next_work(n, hk, ok);
      if (!U) break;
      const int kv_row0 = __ldg(U + BU_KV_ROW0), kv_rows = __ldg(U + BU_KV_ROWS);
      BwdIter iter;
#pragma unroll 1
      for (iter.init(U, a.qranges, g); iter.valid; iter.advance(), ++it) {
        const int h = (hk - a.hk_begin) * g + iter.hh;   // head index within the accumulators of this pass
        const int q_row = iter.q_row, q_valid = iter.q_valid;
        ok = mbar_wait_warp(BAR(B_DQFULL), it & 1, wctx, 132);
        if (!ok) break;
        tc_fence_after();
        if constexpr (DQ_T) {
          // thread = head-dim index, columns = queries: a warp adds 32 consecutive floats per query.
          char* dst = reinterpret_cast<char*>(a.dq_acc + ((int64_t)q_row * a.hq_acc + h) * D + row);
          const int64_t stride = (int64_t)a.hq_acc * D * 4;
          if (q_valid == 128) {
            // whole tile into registers, columns handed back at once, then the reductions: they are
            // slow (L2 round trips) and must not sit between the tile and the issuer's next product
            uint32_t qa[64], qb[64];
#pragma unroll
            for (int c = 0; c < 2; ++c) {
              tmem_ld32(t_dq + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&qa[c * 32]));
              tmem_ld32(t_dq + 64 + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&qb[c * 32]));
            }
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(BAR(B_DQEMPTY));
            // two rolled trips of 64 reductions (the second half moves down in between): half the
            // code of a fully unrolled tile, which matters more to the instruction cache than the moves.
            // The reductions are paced (a short sleep after every 16) so that they spread over the time
            // a tile takes: sent back to back they keep the load/store queues of the SM full, and every
            // barrier poll and shared-memory access of the other warps then waits behind them.  Measured:
            // any pause that sums to 1.2-2 us per tile gives the same gain; 3 us makes this warp the bound.
#pragma unroll 1
            for (int hlf = 0; hlf < 2; ++hlf) {
#pragma unroll
              for (int c = 0; c < 64; ++c) {
                red_add_f32(reinterpret_cast<float*>(dst), __uint_as_float(qa[c]));
                dst += stride;
                if ((c & 15) == 15) __nanosleep(200);
              }
#pragma unroll
              for (int c = 0; c < 64; ++c) qa[c] = qb[c];
            }
          } else {
            // ragged tile (end of a chunk): rolled loop over 16-query slices
#pragma unroll 1
            for (int c16 = 0; c16 < 8; ++c16) {
              uint32_t qv[16];
              tmem_ld16(t_dq + c16 * 16, qv);
              tc_wait_ld();
              if (c16 == 7) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(BAR(B_DQEMPTY));
              }
              const int nv = q_valid - c16 * 16;
#pragma unroll
              for (int c = 0; c < 16; ++c) {
                if (c < nv) red_add_f32(reinterpret_cast<float*>(dst), __uint_as_float(qv[c]));
                dst += stride;
              }
            }
          }
        } else {
          float* dst = a.dq_acc + (((int64_t)q_row + row) * a.hq_acc + h) * D;
#pragma unroll 1
          for (int c16 = 0; c16 < D / 16; ++c16) {
            uint32_t qv[16];
            tmem_ld16(t_dq + c16 * 16, qv);
            tc_wait_ld();
            if (c16 == D / 16 - 1) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(BAR(B_DQEMPTY));
            }
            if (row < q_valid) {
#pragma unroll
              for (int c = 0; c < 16; c += 4)
                red_add_v4_f32(dst + c16 * 16 + c, __uint_as_float(qv[c]), __uint_as_float(qv[c + 1]),
                               __uint_as_float(qv[c + 2]), __uint_as_float(qv[c + 3]));
            }
          }
        }
      }
      if (!ok) break;
      // unit epilogue: dK, dV rows of this key tile
      ok = mbar_wait_warp(BAR(B_ACCFULL), n & 1, wctx, 133);
      ++n;
      if (!ok) break;
      tc_fence_after();
      const int64_t orow = ((int64_t)kv_row0 + row) * a.hkv + hk;
#pragma unroll 1
      for (int which = 0; which < 2; ++which) {
        __nv_bfloat16* dst = (which == 0 ? a.dv : a.dk) + orow * D;
        const uint32_t t_acc = which == 0 ? t_dv : t_dk;
#pragma unroll 1
        for (int c = 0; c < D / 16; ++c) {
          uint32_t av[16];
          tmem_ld16(t_acc + c * 16, av);
          tc_wait_ld();
          if (row < kv_rows) {
#pragma unroll
            for (int i = 0; i < 16; i += 8) {
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(av[i]), __uint_as_float(av[i + 1]));
              v4.y = pack_bf16(__uint_as_float(av[i + 2]), __uint_as_float(av[i + 3]));
              v4.z = pack_bf16(__uint_as_float(av[i + 4]), __uint_as_float(av[i + 5]));
              v4.w = pack_bf16(__uint_as_float(av[i + 6]), __uint_as_float(av[i + 7]));
              *reinterpret_cast<uint4*>(dst + c * 16 + i) = v4;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR(B_ACCEMPTY));
    }
  }

  wait_teardown(wctx);
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace fcp
