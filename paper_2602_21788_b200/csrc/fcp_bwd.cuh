// Backward attention over the block plan, grouped by KV chunk: the derivative of Eq. 1 of the paper
// with the causal mask.  One persistent grid; a work unit = (128-key tile of a KV chunk, KV head).
// The unit keeps its K and V tiles in shared memory and dK, dV in tensor memory while it walks over
// every (Q tile, query head of the group) of every block pair that attends to the chunk:
//
//   S^T  = K Q^T                       (UMMA, smem x smem)      TMEM cols [  0,128)
//   dP^T = V dO^T                      (UMMA, smem x smem)      TMEM cols [128,256)
//   P^T  = exp2(S^T*c - lse2[q])       (CUDA cores, thread = key row), bf16 over S^T
//   dV  += P^T dO                      (UMMA, TMEM x smem)      TMEM cols [256,384)
//   dS^T = scale * P^T o (dP^T - delta[q])                      bf16 over dP^T, and to smem
//   dK  += dS^T Q                      (UMMA, TMEM x smem)      TMEM cols [384,512)
//   dQ   = dS K                        (UMMA, smem x smem)      over S^T; fp32 atomics to the dQ accumulator
//
// Roles: warp 0 TMA producer, warp 1 UMMA issuer, warps 2..5 element-wise math and epilogues.
#pragma once
#include "fcp_plan.hpp"
#include "sm100_ptx.cuh"

namespace fcp {

constexpr int BWD_THREADS = 192;
constexpr int BWD_QDO_STAGES = 2;

template <int D>
struct BwdSmem {
  static constexpr int TILE_BYTES = 128 * D * 2;
  static constexpr int K_OFF = 0;
  static constexpr int V_OFF = TILE_BYTES;
  static constexpr int DS_OFF = 2 * TILE_BYTES;                         // [2][128 keys][64 q] bf16, swizzled
  static constexpr int Q_OFF = DS_OFF + 128 * 128 * 2;
  static constexpr int DO_OFF = Q_OFF + BWD_QDO_STAGES * TILE_BYTES;
  static constexpr int ROWS_OFF = DO_OFF + BWD_QDO_STAGES * TILE_BYTES;  // lse2[128], delta[128] fp32
  static constexpr int BAR_OFF = ROWS_OFF + 1024;
  static constexpr int N_BARS = 2 + 2 * BWD_QDO_STAGES + 9;
  static constexpr int MISC_OFF = BAR_OFF + N_BARS * 8;
  static constexpr int TOTAL = MISC_OFF + 16;
  static constexpr int DYN_BYTES = TOTAL + 1024;
};

struct BwdArgs {
  const int32_t* units;     // [n_units][8]
  const int32_t* qranges;   // [n][4]
  int32_t n_units, hq, hkv;
  int64_t T, t_stride;
  float scale, scale_log2;
  const float* delta_t;     // [hq][t_stride]
  const float* lse2_t;      // [hq][t_stride], log2 units
  float* dq_acc;            // [T][hq][D] fp32, zero-initialised
  __nv_bfloat16* dk;        // [T][hkv][D]
  __nv_bfloat16* dv;
  int32_t* status;
};

// Walks the (Q range, Q tile, head-of-group) iterations of one unit in the order every role uses.
// f(q_row, q_valid, causal_tile, head_in_group) returns false to stop.
template <class F>
__device__ __forceinline__ void bwd_for_each_iter(const int32_t* U, const int32_t* qranges, int g, F&& f) {
  const int first = __ldg(U + BU_FIRST_QRANGE), nq = __ldg(U + BU_N_QRANGES), kv_tile = __ldg(U + BU_KV_TILE);
  for (int r = 0; r < nq; ++r) {
    const int32_t* Q = qranges + (size_t)(first + r) * FCP_BWD_QRANGE_W;
    const int qb = __ldg(Q + BQ_BEGIN), qe = __ldg(Q + BQ_END), diag = __ldg(Q + BQ_DIAG);
    for (int t = diag ? kv_tile : 0; qb + t * 128 < qe; ++t) {
      const int q_row = qb + t * 128;
      const int q_valid = min(128, qe - q_row);
      for (int hh = 0; hh < g; ++hh)
        if (!f(q_row, q_valid, diag && t == kv_tile, hh)) return;
    }
  }
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

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = sbase + SM::BAR_OFF;
  auto BAR = [&](int i) { return bar0 + 8u * (uint32_t)i; };
  const int B_KVFULL = 0, B_KVFREE = 1, B_QDOFULL = 2, B_QDOFREE = 2 + BWD_QDO_STAGES, B0 = 2 + 2 * BWD_QDO_STAGES;
  const int B_SFULL = B0, B_DPFULL = B0 + 1, B_PFULL = B0 + 2, B_DSFULL = B0 + 3, B_DQFULL = B0 + 4,
            B_DQEMPTY = B0 + 5, B_ACCFULL = B0 + 6, B_ACCEMPTY = B0 + 7, B_ROWS = B0 + 8;
  volatile uint32_t* tmem_slot = (volatile uint32_t*)(smem + SM::MISC_OFF);
  volatile int* abort_flag = (volatile int*)(smem + SM::MISC_OFF + 4);
  const WaitCtx wctx{abort_flag, a.status};
  float* s_lse = (float*)(smem + SM::ROWS_OFF);
  float* s_delta = s_lse + 128;

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
    mbar_init(BAR(B_PFULL), 128);
    mbar_init(BAR(B_DSFULL), 128);
    mbar_init(BAR(B_DQFULL), 1);
    mbar_init(BAR(B_DQEMPTY), 128);
    mbar_init(BAR(B_ACCFULL), 1);
    mbar_init(BAR(B_ACCEMPTY), 128);
    mbar_init(BAR(B_ROWS), 128);
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
  const int64_t n_work = (int64_t)a.n_units * a.hkv;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t ucnt = 0, it = 0;
      bool ok = true;
      for (int64_t w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
        const int32_t* U = a.units + (size_t)(w / a.hkv) * FCP_BWD_UNIT_W;
        const int hk = (int)(w % a.hkv);
        const int kv_row0 = __ldg(U + BU_KV_ROW0);
        ok = mbar_wait(BAR(B_KVFREE), (ucnt & 1) ^ 1, wctx, 110);
        ++ucnt;
        if (!ok) break;
        mbar_expect_tx(BAR(B_KVFULL), 2 * SM::TILE_BYTES);
        for (int kb = 0; kb < KBLK; ++kb) {
          tma_load_3d(sbase + SM::K_OFF + kb * BLK_BYTES, &tm_k, BAR(B_KVFULL), kb * 64, hk, kv_row0);
          tma_load_3d(sbase + SM::V_OFF + kb * BLK_BYTES, &tm_v, BAR(B_KVFULL), kb * 64, hk, kv_row0);
        }
        bwd_for_each_iter(U, a.qranges, g, [&](int q_row, int, bool, int hh) {
          const uint32_t st = it % BWD_QDO_STAGES;
          ok = mbar_wait(BAR(B_QDOFREE + st), ((it / BWD_QDO_STAGES) & 1) ^ 1, wctx, 111);
          if (!ok) return false;
          mbar_expect_tx(BAR(B_QDOFULL + st), 2 * SM::TILE_BYTES);
          const int h = hk * g + hh;
          for (int kb = 0; kb < KBLK; ++kb) {
            tma_load_3d(sbase + SM::Q_OFF + st * SM::TILE_BYTES + kb * BLK_BYTES, &tm_q, BAR(B_QDOFULL + st), kb * 64, h, q_row);
            tma_load_3d(sbase + SM::DO_OFF + st * SM::TILE_BYTES + kb * BLK_BYTES, &tm_do, BAR(B_QDOFULL + st), kb * 64, h, q_row);
          }
          ++it;
          return true;
        });
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC_ST = make_idesc(128, 128, 0, 0);   // K-major x K-major -> [keys][queries]
      constexpr uint32_t IDESC_ACC = make_idesc(128, D, 0, 1);    // TMEM A, MN-major B -> dV, dK
      constexpr uint32_t IDESC_DQ = make_idesc(128, D, 1, 1);     // MN-major A (dS), MN-major B (K)
      uint32_t ucnt = 0, it = 0;
      bool ok = true;
      for (int64_t w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
        const int32_t* U = a.units + (size_t)(w / a.hkv) * FCP_BWD_UNIT_W;
        const int n_iter = __ldg(U + BU_COST) * g;
        ok = mbar_wait(BAR(B_KVFULL), ucnt & 1, wctx, 120);
        if (!ok) break;
        const uint32_t kbase = sbase + SM::K_OFF, vbase = sbase + SM::V_OFF, dsbase = sbase + SM::DS_OFF;
        for (int i = 0; i < n_iter && ok; ++i, ++it) {
          const uint32_t st = it % BWD_QDO_STAGES;
          const uint32_t qbase = sbase + SM::Q_OFF + st * SM::TILE_BYTES, dobase = sbase + SM::DO_OFF + st * SM::TILE_BYTES;
          ok = mbar_wait(BAR(B_QDOFULL + st), (it / BWD_QDO_STAGES) & 1, wctx, 121);
          if (ok) ok = mbar_wait(BAR(B_DQEMPTY), (it & 1) ^ 1, wctx, 122);   // S^T columns drained of the last dQ
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * BLK_BYTES + (k % 4) * 32;
            umma_ss(tmem + C_S, make_sdesc(kbase + off, 16, 1024), make_sdesc(qbase + off, 16, 1024), IDESC_ST, k > 0);
          }
          tc_commit(BAR(B_SFULL));
#pragma unroll
          for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * BLK_BYTES + (k % 4) * 32;
            umma_ss(tmem + C_DP, make_sdesc(vbase + off, 16, 1024), make_sdesc(dobase + off, 16, 1024), IDESC_ST, k > 0);
          }
          tc_commit(BAR(B_DPFULL));
          // dV += P^T dO
          ok = mbar_wait(BAR(B_PFULL), it & 1, wctx, 123);
          if (ok && i == 0) ok = mbar_wait(BAR(B_ACCEMPTY), (ucnt & 1) ^ 1, wctx, 124);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_ts(tmem + C_DV, tmem + C_S + k * 8, make_sdesc(dobase + k * 2048, BLK_BYTES, 1024), IDESC_ACC,
                    (i > 0 || k > 0) ? 1u : 0u);
          // dK += dS^T Q ; dQ = dS K
          ok = mbar_wait(BAR(B_DSFULL), it & 1, wctx, 125);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_ts(tmem + C_DK, tmem + C_DP + k * 8, make_sdesc(qbase + k * 2048, BLK_BYTES, 1024), IDESC_ACC,
                    (i > 0 || k > 0) ? 1u : 0u);
#pragma unroll
          for (int k = 0; k < 8; ++k)
            umma_ss(tmem + C_S, make_sdesc(dsbase + k * 2048, BLK_BYTES, 1024), make_sdesc(kbase + k * 2048, BLK_BYTES, 1024),
                    IDESC_DQ, k > 0);
          tc_commit(BAR(B_DQFULL));
          tc_commit(BAR(B_QDOFREE + st));
        }
        if (!ok) break;
        tc_commit(BAR(B_ACCFULL));
        tc_commit(BAR(B_KVFREE));
        ++ucnt;
      }
    }
  } else {
    // ------------------------------------------------------------------ element-wise math, epilogues
    const int rb = warp & 3;
    const int row = rb * 32 + lane;             // key row of S^T / dP^T / dK / dV; query row of dQ
    const int ctid = threadIdx.x - 64;          // 0..127 among the compute threads
    const uint32_t t_s = tmem_addr(tmem, rb * 32, C_S), t_dp = tmem_addr(tmem, rb * 32, C_DP);
    const uint32_t t_dv = tmem_addr(tmem, rb * 32, C_DV), t_dk = tmem_addr(tmem, rb * 32, C_DK);
    uint8_t* ds_row = smem + SM::DS_OFF + row * 128;
    uint32_t ucnt = 0, it = 0;
    bool ok = true;
    for (int64_t w = blockIdx.x; w < n_work && ok; w += gridDim.x) {
      const int32_t* U = a.units + (size_t)(w / a.hkv) * FCP_BWD_UNIT_W;
      const int hk = (int)(w % a.hkv);
      const int kv_row0 = __ldg(U + BU_KV_ROW0), kv_rows = __ldg(U + BU_KV_ROWS);
      bwd_for_each_iter(U, a.qranges, g, [&](int q_row, int q_valid, bool causal, int hh) {
        const int h = hk * g + hh;
        // Per-query-row statistics of this tile -> shared memory.  Overwriting the previous tile's
        // values is safe: this thread has seen that tile's dQ, which the issuer only produces
        // after all 128 threads finished reading them.  The mbarrier orders the writes before the
        // reads below.
        {
          const int64_t t = (int64_t)q_row + ctid;
          const bool in = t < a.T;
          s_lse[ctid] = in ? __ldg(a.lse2_t + (int64_t)h * a.t_stride + t) : 0.f;
          s_delta[ctid] = in ? __ldg(a.delta_t + (int64_t)h * a.t_stride + t) : 0.f;
        }
        mbar_arrive(BAR(B_ROWS));
        ok = mbar_wait_warp(BAR(B_ROWS), it & 1, wctx, 134);
        if (!ok) return false;
        // valid query columns of this key row: [lo, hi)
        const int hi = row < kv_rows ? q_valid : 0;
        const int lo = causal ? max(0, kv_row0 + row - q_row) : 0;

        ok = mbar_wait_warp(BAR(B_SFULL), it & 1, wctx, 130);
        if (!ok) return false;
        tc_fence_after();
        uint32_t pk[64];                        // P^T of this key row, bf16 pairs
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t sv[32];
          tmem_ld32(t_s + c * 32, sv);
          tc_wait_ld();
          uint32_t out[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int c0 = c * 32 + 2 * i;
            const float2 l2 = *reinterpret_cast<const float2*>(s_lse + c0);
            float p0 = ex2(fmaf(__uint_as_float(sv[2 * i]), a.scale_log2, -l2.x));
            float p1 = ex2(fmaf(__uint_as_float(sv[2 * i + 1]), a.scale_log2, -l2.y));
            p0 = (c0 >= lo && c0 < hi) ? p0 : 0.f;
            p1 = (c0 + 1 >= lo && c0 + 1 < hi) ? p1 : 0.f;
            out[i] = pack_bf16(p0, p1);
            pk[c * 16 + i] = out[i];
          }
          tmem_st16(t_s + c * 16, out);
        }
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(BAR(B_PFULL));

        ok = mbar_wait_warp(BAR(B_DPFULL), it & 1, wctx, 131);
        if (!ok) return false;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t dv_[32];
          tmem_ld32(t_dp + c * 32, dv_);
          tc_wait_ld();
          uint32_t out[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const int c0 = c * 32 + 2 * i;
            const float2 dl = *reinterpret_cast<const float2*>(s_delta + c0);
            const uint32_t pp = pk[c * 16 + i];
            const float p0 = __uint_as_float(pp << 16), p1 = __uint_as_float(pp & 0xffff0000u);
            const float d0 = p0 * (__uint_as_float(dv_[2 * i]) - dl.x) * a.scale;
            const float d1 = p1 * (__uint_as_float(dv_[2 * i + 1]) - dl.y) * a.scale;
            out[i] = pack_bf16(d0, d1);
          }
          tmem_st16(t_dp + c * 16, out);
          // the same 32 values -> shared memory, keys x queries with queries contiguous
          // (MN-major A operand of dQ = dS K): 4 x 16-byte chunks, 128-byte swizzle
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int chunk = c * 4 + ch;                       // 16-byte chunk index along the 128 queries
            const int blk = chunk >> 3, cc = chunk & 7;
            uint4 v4 = make_uint4(out[ch * 4], out[ch * 4 + 1], out[ch * 4 + 2], out[ch * 4 + 3]);
            *reinterpret_cast<uint4*>(ds_row + blk * BLK_BYTES + ((cc ^ (row & 7)) << 4)) = v4;
          }
        }
        fence_proxy_async_smem();
        tc_wait_st();
        tc_fence_before();
        mbar_arrive(BAR(B_DSFULL));

        // dQ tile: rows are queries now
        ok = mbar_wait_warp(BAR(B_DQFULL), it & 1, wctx, 132);
        if (!ok) return false;
        tc_fence_after();
        float* dst = a.dq_acc + (((int64_t)q_row + row) * a.hq + h) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t qv[32];
          tmem_ld32(t_s + c * 32, qv);
          tc_wait_ld();
          if (row < q_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              atomicAdd(reinterpret_cast<float4*>(dst + c * 32 + i),
                        make_float4(__uint_as_float(qv[i]), __uint_as_float(qv[i + 1]), __uint_as_float(qv[i + 2]),
                                    __uint_as_float(qv[i + 3])));
          }
        }
        tc_fence_before();
        mbar_arrive(BAR(B_DQEMPTY));
        ++it;
        return true;
      });
      if (!ok) break;
      // unit epilogue: dK, dV rows of this key tile
      ok = mbar_wait_warp(BAR(B_ACCFULL), ucnt & 1, wctx, 133);
      ++ucnt;
      if (!ok) break;
      tc_fence_after();
      const int64_t orow = ((int64_t)kv_row0 + row) * a.hkv + hk;
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        __nv_bfloat16* dst = (which == 0 ? a.dv : a.dk) + orow * D;
        const uint32_t t_acc = which == 0 ? t_dv : t_dk;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t av[32];
          tmem_ld32(t_acc + c * 32, av);
          tc_wait_ld();
          if (row < kv_rows) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(av[i]), __uint_as_float(av[i + 1]));
              v4.y = pack_bf16(__uint_as_float(av[i + 2]), __uint_as_float(av[i + 3]));
              v4.z = pack_bf16(__uint_as_float(av[i + 4]), __uint_as_float(av[i + 5]));
              v4.w = pack_bf16(__uint_as_float(av[i + 6]), __uint_as_float(av[i + 7]));
              *reinterpret_cast<uint4*>(dst + c * 32 + i) = v4;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(BAR(B_ACCEMPTY));
    }
  }

  if (*abort_flag) {
    const unsigned long long t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

}  // namespace fcp
