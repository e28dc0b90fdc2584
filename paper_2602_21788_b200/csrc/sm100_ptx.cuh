// Thin wrappers over the sm_100a PTX this library uses: mbarrier, TMA tile loads, tcgen05
// (tensor memory allocation, UMMA issue/commit, TMEM loads/stores) and the descriptor encodings.
// Every wait is bounded: after FCP_WAIT_NS without progress the waiter records a status word and
// returns false, and the caller unwinds to its teardown instead of spinning.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

namespace fcp {

constexpr unsigned long long FCP_WAIT_NS = 2000000000ull;  // 2 s: far above any legitimate wait

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ uint32_t globaltimer_lo() {
  uint32_t t;
  asm volatile("mov.u32 %0, %%globaltimer_lo;" : "=r"(t));
  return t;
}

__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
}

// ----------------------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.shared::cta.b64 st, [%0];\n\t}" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("{\n\t.reg .b64 st;\n\tmbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1;\n\t}" ::"r"(bar),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Non-blocking look at a barrier phase.  An issuing thread sends this ahead of a batch of UMMAs for
// the barrier it will need after the batch: the answer travels while the batch is issued, and the
// blocking wait (whose round trip through a busy memory pipe costs hundreds of clocks even when the
// phase completed long ago) is skipped if it was already there.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// Shared per-CTA abort word + global status word.  `abort_flag` lives in shared memory: zero while
// all is well, else 0x40000000 | the `where` code of the first wait that gave up.
struct WaitCtx {
  volatile int* abort_flag;
  int* status;                // global: [0] status, [1] where, [2] block, [3] reserved
  uint32_t limit_ns;          // a wait gives up after this long without progress (below 2^32 ns)
};

// Bounded wait.  Returns false if the CTA is aborting (this waiter timed out, or another did).
// The body is inlined at every wait site of the persistent kernels, so it is kept to a few
// instructions: the slow path only looks at the clock and the abort word; the status words are
// written once, by wait_teardown().
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx& ctx, int where) {
  // A phase that completed earlier is seen by the non-blocking test in tens of clocks; try_wait, which
  // may park the thread, was measured at 600-900 clocks on a busy SM even then.
  if (mbar_test(bar, parity)) return true;
  uint32_t spins = 0, t0 = 0;
#pragma unroll 1
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 2047u) == 0) {
      // low word of the nanosecond timer: differences are exact modulo 2^32 (4.29 s), enough for
      // the 2 s limit as long as the clock is looked at more often than that
      const uint32_t now = globaltimer_lo();
      if (spins == 2048u) t0 = now;
      const int flag = *ctx.abort_flag;
      if (flag != 0 || now - t0 > ctx.limit_ns) {
        if (flag == 0) *ctx.abort_flag = 0x40000000 | where;
        return false;
      }
    }
  }
  return true;
}

// End of a persistent kernel, called by every thread before the CTA-wide barrier that precedes the
// release of tensor memory.  If a wait gave up: record who (first CTA wins) and give copies and MMAs
// still in flight time to land before the CTA's shared and tensor memory are released.
__device__ __forceinline__ void wait_teardown(const WaitCtx& ctx) {
  const int flag = *ctx.abort_flag;
  if (flag == 0) return;
  if (threadIdx.x == 0 && atomicCAS(ctx.status, 0, -6 /* FCP_ERR_TIMEOUT */) == 0) {
    ctx.status[1] = flag & 0xFFFF;
    ctx.status[2] = (int)blockIdx.x;
    ctx.status[3] = 0;
  }
  const unsigned long long t0 = globaltimer_ns();
  while (globaltimer_ns() - t0 < 2000000ull) __nanosleep(1000);
}

// Same, for code that must stay warp-convergent (it is followed by .sync.aligned instructions):
// the verdict is made uniform across the warp.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const WaitCtx& ctx, int where) {
  const bool ok = mbar_wait(bar, parity, ctx, where);
  return __all_sync(0xffffffffu, ok);
}

// ----------------------------------------------------------------------------- TMA
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// 3-D tile load (coordinates innermost first), completion counted in bytes on `bar`.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* m, uint32_t bar, int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst), "l"(m), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ----------------------------------------------------------------------------- tcgen05
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Arrive on `bar` once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]   (bf16 in, fp32 accumulate)
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B.
//   bits [4,6) D format (1 = f32), [7,10) A format (1 = bf16), [10,13) B format (1 = bf16),
//   bit 15 A major (0 = K, 1 = MN), bit 16 B major, [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Shared-memory matrix descriptor for 128-byte-swizzled tiles whose rows are 128 bytes wide
// (64 bf16) and whose 8-row groups are 1024 bytes apart — exactly what a TMA box of 64 x rows
// elements with 128B swizzle writes.
//   bits [0,14) start address >> 4, [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4,
//   [46,48) version (1 on sm_100), [61,64) layout (2 = 128-byte swizzle).
// K-major operand (the 64 contiguous elements run along K): SBO = 1024 is the step between 8-row
// groups along M/N; LBO is not used by the swizzled K-major form.
// MN-major operand (the 64 contiguous elements run along M/N): SBO = 1024 is the step between
// 8-row groups along K; LBO is the step between 64-element column blocks along M/N.
__device__ __forceinline__ uint64_t make_sdesc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// The same descriptor split into its two 32-bit words, so that issue loops only add a byte offset to
// the low word (start address field) instead of rebuilding all 64 bits per instruction.
__device__ __forceinline__ uint32_t sdesc_lo(uint32_t saddr, uint32_t lbo_bytes) {
  return ((saddr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ constexpr uint32_t sdesc_hi(uint32_t sbo_bytes) {
  return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ uint64_t sdesc_pack(uint32_t lo, uint32_t hi) {
  uint64_t d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}

// One 128 x N x (16*KSTEPS) product.  Fully unrolled with the descriptor offsets folded into
// constants: a single thread issues these, and a rolled loop's dependent integer arithmetic (about
// 85 clocks per trip) would be slower than the 64 clocks a 128x128x16 UMMA takes to execute.
// K-major A and B tiles of [128][64]-element swizzled blocks: K step k lives in block k/4 at byte
// offset (k%4)*32 of every row.
//
// The helpers are called by a whole warp in uniform control flow; only `leader` (one lane) executes
// the UMMA itself.  Keeping the descriptor arithmetic outside the divergent part lets the compiler
// hold it in the warp-uniform datapath instead of re-deriving it in one lane's registers.
template <int KSTEPS>
__device__ __forceinline__ void umma_loop_kk(bool leader, uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, uint32_t idesc) {
  const uint32_t hi = sdesc_hi(1024), alo = sdesc_lo(a_addr, 16), blo = sdesc_lo(b_addr, 16);
#pragma unroll
  for (int k = 0; k < KSTEPS; ++k) {
    const uint32_t off = (uint32_t)(k >> 2) * (16384u >> 4) + (uint32_t)(k & 3) * 2u;
    const uint64_t ad = sdesc_pack(alo + off, hi), bd = sdesc_pack(blo + off, hi);
    if (leader) umma_ss(d_tmem, ad, bd, idesc, k > 0 ? 1u : 0u);
  }
}
// MN-major A and B (64-element blocks 16384 bytes apart): K step k is rows [16k, 16k+16) = +2048 bytes.
__device__ __forceinline__ void umma_loop_mm(bool leader, uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, uint32_t idesc) {
  const uint32_t hi = sdesc_hi(1024), alo = sdesc_lo(a_addr, 16384), blo = sdesc_lo(b_addr, 16384);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint64_t ad = sdesc_pack(alo + k * 128u, hi), bd = sdesc_pack(blo + k * 128u, hi);
    if (leader) umma_ss(d_tmem, ad, bd, idesc, k > 0 ? 1u : 0u);
  }
}
// K-major A ([128][64]-element swizzled blocks, as in umma_loop_kk) and MN-major B (as in
// umma_loop_mm); `acc` = accumulate into D from the first step on.
__device__ __forceinline__ void umma_loop_km(bool leader, uint32_t d_tmem, uint32_t a_addr, uint32_t b_addr, uint32_t idesc,
                                             uint32_t acc) {
  const uint32_t hi = sdesc_hi(1024), alo = sdesc_lo(a_addr, 16), blo = sdesc_lo(b_addr, 16384);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t off = (uint32_t)(k >> 2) * (16384u >> 4) + (uint32_t)(k & 3) * 2u;
    const uint64_t ad = sdesc_pack(alo + off, hi), bd = sdesc_pack(blo + k * 128u, hi);
    if (leader) umma_ss(d_tmem, ad, bd, idesc, (acc | (k > 0)) ? 1u : 0u);
  }
}
// A from TMEM (bf16 pairs, 8 columns per K step; with `split` the second four steps start at
// column 64), MN-major B.  `acc` = accumulate into D from the first step on.
__device__ __forceinline__ void umma_loop_ts(bool leader, uint32_t d_tmem, uint32_t a_tmem, bool split, uint32_t b_addr,
                                             uint32_t idesc, uint32_t acc) {
  const uint32_t hi = sdesc_hi(1024), blo = sdesc_lo(b_addr, 16384);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t col = (split && k >= 4) ? 64u + 8u * (k - 4) : 8u * k;
    const uint64_t bd = sdesc_pack(blo + k * 128u, hi);
    if (leader) umma_ts(d_tmem, a_tmem + col, bd, idesc, (acc | (k > 0)) ? 1u : 0u);
  }
}
__device__ __forceinline__ void tc_commit_if(bool leader, uint32_t bar) {
  if (leader) tc_commit(bar);
}

// TMEM address = (lane << 16) | column.
__device__ __forceinline__ uint32_t tmem_addr(uint32_t base, uint32_t lane, uint32_t col) {
  return base + (lane << 16) + col;
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp gets lane (lane_base + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]),
        "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]),
        "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

}  // namespace fcp
