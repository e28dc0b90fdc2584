// Device side of libfcp: launchers behind the C ABI, the HBM-bound kernels (LSE merge, backward
// preprocess, dQ conversion) and the glue around the tensor-core kernels of fcp_fwd.cuh and
// fcp_bwd.cuh.  No call here allocates device memory except fcp_plan_upload.
#include <cstdio>
#include <cstring>
#include <vector>

#include "fcp_bwd.cuh"
#include "fcp_fwd.cuh"

using namespace fcp;

#define FCP_CUDA_CHECK(expr)                                                             \
  do {                                                                                   \
    cudaError_t e_ = (expr);                                                             \
    if (e_ != cudaSuccess) {                                                             \
      fcp_set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(e_), __FILE__, __LINE__); \
      return FCP_ERR_CUDA;                                                               \
    }                                                                                    \
  } while (0)

// ---------------------------------------------------------------------------------------------
// Tensor maps
// ---------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = (EncodeTiledFn)p;
  return fn;
}

// bf16 tensor [T][H][D]; box = 64 columns x 1 head x `box_rows` tokens, 128-byte swizzle, zero fill.
int make_thd_map(CUtensorMap* m, const void* base, int64_t T, int H, int D, int box_rows) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) {
    fcp_set_error("cuTensorMapEncodeTiled is not available from the driver");
    return FCP_ERR_CUDA;
  }
  if (((uintptr_t)base & 15) != 0) {
    fcp_set_error("tensor base %p is not 16-byte aligned", base);
    return FCP_ERR_INVALID_ARG;
  }
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)H * D * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    fcp_set_error("cuTensorMapEncodeTiled failed with %d", (int)r);
    return FCP_ERR_CUDA;
  }
  return FCP_OK;
}

// Records an event pair around a kernel launch when the plan is in profiling mode.
struct ProfScope {
  const fcp_plan* plan;
  int kind;
  cudaStream_t st;
  int slot = -1;
  ProfScope(const fcp_plan* p, int k, cudaStream_t s) : plan(p), kind(k), st(s) {
    if (plan && plan->profiling && plan->prof_ev[kind][0][0]) {
      slot = (int)(plan->prof_n[kind] % 64);
      cudaEventRecord((cudaEvent_t)plan->prof_ev[kind][slot][0], st);
    }
  }
  ~ProfScope() {
    if (slot >= 0) {
      cudaEventRecord((cudaEvent_t)plan->prof_ev[kind][slot][1], st);
      ++plan->prof_n[kind];
    }
  }
};

int check_plan(const fcp_plan* plan) {
  if (!plan) {
    fcp_set_error("plan is NULL");
    return FCP_ERR_INVALID_ARG;
  }
  if (!plan->d_blob) {
    fcp_set_error("plan has no device copy: call fcp_plan_upload first");
    return FCP_ERR_NOT_UPLOADED;
  }
  return FCP_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// LSE merge (HBM bound).  One thread owns 8 output columns of one (token, head) row: it reads the
// row's slot log-sum-exps, forms the exact weights and accumulates 2 x 128-bit loads per slot.
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) fcp_merge_kernel(const int32_t* __restrict__ units, const int32_t* __restrict__ slot_offset,
                                                        const int32_t* __restrict__ slot_rows, const float* __restrict__ o_partial,
                                                        const float* __restrict__ lse_partial, int head_begin, int head_count,
                                                        int hq, __nv_bfloat16* __restrict__ o, float* __restrict__ o_f32, float* __restrict__ lse) {
  constexpr int TPR = D / 8;                 // threads per (token, head) row
  constexpr int RPP = 256 / TPR;             // rows per pass
  const int32_t* U = units + (size_t)blockIdx.x * FCP_MERGE_UNIT_W;
  const int tok0 = U[MU_TOK_BEGIN], ntok = U[MU_N_TOK], chunk = U[MU_CHUNK], ctok0 = U[MU_CHUNK_TOK_BEGIN];
  const int s0 = slot_offset[chunk], ns = slot_offset[chunk + 1] - s0;
  const int sub = threadIdx.x % TPR, rloc = threadIdx.x / TPR;
  const int n_rows = ntok * head_count;
  for (int r = rloc; r < n_rows; r += RPP) {
    const int t = tok0 + r / head_count, hl = r % head_count;
    const int64_t rel = t - ctok0;
    float m = -INFINITY;
    for (int s = 0; s < ns; ++s) m = fmaxf(m, __ldg(lse_partial + ((int64_t)slot_rows[s0 + s] + rel) * head_count + hl));
    float z = 0.f;
    for (int s = 0; s < ns; ++s)
      z += __expf(__ldg(lse_partial + ((int64_t)slot_rows[s0 + s] + rel) * head_count + hl) - m);
    const float L = m + __logf(z);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int s = 0; s < ns; ++s) {
      const int64_t prow = ((int64_t)slot_rows[s0 + s] + rel) * head_count + hl;
      const float wgt = __expf(__ldg(lse_partial + prow) - L);
      const float4* src = reinterpret_cast<const float4*>(o_partial + prow * D + sub * 8);
      const float4 a0 = __ldcs(src), a1 = __ldcs(src + 1);
      acc[0] += wgt * a0.x; acc[1] += wgt * a0.y; acc[2] += wgt * a0.z; acc[3] += wgt * a0.w;
      acc[4] += wgt * a1.x; acc[5] += wgt * a1.y; acc[6] += wgt * a1.z; acc[7] += wgt * a1.w;
    }
    const int64_t orow = (int64_t)t * hq + head_begin + hl;
    uint4 pk;
    pk.x = pack_bf16(acc[0], acc[1]); pk.y = pack_bf16(acc[2], acc[3]);
    pk.z = pack_bf16(acc[4], acc[5]); pk.w = pack_bf16(acc[6], acc[7]);
    *reinterpret_cast<uint4*>(o + orow * D + sub * 8) = pk;
    if (o_f32) {
      float4* dst = reinterpret_cast<float4*>(o_f32 + orow * D + sub * 8);
      dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
      dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
    }
    if (sub == 0) lse[orow] = L;
  }
}

// ---------------------------------------------------------------------------------------------
// Backward preprocess (HBM bound): delta[h][t] = scale * sum_c dO[t,h,c] * O[t,h,c], and the forward LSE
// transposed to [h][t] in log2 units, the layout the backward kernel's per-tile loads want.
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) fcp_delta_kernel(const __nv_bfloat16* __restrict__ o, const __nv_bfloat16* __restrict__ d_o,
                                                        const float* __restrict__ lse, int64_t T, int hq, int h0, int hc,
                                                        int64_t t_stride, float scale, float* __restrict__ delta_t,
                                                        float* __restrict__ lse2_t) {
  // heads [h0, h0 + hc) of the [T][hq][D] tensors; the outputs hold hc heads, numbered from 0
  constexpr int TPR = D / 8;
  const int64_t row = ((int64_t)blockIdx.x * 256 + threadIdx.x) / TPR;   // (token, head of the pass) row
  const int sub = threadIdx.x % TPR;
  const int64_t t = row / hc;
  const int hl = (int)(row - t * hc);
  const int64_t src = t * hq + h0 + hl;
  float acc = 0.f;
  if (row < T * hc) {
    const uint4 a = *reinterpret_cast<const uint4*>(o + src * D + sub * 8);
    const uint4 b = *reinterpret_cast<const uint4*>(d_o + src * D + sub * 8);
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 fa = __bfloat1622float2(pa[i]), fb = __bfloat1622float2(pb[i]);
      acc += fa.x * fb.x + fa.y * fb.y;
    }
  }
#pragma unroll
  for (int off = TPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
  if (row < T * hc && sub == 0) {
    delta_t[hl * t_stride + t] = acc * scale;
    lse2_t[hl * t_stride + t] = lse[src] * 1.4426950408889634f;
  }
}

// fp32 dQ accumulator [T][hc][D] -> bf16 dq [T][hq][D], heads [h0, h0 + hc); n8 = T*hc*D/8 groups of
// eight values, row8 = hc*D/8 groups per token of the accumulator
__global__ void __launch_bounds__(256) fcp_dq_convert_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq,
                                                             int64_t n8, int64_t row8, int64_t dst_row8, int64_t dst_off8) {
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n8; i += (int64_t)gridDim.x * 256) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(acc) + 2 * i);
    const float4 b = __ldcs(reinterpret_cast<const float4*>(acc) + 2 * i + 1);
    uint4 pk;
    pk.x = pack_bf16(a.x, a.y); pk.y = pack_bf16(a.z, a.w);
    pk.z = pack_bf16(b.x, b.y); pk.w = pack_bf16(b.z, b.w);
    int64_t j = i;
    if (row8 != dst_row8) {
      const int64_t t = i / row8;
      j = t * dst_row8 + dst_off8 + (i - t * row8);
    }
    reinterpret_cast<uint4*>(dq)[j] = pk;
  }
}

// ---------------------------------------------------------------------------------------------
// Plan upload / destroy / status
// ---------------------------------------------------------------------------------------------
extern "C" int fcp_plan_upload(fcp_plan* plan, void* stream) {
  if (!plan) return FCP_ERR_INVALID_ARG;
  if (plan->d_blob) return FCP_OK;
  int dev = 0;
  FCP_CUDA_CHECK(cudaGetDevice(&dev));
  cudaDeviceProp prop;
  FCP_CUDA_CHECK(cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) {
    fcp_set_error("device %d is sm_%d%d; this library is built for sm_100a only", dev, prop.major, prop.minor);
    return FCP_ERR_CUDA;
  }
  plan->device = dev;
  plan->sm_count = prop.multiProcessorCount;
  constexpr int NT = 10;
  const std::vector<int32_t>* tabs[NT] = {&plan->fwd_units, &plan->bwd_units, &plan->bwd_qranges, &plan->merge_units,
                                          &plan->slot_offset, &plan->slot_rows, &plan->bwd_work, &plan->fused_units,
                                          &plan->row_limit, &plan->first_query};
  size_t off[NT + 1];
  size_t total = 256;  // status words first
  for (int i = 0; i < NT; ++i) {
    off[i] = total;
    total += (tabs[i]->size() * 4 + 255) / 256 * 256;
  }
  off[NT] = total;
  void* blob = nullptr;
  FCP_CUDA_CHECK(cudaMalloc(&blob, total));
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(blob, 0, 256, st);
  for (int i = 0; i < NT && e == cudaSuccess; ++i)
    if (!tabs[i]->empty())
      e = cudaMemcpyAsync((char*)blob + off[i], tabs[i]->data(), tabs[i]->size() * 4, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) {
    cudaFree(blob);
    fcp_set_error("plan upload failed: %s", cudaGetErrorString(e));
    return FCP_ERR_CUDA;
  }
  plan->d_blob = blob;
  plan->d_status = (int32_t*)blob;
  plan->d_fwd_units = (int32_t*)((char*)blob + off[0]);
  plan->d_bwd_units = (int32_t*)((char*)blob + off[1]);
  plan->d_bwd_qranges = (int32_t*)((char*)blob + off[2]);
  plan->d_merge_units = (int32_t*)((char*)blob + off[3]);
  plan->d_slot_offset = (int32_t*)((char*)blob + off[4]);
  plan->d_slot_rows = (int32_t*)((char*)blob + off[5]);
  plan->d_bwd_work = (int32_t*)((char*)blob + off[6]);
  plan->d_fused_units = (int32_t*)((char*)blob + off[7]);
  plan->d_row_limit = plan->row_limit.empty() ? nullptr : (int32_t*)((char*)blob + off[8]);
  plan->d_first_query = plan->first_query.empty() ? nullptr : (int32_t*)((char*)blob + off[9]);
  // opt in to the large dynamic shared memory of the tensor-core kernels once
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_fwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<64>::DYN_BYTES));
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_fwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<128>::DYN_BYTES));
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<64>::DYN_BYTES));
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<128>::DYN_BYTES));
  return FCP_OK;
}

extern "C" int fcp_plan_set_profiling(fcp_plan* plan, int32_t enable) {
  if (!plan) return FCP_ERR_INVALID_ARG;
  for (int k = 0; k < FCP_KERNEL_KINDS; ++k) {
    plan->prof_n[k] = 0;
    for (int i = 0; i < 64; ++i)
      for (int e = 0; e < 2; ++e) {
        if (enable && !plan->prof_ev[k][i][e]) {
          cudaEvent_t ev;
          FCP_CUDA_CHECK(cudaEventCreate(&ev));
          plan->prof_ev[k][i][e] = ev;
        } else if (!enable && plan->prof_ev[k][i][e]) {
          cudaEventDestroy((cudaEvent_t)plan->prof_ev[k][i][e]);
          plan->prof_ev[k][i][e] = nullptr;
        }
      }
  }
  plan->profiling = enable != 0;
  return FCP_OK;
}

extern "C" int fcp_plan_kernel_ms(const fcp_plan* plan, int32_t kind, int32_t* launches, float* mean_ms) {
  if (!plan || kind < 0 || kind >= FCP_KERNEL_KINDS || !launches || !mean_ms) return FCP_ERR_INVALID_ARG;
  const int n = (int)std::min<int64_t>(plan->prof_n[kind], 64);
  double sum = 0.0;
  for (int i = 0; i < n; ++i) {
    float ms = 0.f;
    FCP_CUDA_CHECK(cudaEventElapsedTime(&ms, (cudaEvent_t)plan->prof_ev[kind][i][0], (cudaEvent_t)plan->prof_ev[kind][i][1]));
    sum += ms;
  }
  *launches = (int32_t)plan->prof_n[kind];
  *mean_ms = n ? (float)(sum / n) : 0.f;
  return FCP_OK;
}

extern "C" int fcp_plan_destroy(fcp_plan* plan) {
  if (!plan) return FCP_OK;
  for (fcp_plan* g : plan->groups) fcp_plan_destroy(g);
  plan->groups.clear();
  for (void* e : plan->host_events) if (e) cudaEventDestroy((cudaEvent_t)e);
  plan->host_events.clear();
  if (plan->host_in) cudaStreamDestroy((cudaStream_t)plan->host_in);
  if (plan->host_out) cudaStreamDestroy((cudaStream_t)plan->host_out);
  plan->host_in = plan->host_out = nullptr;
  fcp_plan_set_profiling(plan, 0);
  if (plan->d_blob) cudaFree(plan->d_blob);
  delete plan;
  return FCP_OK;
}

extern "C" int fcp_last_device_status(const fcp_plan* plan, int32_t* status) {
  if (!status) return FCP_ERR_INVALID_ARG;
  int rc = check_plan(plan);
  if (rc != FCP_OK) return rc;
  FCP_CUDA_CHECK(cudaDeviceSynchronize());
  FCP_CUDA_CHECK(cudaMemcpy(status, plan->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost));
  // kernels launched by the host entry point report into the status words of its sequence groups
  for (const fcp_plan* g : plan->groups) {
    if (status[0] != 0) break;
    FCP_CUDA_CHECK(cudaMemcpy(status, g->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost));
  }
  return FCP_OK;
}

// scratch layout of fcp_attn_bwd: [dq fp32 accumulator T*hq*D] [delta_t hq*Tpad] [lse2_t hq*Tpad]
static inline int64_t bwd_tpad(int64_t T) { return (T + 255) / 256 * 256 + 256; }

extern "C" int fcp_plan_workspace_bytes(const fcp_plan* plan, int32_t heads_per_pass, int64_t* o_partial_bytes,
                                        int64_t* lse_partial_bytes, int64_t* bwd_scratch_bytes) {
  if (!plan || heads_per_pass <= 0 || heads_per_pass > plan->params.hq) {
    fcp_set_error("fcp_plan_workspace_bytes: invalid argument");
    return FCP_ERR_INVALID_ARG;
  }
  const int64_t D = plan->params.head_dim;
  if (o_partial_bytes) *o_partial_bytes = plan->R * heads_per_pass * D * 4;
  if (lse_partial_bytes) *lse_partial_bytes = plan->R * heads_per_pass * 4;
  if (bwd_scratch_bytes)
    *bwd_scratch_bytes = plan->T * plan->params.hq * D * 4 + 2 * bwd_tpad(plan->T) * plan->params.hq * 4;
  return FCP_OK;
}

// ---------------------------------------------------------------------------------------------
// Compute calls
// ---------------------------------------------------------------------------------------------
static int check_heads(const fcp_plan* plan, int head_begin, int head_count) {
  if (head_begin < 0 || head_count <= 0 || head_begin + head_count > plan->params.hq) {
    fcp_set_error("head range [%d, %d) outside [0, %d)", head_begin, head_begin + head_count, plan->params.hq);
    return FCP_ERR_INVALID_ARG;
  }
  return FCP_OK;
}

namespace {
// `fused`: run the merge-on-the-fly units (every row goes straight to o_direct / lse_direct, no partials)
int launch_fwd(const fcp_plan* plan, const void* q, const void* k, const void* v, int32_t head_begin, int32_t head_count,
               float* o_partial, float* lse_partial, void* o_direct, float* lse_direct, float* o_f32_direct, bool fused,
               void* stream) {
  int rc = check_plan(plan);
  if (rc != FCP_OK) return rc;
  if (!q || !k || !v || (!fused && (!o_partial || !lse_partial)) || (fused && (!o_direct || !lse_direct))) {
    fcp_set_error("forward attention: NULL buffer");
    return FCP_ERR_INVALID_ARG;
  }
  if ((rc = check_heads(plan, head_begin, head_count)) != FCP_OK) return rc;
  if (!fused && !plan->row_limit.empty()) {
    fcp_set_error("the per-item partial path (fcp_attn_fwd, fcp_attn_fwd_merged) is causal only; a plan with "
                  "bidirectional spans runs through fcp_attn_fwd_fused");
    return FCP_ERR_UNSUPPORTED;
  }
  const fcp_params& P = plan->params;
  CUtensorMap tq, tk, tv;
  if ((rc = make_thd_map(&tq, q, plan->T, P.hq, P.head_dim, 128)) != FCP_OK) return rc;
  if ((rc = make_thd_map(&tk, k, plan->T, P.hkv, P.head_dim, 128)) != FCP_OK) return rc;
  if ((rc = make_thd_map(&tv, v, plan->T, P.hkv, P.head_dim, 128)) != FCP_OK) return rc;
  FwdArgs a;
  a.units = fused ? plan->d_fused_units : plan->d_fwd_units;
  a.n_units = (int32_t)((fused ? plan->fused_units.size() : plan->fwd_units.size()) / FCP_FWD_UNIT_W);
  a.head_begin = head_begin;
  a.head_count = head_count;
  a.hq = P.hq;
  a.hkv = P.hkv;
  {
    const int g = P.hq / P.hkv;
    a.head_group = (head_begin % g == 0 && head_count % g == 0) ? g : 1;
  }
  a.scale_log2 = P.scale * 1.4426950408889634f;
  a.o_partial = o_partial;
  a.lse_partial = lse_partial;
  a.o_direct = (__nv_bfloat16*)o_direct;
  a.lse_direct = lse_direct;
  a.o_f32_direct = o_f32_direct;
  a.row_limit = fused ? plan->d_row_limit : nullptr;
  a.status = plan->d_status;
  const int64_t n_work = (int64_t)a.n_units * head_count;
  const int grid = (int)std::min<int64_t>(n_work, plan->sm_count);
  if (grid == 0) return FCP_OK;
  cudaStream_t st = (cudaStream_t)stream;
  // the grid's work counter (the status block's word 17; word 16 is the backward grid's)
  a.work_counter = plan->d_status + 17;
  FCP_CUDA_CHECK(cudaMemsetAsync(a.work_counter, 0, sizeof(int32_t), st));
  ProfScope prof(plan, 0, st);
  if (P.head_dim == 128)
    fcp_fwd_kernel<128><<<grid, FWD_THREADS, FwdSmem<128>::DYN_BYTES, st>>>(tq, tk, tv, a);
  else
    fcp_fwd_kernel<64><<<grid, FWD_THREADS, FwdSmem<64>::DYN_BYTES, st>>>(tq, tk, tv, a);
  FCP_CUDA_CHECK(cudaGetLastError());
  return FCP_OK;
}

int launch_merge(const fcp_plan* plan, const float* o_partial, const float* lse_partial, int32_t head_begin,
                 int32_t head_count, void* o, float* o_f32, float* lse, int n_units, void* stream) {
  const fcp_params& P = plan->params;
  if (n_units == 0) return FCP_OK;
  cudaStream_t st = (cudaStream_t)stream;
  ProfScope prof(plan, 1, st);
  if (P.head_dim == 128)
    fcp_merge_kernel<128><<<n_units, 256, 0, st>>>(plan->d_merge_units, plan->d_slot_offset, plan->d_slot_rows, o_partial,
                                                   lse_partial, head_begin, head_count, P.hq, (__nv_bfloat16*)o, o_f32, lse);
  else
    fcp_merge_kernel<64><<<n_units, 256, 0, st>>>(plan->d_merge_units, plan->d_slot_offset, plan->d_slot_rows, o_partial,
                                                  lse_partial, head_begin, head_count, P.hq, (__nv_bfloat16*)o, o_f32, lse);
  FCP_CUDA_CHECK(cudaGetLastError());
  return FCP_OK;
}
}  // namespace

extern "C" int fcp_attn_fwd(const fcp_plan* plan, const void* q, const void* k, const void* v, int32_t head_begin,
                            int32_t head_count, float* o_partial, float* lse_partial, void* stream) {
  return launch_fwd(plan, q, k, v, head_begin, head_count, o_partial, lse_partial, nullptr, nullptr, nullptr, false, stream);
}

extern "C" int fcp_attn_fwd_fused(const fcp_plan* plan, const void* q, const void* k, const void* v, int32_t head_begin,
                                  int32_t head_count, void* o, float* o_f32, float* lse, void* stream) {
  return launch_fwd(plan, q, k, v, head_begin, head_count, nullptr, nullptr, o, lse, o_f32, true, stream);
}

extern "C" int fcp_attn_fwd_merged(const fcp_plan* plan, const void* q, const void* k, const void* v, int32_t head_begin,
                                   int32_t head_count, float* o_partial, float* lse_partial, void* o, float* lse,
                                   void* stream) {
  if (!o || !lse) {
    fcp_set_error("fcp_attn_fwd_merged: NULL output");
    return FCP_ERR_INVALID_ARG;
  }
  int rc = launch_fwd(plan, q, k, v, head_begin, head_count, o_partial, lse_partial, o, lse, nullptr, false, stream);
  if (rc != FCP_OK) return rc;
  return launch_merge(plan, o_partial, lse_partial, head_begin, head_count, o, nullptr, lse, plan->n_merge_multi, stream);
}

extern "C" int fcp_lse_merge(const fcp_plan* plan, const float* o_partial, const float* lse_partial,
                             int32_t head_begin, int32_t head_count, void* o, float* o_f32, float* lse,
                             void* stream) {
  int rc = check_plan(plan);
  if (rc != FCP_OK) return rc;
  if (!o_partial || !lse_partial || !o || !lse) {
    fcp_set_error("fcp_lse_merge: NULL buffer");
    return FCP_ERR_INVALID_ARG;
  }
  if ((rc = check_heads(plan, head_begin, head_count)) != FCP_OK) return rc;
  if (!plan->row_limit.empty()) {
    fcp_set_error("fcp_lse_merge: the per-item partial path is causal only; this plan has bidirectional spans");
    return FCP_ERR_UNSUPPORTED;
  }
  return launch_merge(plan, o_partial, lse_partial, head_begin, head_count, o, o_f32, lse,
                      (int)(plan->merge_units.size() / FCP_MERGE_UNIT_W), stream);
}

namespace {
// Everything the backward launches need besides the caller's tensors: device tables, status words,
// work counter, SM count.  fcp_attn_bwd_heads takes them from the uploaded plan, fcp_attn_bwd_noalloc
// from the built-in arena.
struct BwdTables {
  const int32_t *units, *qranges, *order, *first_query;
  int32_t* status;
  int32_t* counter;
  int sm_count;
};

// scratch layout: [dq fp32 accumulator T*hc*D] [delta_t hc*Tpad] [lse2_t hc*Tpad], hc = query heads of the pass
int64_t bwd_scratch_need(const fcp_plan* plan, int kv_heads) {
  const int64_t hc = (int64_t)kv_heads * (plan->params.hq / plan->params.hkv);
  return plan->T * hc * plan->params.head_dim * 4 + 2 * bwd_tpad(plan->T) * hc * 4;
}

// Launches of one backward pass over KV heads [hk0, hk0 + hkc): clear, delta, main kernel, dQ conversion.
// `prof` may be NULL (no event timing).
int run_bwd(const fcp_plan* plan, const BwdTables& tb, const void* q, const void* k, const void* v, const void* o,
            const void* d_o, const float* lse, int hk0, int hkc, void* dq, void* dk, void* dv, void* scratch,
            const fcp_plan* prof, cudaStream_t st) {
  const fcp_params& P = plan->params;
  const int64_t T = plan->T, D = P.head_dim;
  const int g = P.hq / P.hkv;
  const int h0 = hk0 * g, hc = hkc * g;
  const int64_t need = bwd_scratch_need(plan, hkc);
  const int64_t tpad = bwd_tpad(T);
  float* dq_acc = (float*)scratch;
  float* delta_t = dq_acc + T * hc * D;
  float* lse2_t = delta_t + tpad * hc;
  int rc;
  {
    ProfScope ps(prof, 2, st);
    FCP_CUDA_CHECK(cudaMemsetAsync(scratch, 0, (size_t)need, st));
    FCP_CUDA_CHECK(cudaMemsetAsync(tb.counter, 0, sizeof(int32_t), st));
    const int64_t blocks = (T * hc * (D / 8) + 255) / 256;
    if (D == 128)
      fcp_delta_kernel<128><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, T, P.hq,
                                                              h0, hc, tpad, P.scale, delta_t, lse2_t);
    else
      fcp_delta_kernel<64><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)d_o, lse, T, P.hq,
                                                             h0, hc, tpad, P.scale, delta_t, lse2_t);
    FCP_CUDA_CHECK(cudaGetLastError());
  }
  CUtensorMap tq, tk, tv, tdo;
  if ((rc = make_thd_map(&tq, q, T, P.hq, (int)D, 128)) != FCP_OK) return rc;
  if ((rc = make_thd_map(&tk, k, T, P.hkv, (int)D, 128)) != FCP_OK) return rc;
  if ((rc = make_thd_map(&tv, v, T, P.hkv, (int)D, 128)) != FCP_OK) return rc;
  if ((rc = make_thd_map(&tdo, d_o, T, P.hq, (int)D, 128)) != FCP_OK) return rc;
  BwdArgs a;
  a.units = tb.units;
  a.qranges = tb.qranges;
  a.work = tb.order;
  a.n_units = (int32_t)plan->bwd_work.size();
  a.n_work = a.n_units * hkc;
  a.counter = tb.counter;
  a.hq = P.hq;
  a.hkv = P.hkv;
  a.hk_begin = hk0;
  a.hq_acc = hc;
  a.T = T;
  a.t_stride = tpad;
  a.scale = P.scale;
  a.scale_log2 = P.scale * 1.4426950408889634f;
  a.delta_t = delta_t;
  a.lse2_t = lse2_t;
  a.dq_acc = dq_acc;
  a.first_query = tb.first_query;
  a.dk = (__nv_bfloat16*)dk;
  a.dv = (__nv_bfloat16*)dv;
  a.status = tb.status;
  const int grid = (int)std::min<int64_t>(a.n_work, tb.sm_count);
  if (grid > 0) {
    ProfScope ps(prof, 3, st);
    if (D == 128)
      fcp_bwd_kernel<128><<<grid, BWD_THREADS, BwdSmem<128>::DYN_BYTES, st>>>(tq, tk, tv, tdo, a);
    else
      fcp_bwd_kernel<64><<<grid, BWD_THREADS, BwdSmem<64>::DYN_BYTES, st>>>(tq, tk, tv, tdo, a);
    FCP_CUDA_CHECK(cudaGetLastError());
  }
  {
    const int64_t n8 = T * hc * D / 8;
    const int blocks = (int)std::min<int64_t>((n8 + 255) / 256, (int64_t)tb.sm_count * 16);
    ProfScope ps(prof, 4, st);
    fcp_dq_convert_kernel<<<blocks, 256, 0, st>>>(dq_acc, (__nv_bfloat16*)dq, n8, hc * D / 8, P.hq * D / 8, h0 * D / 8);
    FCP_CUDA_CHECK(cudaGetLastError());
  }
  return FCP_OK;
}
}  // namespace

extern "C" int fcp_plan_bwd_scratch_bytes(const fcp_plan* plan, int32_t kv_head_count, int64_t* bytes) {
  if (!plan || !bytes || kv_head_count <= 0 || kv_head_count > plan->params.hkv) {
    fcp_set_error("fcp_plan_bwd_scratch_bytes: invalid argument");
    return FCP_ERR_INVALID_ARG;
  }
  *bytes = bwd_scratch_need(plan, kv_head_count);
  return FCP_OK;
}

extern "C" int fcp_attn_bwd_heads(const fcp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                                  const void* d_o, const float* lse, int32_t kv_head_begin, int32_t kv_head_count,
                                  void* dq, void* dk, void* dv, void* scratch, int64_t scratch_bytes, void* stream) {
  int rc = check_plan(plan);
  if (rc != FCP_OK) return rc;
  if (!q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv || !scratch) {
    fcp_set_error("fcp_attn_bwd: NULL buffer");
    return FCP_ERR_INVALID_ARG;
  }
  if (kv_head_begin < 0 || kv_head_count <= 0 || kv_head_begin + kv_head_count > plan->params.hkv) {
    fcp_set_error("KV head range [%d, %d) outside [0, %d)", kv_head_begin, kv_head_begin + kv_head_count, plan->params.hkv);
    return FCP_ERR_INVALID_ARG;
  }
  const int64_t need = bwd_scratch_need(plan, kv_head_count);
  if (scratch_bytes < need) {
    fcp_set_error("fcp_attn_bwd: scratch of %lld bytes, %lld needed", (long long)scratch_bytes, (long long)need);
    return FCP_ERR_WORKSPACE;
  }
  const BwdTables tb{plan->d_bwd_units, plan->d_bwd_qranges, plan->d_bwd_work, plan->d_first_query, plan->d_status,
                     plan->d_status + 16, plan->sm_count};
  return run_bwd(plan, tb, q, k, v, o, d_o, lse, kv_head_begin, kv_head_count, dq, dk, dv, scratch, plan,
                 (cudaStream_t)stream);
}

extern "C" int fcp_attn_bwd(const fcp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                            const void* d_o, const float* lse, void* dq, void* dk, void* dv, void* scratch,
                            int64_t scratch_bytes, void* stream) {
  if (!plan) {
    fcp_set_error("plan is NULL");
    return FCP_ERR_INVALID_ARG;
  }
  return fcp_attn_bwd_heads(plan, q, k, v, o, d_o, lse, 0, plan->params.hkv, dq, dk, dv, scratch, scratch_bytes, stream);
}

// ---------------------------------------------------------------------------------------------
// Whole path from host buffers
// ---------------------------------------------------------------------------------------------
namespace {
struct HostLayout {
  int64_t q, k, v, d_o, o, lse, dq, dk, dv, scratch, total;
};
inline int64_t al(int64_t x) { return (x + 255) / 256 * 256; }

HostLayout host_layout(const fcp_plan* plan) {
  const fcp_params& P = plan->params;
  const int64_t T = plan->T, D = P.head_dim;
  HostLayout L{};
  int64_t off = 0;
  auto take = [&](int64_t bytes) { int64_t o = off; off += al(bytes); return o; };
  L.q = take(T * P.hq * D * 2);
  L.k = take(T * P.hkv * D * 2);
  L.v = take(T * P.hkv * D * 2);
  L.d_o = take(T * P.hq * D * 2);
  L.o = take(T * P.hq * D * 2);
  L.lse = take(T * P.hq * 4);
  L.dq = take(T * P.hq * D * 2);
  L.dk = take(T * P.hkv * D * 2);
  L.dv = take(T * P.hkv * D * 2);
  L.scratch = take(bwd_scratch_need(plan, P.hkv));
  L.total = off;
  return L;
}
}  // namespace

extern "C" int fcp_host_workspace_bytes(const fcp_plan* plan, int64_t* bytes) {
  if (!plan || !bytes) return FCP_ERR_INVALID_ARG;
  *bytes = host_layout(plan).total;
  return FCP_OK;
}

namespace {
// Cuts the batch into runs of consecutive sequences of about equal token counts (at most 8 runs, at
// least about 8192 tokens each) and plans each run on its own: packed tensors are token-major, so a run
// is one contiguous slice of every tensor and can be copied, computed and copied back independently.
// Also creates the two copy streams and the events the host entry point orders its work with; all of
// it belongs to the plan and is released by fcp_plan_destroy.
int build_host_groups(const fcp_plan* plan, void* stream) {
  if (!plan->groups.empty()) return FCP_OK;
  const int B = plan->B;
  const int64_t T = plan->T;
  const int want = (int)std::max<int64_t>(1, std::min<int64_t>(std::min<int64_t>(8, B), T / 8192));
  std::vector<int32_t> lens(B), degs(B);
  for (int b = 0; b < B; ++b) {
    lens[b] = plan->cu_seqlens[b + 1] - plan->cu_seqlens[b];
    degs[b] = (plan->chunk_offset[b + 1] - plan->chunk_offset[b] - 1) / 2;
  }
  std::vector<fcp_plan*> groups;
  std::vector<int64_t> tok0;
  auto fail = [&](int rc) {
    for (fcp_plan* x : groups) fcp_plan_destroy(x);
    return rc;
  };
  int b0 = 0;
  for (int g = 0; g < want && b0 < B; ++g) {
    int b1 = b0 + 1;
    if (g == want - 1) {
      b1 = B;
    } else {
      const int64_t target = T * (g + 1) / want;
      while (b1 < B - (want - 1 - g) && plan->cu_seqlens[b1] < target) ++b1;
    }
    fcp_plan* sub = nullptr;
    int rc;
    if (plan->span_offset.empty()) {
      rc = fcp_plan_blocks(lens.data() + b0, degs.data() + b0, b1 - b0, &plan->params, &sub);
    } else {                                     // the run's spans, offsets counted from its first one
      std::vector<int32_t> so(b1 - b0 + 1);
      for (int b = b0; b <= b1; ++b) so[b - b0] = plan->span_offset[b] - plan->span_offset[b0];
      rc = fcp_plan_blocks_spans(lens.data() + b0, degs.data() + b0, b1 - b0, so.data(),
                                 plan->spans.data() + 2 * (size_t)plan->span_offset[b0], &plan->params, &sub);
    }
    if (rc == FCP_OK) rc = fcp_plan_upload(sub, stream);
    if (rc != FCP_OK) {
      if (sub) fcp_plan_destroy(sub);
      return fail(rc);
    }
    groups.push_back(sub);
    tok0.push_back(plan->cu_seqlens[b0]);
    b0 = b1;
  }
  tok0.push_back(T);
  // A group whose query tensor alone is hundreds of megabytes (one very long sequence) is additionally cut into
  // passes over whole KV heads, so that its copies overlap its own kernels too: at least ~256 MB of q per pass.
  std::vector<int32_t> passes;
  int64_t total_passes = 0;
  for (size_t g = 0; g < groups.size(); ++g) {
    const int64_t q_bytes = (tok0[g + 1] - tok0[g]) * plan->params.hq * plan->params.head_dim * 2;
    const int32_t np = (int32_t)std::max<int64_t>(1, std::min<int64_t>(plan->params.hkv, q_bytes / (int64_t(256) << 20)));
    passes.push_back(np);
    total_passes += np;
  }
  // streams and events: [0] start, [1] last copy out, then per (group, pass): q, k, v up; dO up; forward done; backward done
  cudaStream_t in = nullptr, out = nullptr;
  std::vector<void*> ev(2 + 4 * (size_t)total_passes, nullptr);
  cudaError_t e = cudaStreamCreateWithFlags(&in, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&out, cudaStreamNonBlocking);
  for (size_t i = 0; i < ev.size() && e == cudaSuccess; ++i) {
    cudaEvent_t x = nullptr;
    e = cudaEventCreateWithFlags(&x, cudaEventDisableTiming);
    ev[i] = x;
  }
  if (e != cudaSuccess) {
    for (void* x : ev) if (x) cudaEventDestroy((cudaEvent_t)x);
    if (in) cudaStreamDestroy(in);
    if (out) cudaStreamDestroy(out);
    fcp_set_error("fcp_attn_fwd_bwd_host: creating copy streams failed: %s", cudaGetErrorString(e));
    return fail(FCP_ERR_CUDA);
  }
  plan->host_in = in;
  plan->host_out = out;
  plan->host_events = std::move(ev);
  plan->groups = std::move(groups);
  plan->group_tok0 = std::move(tok0);
  plan->group_passes = std::move(passes);
  return FCP_OK;
}

// On any early exit of the host entry point: wait for the copies and kernels already queued, so that
// nothing still writes into the caller's buffers after the call has returned an error.
struct HostDrain {
  cudaStream_t a, b, c;
  bool armed = true;
  ~HostDrain() {
    if (!armed) return;
    cudaStreamSynchronize(a);
    cudaStreamSynchronize(b);
    cudaStreamSynchronize(c);
  }
};
}  // namespace

extern "C" int fcp_attn_fwd_bwd_host(const fcp_plan* plan, const void* q_host, const void* k_host, const void* v_host,
                                     const void* d_o_host, void* o_host, float* lse_host, void* dq_host, void* dk_host,
                                     void* dv_host, void* workspace, int64_t workspace_bytes, void* stream) {
  int rc = check_plan(plan);
  if (rc != FCP_OK) return rc;
  if (!q_host || !k_host || !v_host || !d_o_host || !o_host || !lse_host || !dq_host || !dk_host || !dv_host ||
      !workspace) {
    fcp_set_error("fcp_attn_fwd_bwd_host: NULL buffer");
    return FCP_ERR_INVALID_ARG;
  }
  const HostLayout L = host_layout(plan);
  if (L.total > workspace_bytes) {
    fcp_set_error("fcp_attn_fwd_bwd_host: workspace of %lld bytes, %lld needed", (long long)workspace_bytes,
                  (long long)L.total);
    return FCP_ERR_WORKSPACE;
  }
  cudaStream_t st = (cudaStream_t)stream;
  if ((rc = build_host_groups(plan, stream)) != FCP_OK) return rc;
  const fcp_params& P = plan->params;
  const int64_t D = P.head_dim;
  const int64_t rq = (int64_t)P.hq * D * 2, rkv = (int64_t)P.hkv * D * 2, rl = (int64_t)P.hq * 4;   // bytes per token
  char* w = (char*)workspace;
  const int G = (int)plan->groups.size();
  // Three streams: inputs of group g+1 come in and results of group g-1 go out while the kernels of
  // group g run on `stream`.  Everything is ordered after the work already queued on `stream` and is
  // complete when this call returns.
  cudaStream_t s_in = (cudaStream_t)plan->host_in, s_out = (cudaStream_t)plan->host_out;
  auto EV = [&](int i) { return (cudaEvent_t)plan->host_events[i]; };
  // Work is cut twice: into groups (runs of consecutive sequences: contiguous token slices) and, for large groups,
  // into passes over whole KV heads with their query heads (strided slices of every token row: 2-D copies).  The
  // forward pass of a slice needs q, k, v only: dO follows them and arrives while the forward kernel runs; o and
  // lse leave while the backward kernels run (they only read them).
  struct Slice { int g, hk0, hkc, ev0; };
  std::vector<Slice> slices;
  {
    int ev0 = 2;
    for (int g = 0; g < G; ++g) {
      const int np = plan->group_passes[g];
      const int per = (P.hkv + np - 1) / np;
      for (int hk0 = 0; hk0 < P.hkv; hk0 += per, ev0 += 4) slices.push_back(Slice{g, hk0, std::min(per, P.hkv - hk0), ev0});
    }
  }
  const int gq = P.hq / P.hkv;
  HostDrain drain{s_in, s_out, st};
  FCP_CUDA_CHECK(cudaEventRecord(EV(0), st));
  FCP_CUDA_CHECK(cudaStreamWaitEvent(s_in, EV(0), 0));
  FCP_CUDA_CHECK(cudaStreamWaitEvent(s_out, EV(0), 0));
  // copies of the heads [h0, h0 + hc) of nt token rows: width hc * bytes per head, pitch = the row of all heads
  auto copy_heads = [&](char* dst, const char* src, int64_t t0, int64_t nt, int64_t row_bytes, int64_t head_bytes, int h0, int hc,
                        cudaMemcpyKind kind, cudaStream_t cs) {
    return cudaMemcpy2DAsync(dst + t0 * row_bytes + h0 * head_bytes, (size_t)row_bytes, src + t0 * row_bytes + h0 * head_bytes,
                             (size_t)row_bytes, (size_t)(hc * head_bytes), (size_t)nt, kind, cs);
  };
  const int64_t hb = D * 2;   // bytes of one head of one token (bf16)
  for (const Slice& sl : slices) {
    const int64_t t0 = plan->group_tok0[sl.g], nt = plan->group_tok0[sl.g + 1] - t0;
    const int h0 = sl.hk0 * gq, hc = sl.hkc * gq;
    FCP_CUDA_CHECK(copy_heads(w + L.q, (const char*)q_host, t0, nt, rq, hb, h0, hc, cudaMemcpyHostToDevice, s_in));
    FCP_CUDA_CHECK(copy_heads(w + L.k, (const char*)k_host, t0, nt, rkv, hb, sl.hk0, sl.hkc, cudaMemcpyHostToDevice, s_in));
    FCP_CUDA_CHECK(copy_heads(w + L.v, (const char*)v_host, t0, nt, rkv, hb, sl.hk0, sl.hkc, cudaMemcpyHostToDevice, s_in));
    FCP_CUDA_CHECK(cudaEventRecord(EV(sl.ev0), s_in));
    FCP_CUDA_CHECK(copy_heads(w + L.d_o, (const char*)d_o_host, t0, nt, rq, hb, h0, hc, cudaMemcpyHostToDevice, s_in));
    FCP_CUDA_CHECK(cudaEventRecord(EV(sl.ev0 + 1), s_in));
  }
  for (const Slice& sl : slices) {
    const fcp_plan* sub = plan->groups[sl.g];
    const int64_t t0 = plan->group_tok0[sl.g], nt = plan->group_tok0[sl.g + 1] - t0;
    const int h0 = sl.hk0 * gq, hc = sl.hkc * gq;
    FCP_CUDA_CHECK(cudaStreamWaitEvent(st, EV(sl.ev0), 0));
    if ((rc = fcp_attn_fwd_fused(sub, w + L.q + t0 * rq, w + L.k + t0 * rkv, w + L.v + t0 * rkv, h0, hc, w + L.o + t0 * rq,
                                 nullptr, (float*)(w + L.lse + t0 * rl), st)) != FCP_OK)
      return rc;
    FCP_CUDA_CHECK(cudaEventRecord(EV(sl.ev0 + 2), st));
    FCP_CUDA_CHECK(cudaStreamWaitEvent(s_out, EV(sl.ev0 + 2), 0));
    FCP_CUDA_CHECK(copy_heads((char*)o_host, w + L.o, t0, nt, rq, hb, h0, hc, cudaMemcpyDeviceToHost, s_out));
    FCP_CUDA_CHECK(copy_heads((char*)lse_host, w + L.lse, t0, nt, rl, 4, h0, hc, cudaMemcpyDeviceToHost, s_out));
    FCP_CUDA_CHECK(cudaStreamWaitEvent(st, EV(sl.ev0 + 1), 0));
    if ((rc = fcp_attn_bwd_heads(sub, w + L.q + t0 * rq, w + L.k + t0 * rkv, w + L.v + t0 * rkv, w + L.o + t0 * rq,
                                 w + L.d_o + t0 * rq, (float*)(w + L.lse + t0 * rl), sl.hk0, sl.hkc, w + L.dq + t0 * rq,
                                 w + L.dk + t0 * rkv, w + L.dv + t0 * rkv, w + L.scratch, bwd_scratch_need(sub, sl.hkc), st)) != FCP_OK)
      return rc;
    FCP_CUDA_CHECK(cudaEventRecord(EV(sl.ev0 + 3), st));
    FCP_CUDA_CHECK(cudaStreamWaitEvent(s_out, EV(sl.ev0 + 3), 0));
    FCP_CUDA_CHECK(copy_heads((char*)dq_host, w + L.dq, t0, nt, rq, hb, h0, hc, cudaMemcpyDeviceToHost, s_out));
    FCP_CUDA_CHECK(copy_heads((char*)dk_host, w + L.dk, t0, nt, rkv, hb, sl.hk0, sl.hkc, cudaMemcpyDeviceToHost, s_out));
    FCP_CUDA_CHECK(copy_heads((char*)dv_host, w + L.dv, t0, nt, rkv, hb, sl.hk0, sl.hkc, cudaMemcpyDeviceToHost, s_out));
  }
  FCP_CUDA_CHECK(cudaEventRecord(EV(1), s_out));
  FCP_CUDA_CHECK(cudaStreamWaitEvent(st, EV(1), 0));
  FCP_CUDA_CHECK(cudaStreamSynchronize(st));
  drain.armed = false;
  return FCP_OK;
}

// ---------------------------------------------------------------------------------------------
// Backward pass for callers that must not allocate device memory
// ---------------------------------------------------------------------------------------------
// Everything the backward grid needs besides the caller's tensors lives in this one fixed array:
// status words and work counter, the plan's work tables, and the scratch of fcp_attn_bwd (fp32 dQ
// accumulator, delta and LSE rows).  Each GPU that loads the library carries the array until the
// process exits.  In host code `g_noalloc_arena` is only a handle for the runtime's symbol calls,
// never a device pointer: the address kernels may use comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_arena[FCP_NOALLOC_MAX_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_noalloc_ptr[kMaxDevices] = {};   // device address of the arena, per device
int g_noalloc_sms[kMaxDevices] = {};

// One-time set-up for the current device: arena address, SM count, shared-memory opt-in of the
// backward kernel.  None of these allocates.
int noalloc_setup(int dev) {
  if (g_noalloc_ptr[dev]) return FCP_OK;
  void* p = nullptr;
  FCP_CUDA_CHECK(cudaGetSymbolAddress(&p, g_noalloc_arena));
  int sms = 0, major = 0;
  FCP_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  FCP_CUDA_CHECK(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  if (major != 10) {
    fcp_set_error("device %d is not sm_100: this library is built for sm_100a only", dev);
    return FCP_ERR_CUDA;
  }
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_bwd_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<64>::DYN_BYTES));
  FCP_CUDA_CHECK(cudaFuncSetAttribute(fcp_bwd_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<128>::DYN_BYTES));
  g_noalloc_sms[dev] = sms;
  g_noalloc_ptr[dev] = (unsigned char*)p;
  return FCP_OK;
}
}  // namespace

extern "C" int fcp_noalloc_bytes_needed(const fcp_plan* plan, int64_t* bytes) {
  if (!plan || !bytes) return FCP_ERR_INVALID_ARG;
  int64_t scratch = 0;
  fcp_plan_workspace_bytes(plan, 1, nullptr, nullptr, &scratch);
  *bytes = 256 + al((int64_t)plan->bwd_units.size() * 4) + al((int64_t)plan->bwd_qranges.size() * 4) +
           al((int64_t)plan->bwd_work.size() * 4) + al(scratch);
  return FCP_OK;
}

extern "C" int fcp_attn_bwd_noalloc(const fcp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                                    const void* d_o, const float* lse, void* dq, void* dk, void* dv, void* stream) {
  if (!plan || !q || !k || !v || !o || !d_o || !lse || !dq || !dk || !dv) {
    fcp_set_error("fcp_attn_bwd_noalloc: NULL argument");
    return FCP_ERR_INVALID_ARG;
  }
  if (!plan->first_query.empty()) {
    fcp_set_error("fcp_attn_bwd_noalloc: plans with bidirectional spans are not supported here; use fcp_attn_bwd");
    return FCP_ERR_UNSUPPORTED;
  }
  int64_t need = 0;
  fcp_noalloc_bytes_needed(plan, &need);
  if (need > (int64_t)FCP_NOALLOC_MAX_BYTES) {
    fcp_set_error("fcp_attn_bwd_noalloc: this batch needs %lld bytes of scratch, the built-in arena holds %lld; "
                  "use fcp_attn_bwd with a caller-provided scratch buffer",
                  (long long)need, (long long)FCP_NOALLOC_MAX_BYTES);
    return FCP_ERR_WORKSPACE;
  }
  int dev = 0;
  FCP_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) {
    fcp_set_error("fcp_attn_bwd_noalloc: device index %d not supported", dev);
    return FCP_ERR_UNSUPPORTED;
  }
  int rc = noalloc_setup(dev);
  if (rc != FCP_OK) return rc;
  unsigned char* base = g_noalloc_ptr[dev];
  cudaStream_t st = (cudaStream_t)stream;
  const fcp_params& P = plan->params;

  // carve the arena: [status, counter | units | qranges | work | scratch]
  int64_t off = 256;
  int32_t* d_status = (int32_t*)base;
  int32_t* d_units = (int32_t*)(base + off);    off += al((int64_t)plan->bwd_units.size() * 4);
  int32_t* d_qranges = (int32_t*)(base + off);  off += al((int64_t)plan->bwd_qranges.size() * 4);
  int32_t* d_work = (int32_t*)(base + off);     off += al((int64_t)plan->bwd_work.size() * 4);
  unsigned char* d_scratch = base + off;

  // the arena still holds the previous call's data: status, work counter and the dQ accumulator
  // must start at zero (run_bwd clears the last two); the tables are rewritten from the plan's host copy
  FCP_CUDA_CHECK(cudaMemsetAsync(d_status, 0, 256, st));
  if (!plan->bwd_units.empty())
    FCP_CUDA_CHECK(cudaMemcpyAsync(d_units, plan->bwd_units.data(), plan->bwd_units.size() * 4, cudaMemcpyHostToDevice, st));
  if (!plan->bwd_qranges.empty())
    FCP_CUDA_CHECK(cudaMemcpyAsync(d_qranges, plan->bwd_qranges.data(), plan->bwd_qranges.size() * 4, cudaMemcpyHostToDevice, st));
  if (!plan->bwd_work.empty())
    FCP_CUDA_CHECK(cudaMemcpyAsync(d_work, plan->bwd_work.data(), plan->bwd_work.size() * 4, cudaMemcpyHostToDevice, st));

  const BwdTables tb{d_units, d_qranges, d_work, nullptr, d_status, d_status + 16, g_noalloc_sms[dev]};
  return run_bwd(plan, tb, q, k, v, o, d_o, lse, 0, P.hkv, dq, dk, dv, d_scratch, nullptr, st);
}

extern "C" int fcp_noalloc_device_status(int32_t* status) {
  if (!status) return FCP_ERR_INVALID_ARG;
  int dev = 0;
  FCP_CUDA_CHECK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices || !g_noalloc_ptr[dev]) {
    fcp_set_error("fcp_noalloc_device_status: fcp_attn_bwd_noalloc has not run on this device");
    return FCP_ERR_INVALID_ARG;
  }
  FCP_CUDA_CHECK(cudaDeviceSynchronize());
  FCP_CUDA_CHECK(cudaMemcpy(status, g_noalloc_ptr[dev], 4 * sizeof(int32_t), cudaMemcpyDeviceToHost));
  return FCP_OK;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded device-side wait
// ---------------------------------------------------------------------------------------------
// One CTA of one warp; lane 0 waits, through the same mbar_wait / wait_teardown the persistent kernels
// use, on a barrier that nobody will ever arrive at.  The wait limit is an argument (a millisecond or
// so instead of the kernels' two seconds), so the launch ends by itself after about that long.  The
// status words are a device array of their own: no plan is involved and none is marked as failed.
static __device__ int32_t g_wait_probe_status[4];

__global__ void __launch_bounds__(32) fcp_wait_probe_kernel(uint32_t limit_ns, int where) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(b, 1);
    fence_mbar_init();
  }
  __syncwarp();
  const WaitCtx ctx{&abort_flag, g_wait_probe_status, limit_ns};
  if (threadIdx.x == 0) (void)mbar_wait(b, 0, ctx, where);     // phase 0 never completes
  __syncwarp();
  wait_teardown(ctx);
}

extern "C" int fcp_selftest_bounded_wait(uint32_t limit_us, int32_t* status, void* stream) {
  if (!status || limit_us == 0 || limit_us > 100000u) {
    fcp_set_error("fcp_selftest_bounded_wait: status is NULL or the limit is outside [1, 100000] microseconds");
    return FCP_ERR_INVALID_ARG;
  }
  cudaStream_t st = (cudaStream_t)stream;
  void* dst = nullptr;
  FCP_CUDA_CHECK(cudaGetSymbolAddress(&dst, g_wait_probe_status));
  FCP_CUDA_CHECK(cudaMemsetAsync(dst, 0, 4 * sizeof(int32_t), st));
  fcp_wait_probe_kernel<<<1, 32, 0, st>>>(limit_us * 1000u, 901);
  FCP_CUDA_CHECK(cudaGetLastError());
  FCP_CUDA_CHECK(cudaMemcpyAsync(status, dst, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  FCP_CUDA_CHECK(cudaStreamSynchronize(st));
  return FCP_OK;
}
