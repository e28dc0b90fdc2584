/*
 * libfcp — the single-GPU hot path of Flexible Context Parallelism (FCP) for B200 (sm_100a).
 *
 * Varlen causal attention, forward and backward, over a packed batch of sequences of very
 * different lengths.  Every sequence carries its own context-parallel (CP) degree d (any positive
 * integer, Sec. 4.2 "any positive integer parallelism degree"); it is cut evenly along the sequence
 * dimension (Sec. 4.3) into 2d load-balanced chunks, and every (Q chunk, KV chunk) block pair that
 * a virtual rank of a ring-style CP group (Sec. 3.2) would compute is executed on one GPU, giving
 * partial outputs and log-sum-exps that a merge kernel combines exactly.  The per-batch strategy
 * search of Sec. 4.4 (best-fit-decreasing grouping + 2-D dynamic programme, Eq. 7, Algorithm 1)
 * runs on the host and emits the per-sequence degrees.
 *
 * Conventions
 *   - Plain C ABI.  Every function returns an int status (FCP_OK == 0, negative = error) and never
 *     throws or aborts.  fcp_status_string() names a status.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA global memory of the
 *     current device.  The caller owns every buffer it passes; the library owns only fcp_plan
 *     objects (host tables plus, after fcp_plan_upload, a device copy of them).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Compute calls only
 *     enqueue work on it; they do not synchronise and do not allocate device memory.
 *   - Calls that use one plan must be stream-ordered with respect to each other: the plan's device
 *     copy holds the status words and the work counters of the forward and backward grids, so two compute calls
 *     on the same plan that overlap on the GPU (different streams, different threads) race.  Use
 *     one plan per concurrent stream.
 *   - The device status words are sticky: once a kernel has recorded FCP_ERR_TIMEOUT they keep it
 *     for the life of the plan's device copy (fcp_last_device_status reports the first failure).
 *   - Tensors are packed token-major ("THD"), row-major, bf16:
 *         q, o, d_o, dq : [T][hq][D]        k, v, dk, dv : [T][hkv][D]
 *     T = total tokens of the batch, D = head_dim in {64, 128}, hq % hkv == 0; query head h reads
 *     KV head h / (hq/hkv).  lse is fp32 [T][hq], natural log of the sum of exp(scaled scores).
 *   - Limits: T and the number of partial rows R are < 2^31; device byte offsets are 64-bit.
 */
#ifndef FCP_H_
#define FCP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FCP_OK                 0
#define FCP_ERR_INVALID_ARG   (-1)   /* NULL pointer, non-positive size, bad enum                    */
#define FCP_ERR_INFEASIBLE    (-2)   /* planner: the minimum degrees need more than N ranks          */
#define FCP_ERR_UNSUPPORTED   (-3)   /* head_dim not 64/128, hq % hkv != 0, degree > FCP_MAX_DEGREE   */
#define FCP_ERR_WORKSPACE     (-4)   /* a caller-provided workspace is too small                      */
#define FCP_ERR_CUDA          (-5)   /* a CUDA runtime/driver call failed, or no usable device        */
#define FCP_ERR_TIMEOUT       (-6)   /* a bounded device-side wait expired (reported by fcp_last_device_status) */
#define FCP_ERR_NOT_UPLOADED  (-7)   /* compute call on a plan without a device copy                  */

#define FCP_MAX_DEGREE 64            /* largest CP degree of one sequence                             */

typedef struct fcp_plan fcp_plan;

/* Shape of the attention problem.  scale <= 0 selects 1/sqrt(head_dim) (Sec. 3.1, Eq. 1). */
typedef struct fcp_params {
  int32_t hq;        /* query heads                                  */
  int32_t hkv;       /* key/value heads (hq % hkv == 0)               */
  int32_t head_dim;  /* 64 or 128                                     */
  float   scale;     /* softmax scale; <= 0 means 1/sqrt(head_dim)    */
} fcp_params;

/* Profiled coefficients of the cost model, Eqs. 4-6 (Sec. 4.3).  eta is the per-sequence mask
 * efficiency factor (host array of B doubles) or NULL for all-causal (eta = 0). */
typedef struct fcp_cost_coeffs {
  double alpha1, alpha2, alpha3, beta1, beta2, v;
  const double* eta;
} fcp_cost_coeffs;

/* ------------------------------------------------------------------------------------------
 * fcp_plan_strategy — host only.  Sec. 4.4: stage 1 groups the B sequences into K' atomic groups
 * by best-fit-decreasing under the per-rank activation budget E - M_ms (Eq. 3; a sequence that
 * opens a group fixes d_min = ceil(len*M_token / (E - M_ms))); stage 2 is the 2-D dynamic programme
 * DP[i][j] = min_d max(DP[i-1][j-d], T(G_i, d)) of Eq. 7 / Algorithm 1 with strict-less updates,
 * backtracked from DP[K'][N], so the degrees add up to exactly N.  T(G, d) is Eq. 6 with the
 * per-rank reading of Eqs. 4-5: compute terms divided by d, ring communication only when d > 1.
 *   in : seqlens[B] (host), N ranks, E, M_token, M_ms, coefficients
 *   out: group_of[B] (group index of each sequence, groups in creation order), cp_degree[B]
 *        (degree of the sequence's group), *n_groups, *makespan = DP[K'][N]; any may be NULL.
 * Errors: FCP_ERR_INVALID_ARG (NULL inputs, B <= 0, N <= 0, E <= M_ms, non-positive length or
 * M_token), FCP_ERR_INFEASIBLE (sum of d_min > N), FCP_ERR_UNSUPPORTED (N > FCP_MAX_DEGREE).
 */
int fcp_plan_strategy(const int32_t* seqlens, int32_t B, int32_t N, double E, double M_token,
                      double M_ms, const fcp_cost_coeffs* coeffs, int32_t* group_of,
                      int32_t* cp_degree, int32_t* n_groups, double* makespan);

/* ------------------------------------------------------------------------------------------
 * fcp_plan_blocks — host only.  Builds the block plan of a packed batch: for each sequence of
 * length L and degree d the 2d+1 chunk bounds floor(c*L/(2d)) ("evenly into chunks", Sec. 4.3),
 * and for each virtual rank r (owning chunks r and 2d-1-r) and ring step s (holding the KV of
 * rank (r-s) mod d) the causally needed block pairs; pairs with an empty chunk are dropped.  One
 * partial-output slot per (Q chunk, rank, step).  Also derives the kernels' work lists.
 *   in : seqlens[B], cp_degrees[B] (host), params
 *   out: *plan (release with fcp_plan_destroy)
 * Errors: INVALID_ARG (NULL, B <= 0, length <= 0, degree <= 0, T or R >= 2^31),
 * UNSUPPORTED (head_dim, head ratio, degree > FCP_MAX_DEGREE).
 */
int fcp_plan_blocks(const int32_t* seqlens, const int32_t* cp_degrees, int32_t B,
                    const fcp_params* params, fcp_plan** plan);

/* ------------------------------------------------------------------------------------------
 * fcp_plan_blocks_spans — host only.  fcp_plan_blocks for sequences that carry bidirectional spans:
 * multimodal batches let the tokens of an image or a video frame attend to each other in both
 * directions while text stays causal, which is what the mask efficiency factor eta_k > 0 of the
 * cost model stands for (Sec. 4.3, Eq. 4).  Sequence b has the spans span_offset[b] ..
 * span_offset[b+1]-1 of `spans`, each a pair (begin, end) of positions relative to the sequence
 * start, sorted, disjoint, 0 <= begin < end <= length.  Query i sees key j iff j <= i, or both lie
 * in the same span; so query t sees exactly the keys before FCP_TABLE_ROW_LIMIT[t] and key t is
 * seen from query FCP_TABLE_FIRST_QUERY[t] on.  The causal tables (pairs, items, slots) are those
 * of fcp_plan_blocks; FCP_TABLE_SPAN_PAIRS lists the block pairs above the chunk diagonal that the
 * spans add (computed by the rank that owns the Q chunk when the KV chunk's owner visits).
 * fcp_attn_fwd_fused and fcp_attn_bwd apply the mask; the per-item partial path (fcp_attn_fwd,
 * fcp_attn_fwd_merged, fcp_lse_merge) and fcp_attn_bwd_noalloc are causal only and return
 * FCP_ERR_UNSUPPORTED for such a plan.  span_offset == NULL means no spans.
 * fcp_span_mask_efficiency gives the eta_k of one sequence for fcp_plan_strategy: visible
 * (query, key) pairs over the causal count L(L+1)/2, minus 1.
 */
int fcp_plan_blocks_spans(const int32_t* seqlens, const int32_t* cp_degrees, int32_t B,
                          const int32_t* span_offset, const int32_t* spans,
                          const fcp_params* params, fcp_plan** plan);
int fcp_span_mask_efficiency(int32_t length, const int32_t* spans, int32_t n_spans, double* eta);

/* Tables readable through fcp_plan_get.  All are int32, row-major, host memory owned by the plan.
 * Rows are in the canonical order (sequence, rank, step, q_chunk, kv_chunk).                     */
#define FCP_TABLE_CU_SEQLENS    0  /* [B+1]                     packed-token offsets of the sequences */
#define FCP_TABLE_CHUNK_OFFSET  1  /* [B+1]                     offsets into CHUNK_BOUNDS             */
#define FCP_TABLE_CHUNK_BOUNDS  2  /* [sum(2d+1)]               packed-token chunk bounds             */
#define FCP_TABLE_PAIRS         3  /* [n_pairs][6]  seq, rank, step, q_chunk, kv_chunk, kind (0 FULL, 1 DIAG) */
#define FCP_TABLE_ITEMS         4  /* [n_items][8]  seq, rank, step, q_chunk, slot, part_row0, n_pairs, first_pair */
#define FCP_TABLE_SLOT_OFFSET   5  /* [n_chunks+1]              offsets into SLOT_ROWS, chunks in (seq, chunk) order */
#define FCP_TABLE_SLOT_ROWS     6  /* [sum n_slots]             part_row0 of each slot of each chunk  */
#define FCP_TABLE_FWD_UNITS     7  /* [n_fwd_units][16]         derived; execution order, not canonical */
#define FCP_TABLE_BWD_UNITS     8  /* [n_bwd_units][8]          derived                               */
#define FCP_TABLE_BWD_QRANGES   9  /* [n_bwd_qranges][4]        derived                               */
#define FCP_TABLE_MERGE_UNITS  10  /* [n_merge_units][4]        derived                               */
#define FCP_TABLE_BWD_WORK     11  /* [n_bwd_units]             derived: backward units in execution order (per KV head) */
#define FCP_TABLE_FUSED_UNITS  12  /* [n_fused_units][16]       derived: work units of fcp_attn_fwd_fused       */
#define FCP_TABLE_ROW_LIMIT    13  /* [T] or empty              first key (packed index) query t does not see   */
#define FCP_TABLE_FIRST_QUERY  14  /* [T] or empty              first query (packed index) that sees key t      */
#define FCP_TABLE_SPAN_PAIRS   15  /* [n][5]  seq, rank, step, q_chunk, kv_chunk (> q_chunk): pairs a span adds  */

/* fcp_plan_get: *host_ptr = first element of the table, *count = number of int32 elements. */
int fcp_plan_get(const fcp_plan* plan, int32_t which, const int32_t** host_ptr, int64_t* count);

/* Scalar facts about a plan: which in {0: T, 1: R (partial rows), 2: n_pairs, 3: n_items,
 * 4: n_fwd_units, 5: n_bwd_units, 6: n_merge_units, 7: B, 8: the leading merge units that belong
 * to Q chunks with two or more slots (all that fcp_attn_fwd_merged has to merge), 9: n_fused_units}. */
int fcp_plan_info(const fcp_plan* plan, int32_t which, int64_t* value);

/* Bytes the caller must provide: o_partial = R*heads_per_pass*D*4, lse_partial = R*heads_per_pass*4,
 * bwd_scratch (all hq heads at once) for fcp_attn_bwd.  Any output pointer may be NULL.          */
int fcp_plan_workspace_bytes(const fcp_plan* plan, int32_t heads_per_pass, int64_t* o_partial_bytes,
                             int64_t* lse_partial_bytes, int64_t* bwd_scratch_bytes);
/* Scratch bytes of fcp_attn_bwd_heads for a pass over kv_head_count KV heads (and their query
 * heads): about 4*T*(kv_head_count*hq/hkv)*D bytes.                                               */
int fcp_plan_bwd_scratch_bytes(const fcp_plan* plan, int32_t kv_head_count, int64_t* bytes);

/* Copies the plan's work tables to the current device (the only device allocation the library
 * makes; freed by fcp_plan_destroy).  Must precede the compute calls.  Synchronous.              */
int fcp_plan_upload(fcp_plan* plan, void* stream);
int fcp_plan_destroy(fcp_plan* plan);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_fwd — device.  For every item of the plan and every query head h in
 * [head_begin, head_begin+head_count): softmax(q k^T * scale) v (Eq. 1) restricted to the item's
 * KV ranges with the causal mask k_pos <= q_pos, as a NORMALISED partial output and its
 * log-sum-exp:
 *     o_partial  [R][head_count][D] fp32,   lse_partial [R][head_count] fp32
 * Row r of an item = part_row0 + (token - first token of its Q chunk).
 * q, k, v: device bf16.  Asynchronous on `stream`.
 */
int fcp_attn_fwd(const fcp_plan* plan, const void* q, const void* k, const void* v,
                 int32_t head_begin, int32_t head_count, float* o_partial, float* lse_partial,
                 void* stream);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_fwd_merged — device.  fcp_attn_fwd followed by fcp_lse_merge in one call, for callers
 * that do not need the partials of every item: Q chunks that have a single slot (every chunk of a
 * sequence at degree 1, and the first chunk of any sequence) have nothing to merge, so their
 * normalised partial is rounded to bf16 and written straight to o / lse, and only the chunks
 * with two or more slots go through o_partial / lse_partial (same sizes as for fcp_attn_fwd) and
 * the merge (Sec. 3.2: the merge re-associates the softmax sum; with one term it is the identity).
 * o [T][hq][D] bf16 and lse [T][hq] fp32 are bit-identical to fcp_attn_fwd + fcp_lse_merge.
 * After the call the partial rows of single-slot chunks are unspecified.  Asynchronous on `stream`.
 */
int fcp_attn_fwd_merged(const fcp_plan* plan, const void* q, const void* k, const void* v,
                        int32_t head_begin, int32_t head_count, float* o_partial, float* lse_partial,
                        void* o, float* lse, void* stream);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_fwd_fused — device.  The forward pass with the merge done on the fly: all items of a Q
 * chunk are scheduled onto one CTA, which sweeps the KV ranges of every block pair of the chunk
 * (the same pairs fcp_attn_fwd executes, FCP_TABLE_FUSED_UNITS lists them per work unit) in a
 * single online softmax and writes o [T][hq][D] bf16 and lse [T][hq] fp32 directly (Eq. 1; the
 * merge of Sec. 3.2's ring steps is the re-association the online softmax performs anyway).  No
 * partial buffer is needed.  Adjacent Q chunks of a causal plan are tiled as one run of rows, so
 * no tile is cut at a chunk edge and the running time does not depend on the degrees.  Results
 * agree with fcp_attn_fwd + fcp_lse_merge to rounding (the summation order differs).
 * o_f32 is optional (NULL to skip): the same output [T][hq][D] before the rounding to bf16.
 * Heads [head_begin, head_begin+head_count).  Asynchronous on `stream`.
 */
int fcp_attn_fwd_fused(const fcp_plan* plan, const void* q, const void* k, const void* v,
                       int32_t head_begin, int32_t head_count, void* o, float* o_f32, float* lse,
                       void* stream);

/* ------------------------------------------------------------------------------------------
 * fcp_lse_merge — device.  Exact combination of the slots of every (token, head):
 *     LSE = m + log sum_s exp(lse_s - m),  o = sum_s exp(lse_s - LSE) * o_s     (m = max_s lse_s)
 * (the re-association of the softmax sum implied by ring-style CP, Sec. 3.2).
 * Writes o[T][hq][D] bf16 and lse[T][hq] fp32 for heads [head_begin, head_begin+head_count); the
 * partial buffers have head_count heads (the layout fcp_attn_fwd wrote).  o_f32 is optional
 * (NULL to skip): the same output [T][hq][D] before the rounding to bf16, for callers that keep an
 * fp32 activation stream.
 */
int fcp_lse_merge(const fcp_plan* plan, const float* o_partial, const float* lse_partial,
                  int32_t head_begin, int32_t head_count, void* o, float* o_f32, float* lse,
                  void* stream);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_bwd — device.  Gradients of Eq. 1 with the causal mask, evaluated over the plan's
 * block pairs grouped by KV chunk: with P = exp(S*scale - LSE), delta_i = dO_i . O_i,
 *     dV = P^T dO,  dP = dO V^T,  dS = P o (dP - delta),  dQ = scale dS K,  dK = scale dS^T Q,
 * dK/dV summed over the hq/hkv query heads of a KV head.  o, lse are the merged forward results.
 * scratch: device buffer of at least bwd_scratch_bytes (fcp_plan_workspace_bytes); its contents
 * need not be initialised.  dq/dk/dv: device bf16 outputs (every element is written).
 */
int fcp_attn_bwd(const fcp_plan* plan, const void* q, const void* k, const void* v, const void* o,
                 const void* d_o, const float* lse, void* dq, void* dk, void* dv, void* scratch,
                 int64_t scratch_bytes, void* stream);

/* fcp_attn_bwd_heads — device.  fcp_attn_bwd restricted to the KV heads [kv_head_begin,
 * kv_head_begin + kv_head_count) and the hq/hkv query heads of each: writes dk, dv of those KV
 * heads and dq of those query heads, leaves the other heads of the outputs untouched.  KV heads are
 * independent problems (no sum crosses them), so passes over disjoint ranges give the result of
 * one call over all heads; this bounds the scratch (fcp_plan_bwd_scratch_bytes) and is the unit by
 * which the backward pass can be split over GPUs.  All tensors keep their full [T][heads][D] shape.
 */
int fcp_attn_bwd_heads(const fcp_plan* plan, const void* q, const void* k, const void* v,
                       const void* o, const void* d_o, const float* lse, int32_t kv_head_begin,
                       int32_t kv_head_count, void* dq, void* dk, void* dv, void* scratch,
                       int64_t scratch_bytes, void* stream);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_fwd_bwd_host — the whole path from HOST buffers: copies q, k, v, d_o to the device,
 * runs fcp_attn_fwd_fused and fcp_attn_bwd, and copies o, lse, dq, dk, dv back.  `workspace` is a
 * caller-owned DEVICE buffer of `workspace_bytes` >= fcp_host_workspace_bytes(plan); host pointers
 * should be pinned for the copies to be asynchronous.
 * The batch is cut into up to 8 runs of consecutive sequences (packed tensors are token-major, so a
 * run is one contiguous slice of every tensor), and a run of several hundred megabytes further into
 * passes over whole KV heads (strided slices); the inputs of the next slice come in and the results
 * of the previous one go out while the kernels of the current slice execute (two internal copy
 * streams, ordered after the work already queued on `stream`).  The first call on a plan is the
 * one exception to "compute calls do not allocate": it builds and uploads the plans of the runs
 * and creates the copy streams and events (small allocations, all released by fcp_plan_destroy).
 * Synchronises `stream` before returning; every output is complete then.  On an error return the
 * work already queued has been waited for, so nothing writes into the caller's buffers afterwards.
 */
int fcp_host_workspace_bytes(const fcp_plan* plan, int64_t* bytes);
int fcp_attn_fwd_bwd_host(const fcp_plan* plan, const void* q_host, const void* k_host,
                          const void* v_host, const void* d_o_host, void* o_host, float* lse_host,
                          void* dq_host, void* dk_host, void* dv_host, void* workspace,
                          int64_t workspace_bytes, void* stream);

/* Device-side status words of the kernels run with this plan so far: status[0] = 0 while all is
 * fine, FCP_ERR_TIMEOUT once a bounded wait inside a kernel has expired (sticky, first failure
 * wins); status[1] = code of the wait that gave up, status[2] = its CTA.  Synchronises the device. */
int fcp_last_device_status(const fcp_plan* plan, int32_t* status);

/* ------------------------------------------------------------------------------------------
 * fcp_attn_bwd_noalloc — device.  (The paper has no counterpart: this entry point exists for the
 * way the library gets embedded, not for the method.)
 *
 * Same gradients as fcp_attn_bwd, for callers that are not allowed to allocate device memory when
 * they reach the backward pass: code running under a framework whose memory pool must own every
 * allocation, inside a region where cudaMalloc would synchronise the device or is forbidden
 * outright, or on a device whose memory has already been handed out in full.  Such a caller cannot
 * size and allocate the scratch buffer fcp_attn_bwd wants, and cannot call fcp_plan_upload either.
 * Here the plan stays a host object (no fcp_plan_upload needed), and the work tables, status
 * words and backward scratch all go into one fixed array of FCP_NOALLOC_MAX_BYTES that is part of
 * the library image on every GPU that loads it.  The call itself performs only asynchronous
 * copies, memsets and kernel launches on `stream`.
 *
 *   in : plan (from fcp_plan_blocks), q, k, v, o, d_o (bf16), lse (fp32): device, as for fcp_attn_bwd
 *   out: dq, dk, dv (device bf16, every element written)
 * Limits and rules
 *   - fcp_noalloc_bytes_needed(plan) must not exceed FCP_NOALLOC_MAX_BYTES (roughly
 *     4*T*hq*D bytes plus the tables); larger batches get FCP_ERR_WORKSPACE and must use
 *     fcp_attn_bwd with their own scratch.
 *   - The first call on each device looks up the array's device address and opts the kernel in to
 *     its shared-memory size; make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents (the
 *     function clears what has to start from zero).  Two calls that can overlap on the GPU, on
 *     different streams or from different threads, corrupt each other: serialise them.
 *   - The plan's host tables are read by the asynchronous copies at the moment those copies execute,
 *     not when this function returns: keep the plan alive and unchanged for as long as any copy
 *     issued by this call can still run.
 * fcp_noalloc_device_status reads the status words of the last such call on the current device
 * (synchronises the device; 0 = fine, FCP_ERR_TIMEOUT if a bounded wait in the kernel expired).
 */
#define FCP_NOALLOC_MAX_BYTES (32u << 20)
int fcp_noalloc_bytes_needed(const fcp_plan* plan, int64_t* bytes);
int fcp_attn_bwd_noalloc(const fcp_plan* plan, const void* q, const void* k, const void* v,
                         const void* o, const void* d_o, const float* lse, void* dq, void* dk,
                         void* dv, void* stream);
int fcp_noalloc_device_status(int32_t* status);

/* Kernel timing for benchmarks.  fcp_plan_set_profiling(plan, 1) makes every compute call record a
 * CUDA event pair around each of its kernels on the launching stream (a ring of the last 64 launches
 * per kind); fcp_plan_kernel_ms returns, after the caller has synchronised, the number of recorded
 * launches of `kind` and their mean duration in milliseconds.  kind: 0 forward attention,
 * 1 LSE merge, 2 backward preprocess (accumulator clear + delta), 3 backward attention,
 * 4 dQ conversion.  fcp_plan_set_profiling(plan, 0) stops recording and clears the ring.        */
#define FCP_KERNEL_KINDS 5
int fcp_plan_set_profiling(fcp_plan* plan, int32_t enable);
int fcp_plan_kernel_ms(const fcp_plan* plan, int32_t kind, int32_t* launches, float* mean_ms);

/* fcp_selftest_bounded_wait — device.  Every wait inside the persistent kernels (on an mbarrier fed
 * by TMA, the tensor core or another warp) is bounded: after 2 s without progress the waiter gives
 * up, the CTA unwinds, and FCP_ERR_TIMEOUT appears in the status words instead of a hung GPU.  This
 * call exercises exactly that code on purpose and safely: one warp waits on a barrier nobody
 * arrives at, with the limit set to `limit_us` microseconds (1..100000), so the launch ends by
 * itself after about that long.  Writes the four status words the wait produced to the host array
 * status[4]: {FCP_ERR_TIMEOUT, 901 (the code of the wait site), CTA index 0, 0}.  Uses status words
 * of its own (no plan is involved or marked).  Synchronises `stream`.                             */
int fcp_selftest_bounded_wait(uint32_t limit_us, int32_t* status, void* stream);

const char* fcp_status_string(int status);
const char* fcp_last_error_message(void);

#ifdef __cplusplus
}
#endif
#endif /* FCP_H_ */
