// Private definition of the plan object shared by the host planner and the CUDA launchers.
#pragma once
#include <cstdint>
#include <vector>

#include "fcp.h"

constexpr int FCP_TILE = 128;          // rows of one Q tile / keys of one KV tile
constexpr int FCP_FWD_UNIT_ROWS = 256; // a forward work unit = two adjacent Q tiles of one item
constexpr int FCP_FWD_UNIT_W = 16;
constexpr int FCP_BWD_UNIT_W = 8;
constexpr int FCP_BWD_QRANGE_W = 4;
constexpr int FCP_MERGE_UNIT_W = 4;
constexpr int FCP_MERGE_TOKENS = 16;   // tokens per merge work unit

// Field indices of a forward unit row.
enum {
  FU_Q_ROW0 = 0, FU_Q_ROWS, FU_PART_ROW0, FU_N_RANGES,
  FU_KV0_BEGIN, FU_KV0_END, FU_KV0_DIAG, FU_KV1_BEGIN, FU_KV1_END, FU_KV1_DIAG,
  FU_NT_STAGE0, FU_NT_STAGE1, FU_NT_RANGE0, FU_ITEM, FU_SINGLE_SLOT, FU_RSV1
};
// Field indices of a backward unit row and of a Q range row.
enum { BU_KV_ROW0 = 0, BU_KV_ROWS, BU_FIRST_QRANGE, BU_N_QRANGES, BU_T_FIRST, BU_COST, BU_SEQ, BU_T_MASK_END };
enum { BQ_BEGIN = 0, BQ_END, BQ_DIAG, BQ_RSV };
enum { MU_TOK_BEGIN = 0, MU_N_TOK, MU_CHUNK, MU_CHUNK_TOK_BEGIN };

struct fcp_plan {
  fcp_params params{};
  int32_t B = 0;
  int64_t T = 0;   // total tokens
  int32_t max_seqlen = 0;
  int64_t R = 0;   // rows of the partial buffers
  int32_t n_merge_multi = 0;   // merge units of chunks with two or more slots (they come first in merge_units)
  std::vector<int32_t> cu_seqlens, chunk_offset, chunk_bounds, pairs, items, slot_offset, slot_rows;
  std::vector<int32_t> fwd_units, bwd_units, bwd_qranges, merge_units, bwd_work, fused_units;
  std::vector<int32_t> row_limit, first_query, span_pairs;   // empty unless the plan has bidirectional spans
  std::vector<int32_t> span_offset, spans;                   // the caller's span list ([B+1], [n][2]); empty if none

  // device copy (fcp_plan_upload)
  int device = -1;
  void* d_blob = nullptr;      // one allocation holding every table below
  int32_t* d_fwd_units = nullptr;
  int32_t* d_bwd_units = nullptr;
  int32_t* d_bwd_qranges = nullptr;
  int32_t* d_merge_units = nullptr;
  int32_t* d_bwd_work = nullptr;
  int32_t* d_fused_units = nullptr;
  int32_t* d_row_limit = nullptr;      // nullptr for a causal plan
  int32_t* d_first_query = nullptr;
  int32_t* d_slot_offset = nullptr;
  int32_t* d_slot_rows = nullptr;
  int32_t* d_status = nullptr; // [4]: status word, diagnostic
  int sm_count = 0;

  // Sub-plans over runs of consecutive sequences, built and uploaded at the first call of the host
  // entry point, which pipelines copies and kernels over them (owned by this plan).
  mutable std::vector<fcp_plan*> groups;
  mutable std::vector<int64_t> group_tok0;   // first packed token of each group, plus T at the end
  mutable void* host_in = nullptr;           // cudaStream_t: host -> device copies of the host entry point
  mutable void* host_out = nullptr;          // cudaStream_t: device -> host copies
  mutable std::vector<int32_t> group_passes; // KV-head passes of each group (large groups are also pipelined by KV head)
  mutable std::vector<void*> host_events;    // cudaEvent_t: start, last copy out, then four per (group, pass)

  // optional kernel timing: ring of event pairs per kernel kind (void* = cudaEvent_t)
  bool profiling = false;
  void* prof_ev[FCP_KERNEL_KINDS][64][2] = {};
  mutable int64_t prof_n[FCP_KERNEL_KINDS] = {};
};

void fcp_set_error(const char* fmt, ...);
