// Internal: launcher declarations shared by api.cu and the kernel translation units.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <string>

#include "plan.h"

namespace asv {

struct AttnArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k_pool;
  const __nv_bfloat16* v_pool;
  const int32_t* block_table;
  __nv_bfloat16* out;
  float* lse;               // may be null
  const float* sinks;       // may be null
  int32_t window;           // 0 = full
  float scale_log2;         // sm_scale * log2(e)
  float* part_o;            // [part_rows, D]   unnormalised partial outputs
  float2* part_ml;          // [part_rows]      (running max in log2 units, running sum)
  const WorkItem* items;
  const int32_t* cta_first; // [num_ctas + 1]
  const MergeSeg* merges;
  int32_t num_ctas, num_merges;   // host side: grid sizes
  const int32_t* num_merges_dev;  // the step's merge count, in the workspace
  int32_t rows_step = 0;       // host side: most query rows any (request, kv-head) has in this step; picks the tile width
  // test hooks of the tensor-core kernels (as_plan_set_test_stall): a shorter limit for the bounded waits, and a number of
  // tile copies after which a CTA's producers stop issuing, so that the waits behind them run out
  unsigned long long wait_limit_ns = 0;
  int32_t stall_after_loads = -1;
};

struct AcceptArgs {
  const float* logits;
  int64_t ld;
  int32_t vocab;
  const int32_t* draft_tokens;
  const float* draft_probs;   // may be null
  const float* temperature;   // may be null
  const float* u;
  const float* w;
  const uint64_t* rng;        // device {seed, step}: when set, u and w are drawn in the kernels instead (Philox4x32-10)
  // acceptance from hidden states: no [total_q, ld] logits exist.  zd [total_q] holds the logit of each row's draft
  // token, rec_logits [batch, rec_ld] the logits of the one row per request that recovery samples (row a_i)
  const float* zd = nullptr;
  const float* rec_logits = nullptr;
  int64_t rec_ld = 0;
  int32_t* accept_len;
  int32_t* out_tokens;
  // scratch in the workspace
  float4* row_part;           // [total_q, chunks] (max, argmax bits, scaled max, sum-exp)
  float4* row_final;          // [total_q] the same, folded over the chunks
  int32_t* row_ticket;        // [total_q] chunks finished so far; zero between calls
  int32_t chunks, chunk_elems;
  int32_t* recover_row;       // [batch] row whose recovery distribution must be sampled, or -1
  double* rec_cells;          // [batch, cells, 2] mass of p and of max(0, p - q) per cell of cell_elems entries
  int32_t cells, cell_elems;  // cell_elems divides chunk_elems
};

cudaError_t launch_assign_pages(const DevPlan& P, int32_t* block_table, const int32_t* free_ids,
                                const int32_t* free_first, cudaStream_t s);
cudaError_t launch_append(const DevPlan& P, const __nv_bfloat16* k_new, const __nv_bfloat16* v_new,
                          __nv_bfloat16* k_pool, __nv_bfloat16* v_pool, const int32_t* block_table, cudaStream_t s);
cudaError_t launch_attn_simt(const DevPlan& P, const AttnArgs& A, cudaStream_t s);
cudaError_t launch_attn_merge(const DevPlan& P, const AttnArgs& A, cudaStream_t s);
size_t attn_simt_smem_bytes(int rows, int D);
cudaError_t launch_accept(const DevPlan& P, const AcceptArgs& A, cudaStream_t s);
cudaError_t launch_commit(const DevPlan& P, const int32_t* accept_len, int32_t* seq_lens, int32_t* block_table,
                          int32_t* freed, int32_t* freed_count, int scrub, __nv_bfloat16* k_pool,
                          __nv_bfloat16* v_pool, int32_t* counts /* [batch + 1] scratch */, cudaStream_t s);

// Stores `msg` as the calling thread's last error (what as_last_error() returns) and returns `code`.
int record_error(int code, const std::string& msg);

// status-word bits (mirrors the public AS_FLAG_* values)
constexpr uint32_t kFlagBadPage = 1, kFlagBadToken = 2, kFlagWaitCap = 4, kFlagBadAccept = 8, kFlagBadPlan = 16;

}  // namespace asv
