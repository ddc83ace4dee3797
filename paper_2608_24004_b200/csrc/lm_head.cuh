// Internal: interface of the fused output projection + row argmax kernel.
#pragma once
#include <string>

#include "kernels.cuh"

namespace asv {

struct LmHeadState {         // per-plan cache: tensor maps are rebuilt only when an operand changes
  const void* hidden = nullptr;
  const void* weight = nullptr;
  int H = 0, V = 0, rows = 0;
  alignas(64) unsigned char a_map[128];
  alignas(64) unsigned char w_map[128];
};

// row_final[r] = (largest logit of row r, its lowest column) for r < the step's rows; `keys` is scratch of
// rows_extent 64-bit words.  Returns an AS_* status; on failure `err` holds the reason.
int launch_lm_head_argmax(const DevPlan& P, LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent,
                          int num_sms, unsigned long long* keys, float4* row_final, cudaStream_t s, std::string& err);
// The same plus, for the rows of sampling requests (temperature > 0), the folded (scaled max, sum of exponentials) in
// row_final[r].z / .w and the logit of the row's draft token in zd[r]; tile_part is scratch of rows_extent x
// lm_head_vocab_tiles(V) pairs.
int launch_lm_head_stats(const DevPlan& P, LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent,
                         int num_sms, unsigned long long* keys, float2* tile_part, float* zd, const int32_t* draft_tokens,
                         const float* temperature, float4* row_final, cudaStream_t s, std::string& err);
// fp32 logits of one row per request (row recover_row[i] of request i, zeros where it is negative) into logits[i][0..V):
// the rows' hidden states are gathered into hidden_rows [batch_extent, H] first.
int launch_lm_head_recover_rows(const DevPlan& P, LmHeadState& st, const int32_t* recover_row, const void* hidden, void* hidden_rows,
                                const void* weight, int H, int V, int batch_extent, int num_sms, float* logits, long long ld,
                                cudaStream_t s, std::string& err);
int lm_head_vocab_tiles(int V);
// The acceptance decision alone, from row_final (and zd for sampling requests; no logits are read).
cudaError_t launch_decide(const DevPlan& P, const AcceptArgs& A, cudaStream_t s);
// The recovery draw of the sampling requests (denominator, cell masses, pick), from A.rec_logits.
cudaError_t launch_recover(const DevPlan& P, const AcceptArgs& A, cudaStream_t s);

}  // namespace asv
