// Internal: interface of the tcgen05 / TMA verify-attention kernel.
#pragma once
#include <string>

#include "kernels.cuh"

namespace asv {

// Per-plan cache of tensor maps, keyed by the pool pointers: a model's layers have a pool pair each and one plan
// serves them in turn, so a single entry would be encoded anew (on the host, inside the step) at every call.
struct TcState {
  static constexpr int kEntries = 16;
  struct Entry {
    const void* k_pool = nullptr;
    const void* v_pool = nullptr;
    alignas(64) unsigned char k_map[128];
    alignas(64) unsigned char v_map[128];
  };
  Entry entry[kEntries];
  int next = 0;              // round-robin replacement
};

bool attn_tc_supported(int Hq, int Hkv, int D, int bs, int max_draft, int window);
// True when a tensor-core launch of this width runs the rows-on-M kernel (whose tile cost does not depend on the row count).
bool attn_rows_on_m(int D, int rows);
// Returns an AS_* status; on failure `err` holds the reason.
int launch_attn_tc(const DevPlan& P, const AttnArgs& A, TcState& st, cudaStream_t s, std::string& err);

}  // namespace asv
