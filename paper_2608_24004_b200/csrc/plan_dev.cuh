// Internal: interface of the device-side planner.
#pragma once
#include "kernels.cuh"

namespace asv {

struct PlanDevKind {                  // one layer flavour: where its work list goes and which kernel will read it
  WorkItem* items;
  int32_t* cta_first;                 // [num_ctas + 1]
  MergeSeg* merges;
  int32_t window;
  int32_t num_ctas;
  int32_t rows_inst;                  // row count the launch is configured for (the plan's maximum)
  int32_t row_blocks;                 // most row blocks any request can have (plan_block_positions)
  bool tensor_core, rows_on_m;
};

struct PlanDevArgs {
  const int32_t* seq_lens;            // device
  const int32_t* draft_lens;          // device
  int32_t batch;
  StepHeader* hdr;
  ReqMeta* req;
  int2* row_map;
  int32_t* free_first;                // [batch + 1]
  uint32_t* status;
  int32_t num_kinds;
  PlanDevKind kind[kMaxKinds];
  int32_t G, Hkv, bs, max_blocks, max_draft, max_total_q;
  int64_t max_items, max_merges, max_part_rows;
  int32_t assign, num_free;           // pages are taken from a free list of num_free entries
};

cudaError_t launch_plan_device(const PlanDevArgs& a, int max_batch, cudaStream_t s);

}  // namespace asv
