// Internal: device-visible metadata that as_plan() writes into the workspace and the kernels read.
#pragma once
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

namespace asv {

constexpr int kTileKeys = 128;        // split-KV cut granularity (keys); a multiple of every page size
constexpr int kMaxKinds = 4;
constexpr int kMaxSub = 2;           // attention launches per layer kind and step (requests bucketed by row count)
constexpr int kMaxRows = 256;         // G * (max_draft + 1)

struct ReqMeta {                      // one per request
  int32_t n;                          // committed context length
  int32_t k;                          // draft length
  int32_t cu_q;                       // first row of the request
  int32_t cu_d;                       // first draft of the request
};

struct WorkItem {                     // one contiguous key range of one (request, kv-head) pair
  int32_t req;
  int32_t kv_head;
  int32_t key_begin;                  // absolute positions, key_begin a multiple of kTileKeys
  int32_t key_end;                    // exclusive; <= n + k + 1
  int32_t part_row;                   // -1: this item covers the whole pair and writes the output;
                                      // else first row of its (m, l, O) partial in the partial buffers
  int32_t n, k, cu_q;                 // copy of the request's entry, so a kernel needs one 32-byte load per item
};

struct MergeSeg {                     // a pair that was cut into num_parts items
  int32_t req;
  int32_t kv_head;
  int32_t part_row;                   // partial p of the pair starts at part_row + p * G * (k + 1)
  int32_t num_parts;
  int32_t k, cu_q;                    // the pair's draft length and first row (a row block's own, see plan_block_positions)
};

struct KindLayout {                   // byte offsets into the workspace
  size_t items, cta_first, merges;
};

struct StepHeader {                   // the sizes of the current step, in the workspace: kernels read them from here,
  int32_t batch, total_q, total_d;    // so that their launch parameters need not change from step to step
  int32_t num_merges[kMaxKinds * kMaxSub];   // per layer kind and sub-launch
  int32_t pad;
};

// ---- the split-KV cost model and the cut of one (request, kv-head) pair: one definition for the host planner
// (as_plan) and the device planner (as_plan_device), so that both produce the same work list.

// Fixed cost of an item (staging Q, first-tile set-up, draining the pipeline, epilogue) in eighths of a plain tile:
// 3 plain tiles, from a fit of measured per-CTA durations against (items, tiles) on three workloads (4.0-4.2 us
// per item, 1.38 us per tile).
constexpr int64_t kItemOverhead = 24;
// The rows-on-M kernel pays more per item (a synchronous Q staging, a two-pass first tile for either stream, the merge
// of the two streams in the epilogue) and pays it once per block of 128 rows: per-CTA durations on the GPT-OSS-shaped
// layers and on 1-3 k contexts fit 5.0-7.5 us per (item, row block) and 0.88-0.95 us per tile, i.e. 5-8 tiles.
constexpr int64_t kItemOverheadRows = 64;

// Fixed cost of one piece of a pair with `rows` query rows, in the units of plan_tile_cost.
__host__ __device__ inline int64_t plan_item_overhead(bool tensor_core, bool rows_on_m, int rows) {
  return tensor_core && rows_on_m ? kItemOverheadRows * ((rows + 127) / 128) : kItemOverhead;
}

// Cost of one 128-key tile of a request with `rows` query rows per KV head, in eighths of a plain tile, for the
// kernel that will run the launch (`rows_inst` = the launch's widest request).
__host__ __device__ inline int64_t plan_tile_cost(bool tensor_core, bool rows_on_m, int rows_inst, int rows) {
  if (!tensor_core) return rows / 2 > 1 ? rows / 2 : 1;              // SIMT: work grows with the row count
  if (rows_on_m) return 10 * ((rows + 127) / 128);                    // rows on M: per block of 128 rows
  const int slabs_inst = (rows_inst + 15) / 16;
  const int groups = slabs_inst < 7 ? slabs_inst : 7;                 // softmax warpgroups of the instance
  const int per_group = ((rows + 15) / 16 + groups - 1) / groups;     // 16-row slabs a warpgroup walks per tile
  return 8 + 4 * (per_group - 1);
}

// Row blocks.  The keys-on-M kernel (head_dim 128) is instantiated for up to 112 query rows per (request, kv-head)
// pair and is at its best up to 96; a request with more rows is planned as several pairs by rows, of equal size and at
// most 96 rows where the group size allows: block v covers draft positions [v * pb, (v + 1) * pb), and is to the
// kernels a request of its own with n' = n + v * pb committed entries (the earlier positions of the same step are in
// the pages by then: the append precedes the attention), k' = min(k - v * pb, pb - 1) drafts and first row
// cu_q' = cu_q + v * pb.  Returns pb for a request with k drafts: k + 1 (a single block) when the launch's kernel takes
// all rows of a pair at once (SIMT, rows on M) or the request has no more than 112.
constexpr int kKeysOnMRows = 112;     // widest keys-on-M instance
__host__ __device__ inline int plan_block_positions(bool tensor_core, bool rows_on_m, int G, int k) {
  const int R = G * (k + 1);
  if (!tensor_core || rows_on_m || R <= kKeysOnMRows) return k + 1;
  const int V = (R + 95) / 96;
  int pb = (k + V) / V;                                  // ceil((k + 1) / V)
  while (pb > 1 && pb * G > kKeysOnMRows) --pb;          // (one position's G rows always fit: G <= 112 is required)
  return pb;
}

// CTA that owns cost unit x when C units are dealt evenly to P CTAs.
__host__ __device__ inline int plan_owner(int64_t x, int64_t C, int P) {
  const int64_t o = x * P / C;
  return (int)(o < P - 1 ? o : P - 1);
}

// One pair's t_count tiles, whose tile t starts at cost unit base + t * cpt, are cut at the CTA boundaries.  Given
// the first tile t of a piece, returns its end t_end (exclusive) and the CTA `owner` that runs it; the caller
// walks t = 0, t_end, ... up to t_count.
__host__ __device__ inline void plan_next_piece(int64_t base, int t, int t_count, int64_t cpt, int64_t C, int P, int& t_end,
                                                int& owner) {
  owner = plan_owner(base + t * cpt, C, P);
  t_end = t_count;
  if (owner < P - 1) {
    const int64_t next_x = ((int64_t)(owner + 1) * C + P - 1) / P;   // first cost unit of CTA owner + 1
    const int64_t lim = (next_x - base + cpt - 1) / cpt;
    t_end = (int)(lim < t_count ? lim : t_count);
    // (owner < P - 1 here, so "cost unit x belongs to a CTA <= owner" is x * P < (owner + 1) * C: no division)
    const int64_t bound = (int64_t)(owner + 1) * C;
    while (t_end < t_count && (base + t_end * cpt) * P < bound) ++t_end;
    while (t_end > t + 1 && (base + (t_end - 1) * cpt) * P >= bound) --t_end;
    if (t_end <= t) t_end = t + 1;
  }
}

struct DevPlan {                      // passed by value to kernels
  const StepHeader* hdr;              // device copy of the step's sizes: what kernels use
  const ReqMeta* req;
  const int2* row_map;                // [total_q] (request, j)
  uint32_t* status;
  int32_t batch, total_q, total_d;    // HOST side only: what the grids are sized for (the step's sizes, or the
                                      // plan's maxima when launches must not depend on the step)
  int32_t Hq, Hkv, D, bs, max_blocks, num_blocks, max_draft;
};

}  // namespace asv
