// The step's metadata built on the device: what as_plan() computes on the host and copies over, computed by one
// CTA from seq_lens / draft_lens that already live in device memory (the lengths a commit has just written, the
// draft lengths a device-side drafter chose), so that a whole step - plan, attention, acceptance, commit - can
// be recorded once and replayed without the host reading anything back.  The cost model and the cut of a pair
// are the shared functions of plan.h: the work list equals the host planner's entry for entry.
#include "plan_dev.cuh"

namespace asv {

namespace {

constexpr int kPlanThreadsMax = 1024;

// Exclusive prefix sum of one value per thread over the block; `total` receives the block's sum.
// `scratch` holds one int64 per warp plus one.
__device__ __forceinline__ int64_t block_scan_excl(int64_t v, int64_t* scratch, int64_t& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int64_t incl = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int64_t up = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += up;
  }
  __syncthreads();                       // scratch may still be read from a previous call
  if (lane == 31) scratch[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int64_t w = lane < (int)(blockDim.x >> 5) ? scratch[lane] : 0;
    int64_t wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int64_t up = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= d) wi += up;
    }
    scratch[lane] = wi - w;               // exclusive prefix of the warp totals
    if (lane == 31) scratch[32] = wi;
  }
  __syncthreads();
  total = scratch[32];
  return scratch[warp] + incl - v;
}

// Inclusive prefix maximum of one int per thread over the block (`scratch`: 33 ints).
__device__ __forceinline__ int block_scan_max_incl(int v, int* scratch) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int up = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v = max(v, up);
  }
  __syncthreads();
  if (lane == 31) scratch[warp] = v;
  __syncthreads();
  if (warp == 0) {
    int w = lane < (int)(blockDim.x >> 5) ? scratch[lane] : -1;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, w, d);
      if (lane >= d) w = max(w, up);
    }
    scratch[lane] = w;                     // inclusive maximum over warps 0..lane
  }
  __syncthreads();
  return warp > 0 ? max(v, scratch[warp - 1]) : v;
}

// Leaves an empty step behind (nothing for any later kernel to do) and records why.
__device__ void write_empty_step(const PlanDevArgs& a) {
  for (int x = threadIdx.x; x < (int)(sizeof(StepHeader) / 4); x += blockDim.x) reinterpret_cast<int32_t*>(a.hdr)[x] = 0;
  for (int kd = 0; kd < a.num_kinds; ++kd)
    for (int c = threadIdx.x; c <= a.kind[kd].num_ctas; c += blockDim.x) a.kind[kd].cta_first[c] = 0;
  if (threadIdx.x == 0) atomicOr(a.status, kFlagBadPlan);
}

__global__ void __launch_bounds__(kPlanThreadsMax, 1) plan_kernel(PlanDevArgs a) {
  __shared__ int64_t scratch[33];
  __shared__ int s_last_owner[kPlanThreadsMax];
  __shared__ int s_max[33];
  __shared__ int s_bad;
  const int tid = threadIdx.x;
  const int kPlanThreads = blockDim.x;                 // a multiple of 32, fixed per plan
  const int B = a.batch;
  if (tid == 0) s_bad = 0;
  for (int x = tid; x < (int)(sizeof(StepHeader) / 4); x += kPlanThreads) reinterpret_cast<int32_t*>(a.hdr)[x] = 0;
  __syncthreads();

  // ---- requests: validation, cu_q / cu_d / first free-list slot, row map --------------------------------
  int64_t cq = 0, cd = 0, cf = 0;       // running totals over the chunks of 1024 requests
  for (int base = 0; base < B; base += kPlanThreads) {
    const int i = base + tid;
    int n = 0, k = 0;
    int64_t need = 0;
    bool bad = false;
    if (i < B) {
      n = a.seq_lens[i];
      k = a.draft_lens[i];
      bad = n < 0 || k < 0 || k > a.max_draft;
      if (!bad) {
        const int64_t pages = ((int64_t)n + k + 1 + a.bs - 1) / a.bs;
        bad = pages > a.max_blocks;
        need = pages - ((int64_t)n + a.bs - 1) / a.bs;
      }
      if (bad) {
        s_bad = 1;
        n = k = 0;
        need = 0;
      }
    }
    int64_t tq, td, tf;
    const int64_t eq = block_scan_excl(i < B ? k + 1 : 0, scratch, tq);
    const int64_t ed = block_scan_excl(i < B ? k : 0, scratch, td);
    const int64_t ef = block_scan_excl(need, scratch, tf);
    if (i < B && cq + eq + k + 1 <= a.max_total_q) {
      a.req[i] = ReqMeta{n, k, (int32_t)(cq + eq), (int32_t)(cd + ed)};
      for (int j = 0; j <= k; ++j) a.row_map[cq + eq + j] = make_int2(i, j);
      a.free_first[i] = (int32_t)(cf + ef);
    }
    cq += tq;
    cd += td;
    cf += tf;
  }
  if (tid == 0) a.free_first[B] = (int32_t)cf;
  __syncthreads();
  if (s_bad || cq > a.max_total_q || (a.assign && cf > a.num_free)) {
    write_empty_step(a);
    return;
  }

  // ---- per layer kind: the split-KV work list -----------------------------------------------------------
  for (int kd = 0; kd < a.num_kinds; ++kd) {
    const PlanDevKind& K = a.kind[kd];
    const int P = K.num_ctas;
    // total cost
    int64_t C = 0;
    for (int base = 0; base < B; base += kPlanThreads) {
      const int i = base + tid;
      int64_t c = 0;
      if (i < B) {
        const ReqMeta r = a.req[i];
        const int pb = plan_block_positions(K.tensor_core, K.rows_on_m, a.G, r.k);
        for (int first = 0; first <= r.k; first += pb) {                     // the request's row blocks
          const int n = r.n + first, k = min(r.k - first, pb - 1);
          const int end = n + k + 1;
          const int lo = K.window > 0 ? max(0, n - K.window + 1) : 0;
          const int t_count = (end + kTileKeys - 1) / kTileKeys - lo / kTileKeys;
          const int rows = a.G * (k + 1);
          c += (plan_item_overhead(K.tensor_core, K.rows_on_m, rows) + t_count * plan_tile_cost(K.tensor_core, K.rows_on_m, K.rows_inst, rows)) * a.Hkv;
        }
      }
      int64_t tot;
      block_scan_excl(c, scratch, tot);
      C += tot;
    }
    for (int c = tid; c <= P; c += kPlanThreads) K.cta_first[c] = 0;
    if (C == 0) {
      if (tid == 0) a.hdr->num_merges[kd * kMaxSub] = 0;
      continue;
    }
    // pairs in (request, row block, kv-head) order, 1024 at a time: count the pieces, then emit them.  (A request has one
    // row block unless the kernel holds fewer rows than it has; blocks beyond its draft length are empty pairs.)
    const int pairs = B * K.row_blocks * a.Hkv;
    int64_t c0_run = 0;                  // cost units before the chunk's first pair
    int64_t items_run = 0, merges_run = 0, prow_run = 0;
    int last_owner_run = -1;             // owner of the last item emitted so far
    bool overflow = false;
    for (int base = 0; base < pairs; base += kPlanThreads) {
      const int pr = base + tid;
      int i = 0, g = 0, t_first = 0, t_count = 0, R = 0, end = 0;
      int64_t cpt = 0, pc = 0, ovh = 0;
      ReqMeta r{};
      if (pr < pairs) {
        i = pr / (K.row_blocks * a.Hkv);
        const int vb = (pr / a.Hkv) % K.row_blocks;
        g = pr % a.Hkv;
        r = a.req[i];
        const int pb = plan_block_positions(K.tensor_core, K.rows_on_m, a.G, r.k);
        const int first = vb * pb;
        if (first <= r.k) {
          // the row block as a request of its own
          r.n += first;
          r.k = min(r.k - first, pb - 1);
          r.cu_q += first;
          end = r.n + r.k + 1;
          const int lo = K.window > 0 ? max(0, r.n - K.window + 1) : 0;
          t_first = lo / kTileKeys;
          t_count = (end + kTileKeys - 1) / kTileKeys - t_first;
          R = a.G * (r.k + 1);
          cpt = plan_tile_cost(K.tensor_core, K.rows_on_m, K.rows_inst, R);
          ovh = plan_item_overhead(K.tensor_core, K.rows_on_m, R);
          pc = ovh + t_count * cpt;
        }
      }
      int64_t chunk_cost;
      const int64_t c0 = c0_run + block_scan_excl(pc, scratch, chunk_cost);
      // count
      int parts = 0, last_owner = -1;
      if (pr < pairs)
        for (int t = 0, t_end, o; t < t_count; t = t_end, ++parts) {
          plan_next_piece(c0 + ovh, t, t_count, cpt, C, P, t_end, o);
          last_owner = o;
        }
      int64_t ti, tm, tp;
      const int64_t item0 = items_run + block_scan_excl(parts, scratch, ti);
      const int64_t merge0 = merges_run + block_scan_excl(parts > 1 ? 1 : 0, scratch, tm);
      const int64_t prow0 = prow_run + block_scan_excl(parts > 1 ? (int64_t)parts * R : 0, scratch, tp);
      if (items_run + ti > a.max_items || merges_run + tm > a.max_merges || prow_run + tp > a.max_part_rows) overflow = true;
      // owner of the last item up to and including this pair (owners never decrease; an empty pair has none of its own)
      s_last_owner[tid] = max(last_owner_run, block_scan_max_incl(last_owner, s_max));
      __syncthreads();
      if (!overflow && pr < pairs) {
        // owner of the item before this pair's first
        const int prev_owner = tid == 0 ? last_owner_run : s_last_owner[tid - 1];
        int po = prev_owner, idx = 0;
        for (int t = 0, t_end, o; t < t_count; t = t_end, ++idx) {
          plan_next_piece(c0 + ovh, t, t_count, cpt, C, P, t_end, o);
          WorkItem w;
          w.req = i;
          w.kv_head = g;
          w.key_begin = (t_first + t) * kTileKeys;
          w.key_end = min(end, (t_first + t_end) * kTileKeys);
          w.part_row = parts > 1 ? (int32_t)(prow0 + (int64_t)idx * R) : -1;
          w.n = r.n;
          w.k = r.k;
          w.cu_q = r.cu_q;
          K.items[item0 + idx] = w;
          // cta_first[c] = first item owned by a CTA >= c
          for (int c = po + 1; c <= o; ++c) K.cta_first[c] = (int32_t)(item0 + idx);
          po = o;
        }
        if (parts > 1) K.merges[merge0] = MergeSeg{i, g, (int32_t)prow0, parts, r.k, r.cu_q};
      }
      const int chunk_last = min(kPlanThreads, pairs - base) - 1;
      const int lo_next = s_last_owner[chunk_last];
      __syncthreads();
      last_owner_run = lo_next;
      c0_run += chunk_cost;
      items_run += ti;
      merges_run += tm;
      prow_run += tp;
    }
    if (overflow) {                      // (uniform across the block: it derives from block-wide totals)
      write_empty_step(a);
      return;
    }
    for (int c = last_owner_run + 1 + tid; c <= P; c += kPlanThreads) K.cta_first[c] = (int32_t)items_run;
    if (tid == 0) a.hdr->num_merges[kd * kMaxSub] = (int32_t)merges_run;
    __syncthreads();
  }
  if (tid == 0) {
    a.hdr->batch = B;
    a.hdr->total_q = (int32_t)cq;
    a.hdr->total_d = (int32_t)cd;
    a.hdr->pad = 0;
  }
}

}  // namespace

cudaError_t launch_plan_device(const PlanDevArgs& a, int max_batch, cudaStream_t s) {
  // one thread per (request, kv-head) pair of a full batch, within [128, 1024]: depends on the plan only, so a
  // recorded launch stays valid for every step
  int threads = (max_batch * a.Hkv + 31) / 32 * 32;
  threads = threads < 128 ? 128 : threads > kPlanThreadsMax ? kPlanThreadsMax : threads;
  plan_kernel<<<1, threads, 0, s>>>(a);
  return cudaGetLastError();
}

}  // namespace asv
