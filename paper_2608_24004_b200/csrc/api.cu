// C ABI of the verify-step library: plan object, host-side planner, launches.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/as_verify.h"
#include "attn_tc.cuh"
#include "lm_head.cuh"
#include "plan_dev.cuh"
#include "kernels.cuh"

using namespace asv;

namespace {

thread_local std::string g_last_error;

int fail(int code, const std::string& msg) {
  g_last_error = msg;
  return code;
}
int fail_cuda(cudaError_t e, const char* where) {
  return fail(AS_ERR_CUDA, std::string(where) + ": " + cudaGetErrorString(e));
}
#define AS_CUDA(call)                                   \
  do {                                                  \
    cudaError_t e__ = (call);                           \
    if (e__ != cudaSuccess) return fail_cuda(e__, #call); \
  } while (0)

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

constexpr int kRowClassCut = 48;     // class boundary in query rows: (.., 48], (48, ..)

struct SubLaunch {           // one attention launch: the requests of one row-count class
  int rows_inst = 0;         // widest request of the class in query rows: picks the kernel instance
  int num_items = 0, num_merges = 0;
  size_t off_items = 0, off_cta_first = 0, off_merges = 0;
};

struct KindStep {            // per layer flavour, for the current step
  int impl = AS_ATTN_SIMT;
  int num_ctas = 0, num_items = 0, num_merges = 0;      // totals over the sub-launches
  int num_sub = 1;
  SubLaunch sub[kMaxSub];
};

}  // namespace

namespace asv {
int record_error(int code, const std::string& msg) { return fail(code, msg); }
}  // namespace asv

struct as_plan_s {
  int device = 0, num_sms = 0;
  int num_kinds = 0;
  as_layer_desc kinds[kMaxKinds];
  int max_batch = 0, max_draft = 0, max_blocks = 0, num_blocks = 0;
  int Hq = 0, Hkv = 0, D = 0, bs = 0, G = 0, rows_max = 0;
  int impl_request = AS_ATTN_AUTO;
  int simt_ctas_per_sm = 1;
  bool fixed_launch = false;     // lay the metadata out at fixed offsets and size every grid for the plan's maxima
  int max_ctas = 0, max_part_rows = 0, max_total_q = 0, max_free = 0;
  int accept_chunks_max = 64;
  int accept_cells_max = 1024;
  // workspace layout
  char* ws = nullptr;
  size_t ws_bytes = 0;
  size_t off_status = 0, off_meta = 0, meta_capacity = 0, off_commit_counts = 0, off_part_o = 0, off_part_ml = 0,
         off_row_part = 0, off_row_final = 0, off_row_ticket = 0, off_recover = 0, off_rec_cells = 0, total_bytes = 0;
  // current step
  bool planned = false;
  int batch = 0, total_q = 0, total_d = 0;
  size_t off_req = 0, off_row_map = 0, off_free_first = 0, off_free_ids = 0;
  KindStep step[kMaxKinds];
  std::vector<char> host_meta;
  TcState tc;                 // tensor-map cache of the tensor-core kernel
  LmHeadState lm;             // tensor-map cache of the fused output projection
  LmHeadState lm_rec;         // ... of its second pass over the recovery rows (as_accept_lm_head_sampled)
  cudaEvent_t prof_begin = nullptr, prof_end = nullptr;
  unsigned long long test_wait_limit_ns = 0;   // as_plan_set_test_stall
  int test_stall_after_loads = -1;
  int64_t launches = 0;
};

namespace {

DevPlan dev_plan(const as_plan_s* p) {
  DevPlan d;
  d.hdr = reinterpret_cast<const StepHeader*>(p->ws + p->off_meta);
  d.req = reinterpret_cast<const ReqMeta*>(p->ws + p->off_req);
  d.row_map = reinterpret_cast<const int2*>(p->ws + p->off_row_map);
  d.status = reinterpret_cast<uint32_t*>(p->ws + p->off_status);
  // grids: the step's own sizes, or the plan's maxima when launches must not depend on the step
  d.batch = p->fixed_launch ? p->max_batch : p->batch;
  d.total_q = p->fixed_launch ? p->max_total_q : p->total_q;
  d.total_d = p->fixed_launch ? p->max_total_q : p->total_d;
  d.Hq = p->Hq;
  d.Hkv = p->Hkv;
  d.D = p->D;
  d.bs = p->bs;
  d.max_blocks = p->max_blocks;
  d.num_blocks = p->num_blocks;
  d.max_draft = p->max_draft;
  return d;
}

int pick_impl(const as_plan_s* p, int kind) {
  const bool tc_ok = attn_tc_supported(p->Hq, p->Hkv, p->D, p->bs, p->max_draft, p->kinds[kind].window);
  if (p->impl_request == AS_ATTN_SIMT) return AS_ATTN_SIMT;
  if (p->impl_request == AS_ATTN_TC) return tc_ok ? AS_ATTN_TC : -1;
  return tc_ok ? AS_ATTN_TC : AS_ATTN_SIMT;
}

// Lays the visible keys of every (request, kv-head) pair end to end in 128-key tiles, weighs every tile
// by what it costs the kernel that will run (a tile of a request with many query rows keeps the softmax
// warpgroups busy for longer than the copy of its K/V bytes takes), adds a fixed cost per pair, gives
// CTA c the cost range [c*C/P, (c+1)*C/P), and emits one work item per (pair, CTA) overlap.  Pairs that
// end up in more than one item get a merge record and partial-buffer rows.
void build_work(const as_plan_s* p, int kind, int impl, int P, int rows_inst, const int32_t* seq, const int32_t* dl, int batch,
                const uint8_t* member /* null: every request */, int& part_rows,
                std::vector<WorkItem>& items, std::vector<int32_t>& cta_first, std::vector<MergeSeg>& merges) {
  const int W = p->kinds[kind].window;
  const bool rows_on_m = impl == AS_ATTN_TC && attn_rows_on_m(p->D, rows_inst);
  // a request is one pair per kv-head, or - where the kernel holds fewer rows than the request has - one per block of
  // draft positions (plan_block_positions): `Blk` is what the kernels see as a request
  struct Blk {
    int32_t req, n, k, cu_q, t_first, t_count;
    int64_t cpt, ovh;
  };
  std::vector<Blk> blks;
  int64_t C = 0;
  int cu_q = 0;
  for (int i = 0; i < batch; cu_q += dl[i] + 1, ++i) {
    if (member && !member[i]) continue;                                // not in this launch
    const int pb = plan_block_positions(impl == AS_ATTN_TC, rows_on_m, p->G, dl[i]);
    for (int first = 0; first <= dl[i]; first += pb) {
      Blk b;
      b.req = i;
      b.n = seq[i] + first;
      b.k = std::min(dl[i] - first, pb - 1);
      b.cu_q = cu_q + first;
      const int end = b.n + b.k + 1;
      const int lo = W > 0 ? std::max(0, b.n - W + 1) : 0;
      b.t_first = lo / kTileKeys;
      b.t_count = (end + kTileKeys - 1) / kTileKeys - b.t_first;
      b.cpt = plan_tile_cost(impl == AS_ATTN_TC, rows_on_m, rows_inst, p->G * (b.k + 1));
      b.ovh = plan_item_overhead(impl == AS_ATTN_TC, rows_on_m, p->G * (b.k + 1));
      C += (b.ovh + b.t_count * b.cpt) * p->Hkv;
      blks.push_back(b);
    }
  }
  items.clear();
  merges.clear();
  cta_first.assign(P + 1, 0);
  if (C == 0) return;
  std::vector<int32_t> owners;
  int64_t c0 = 0;
  for (const Blk& b : blks) {
    const int R = p->G * (b.k + 1);
    const int end = b.n + b.k + 1;
    for (int g = 0; g < p->Hkv; ++g) {
      const size_t first_item = items.size();
      int parts = 0;
      for (int t = 0, t_end, o; t < b.t_count; t = t_end, ++parts) {
        plan_next_piece(c0 + b.ovh, t, b.t_count, b.cpt, C, P, t_end, o);
        WorkItem w{};
        w.req = b.req;
        w.kv_head = g;
        w.key_begin = (b.t_first + t) * kTileKeys;
        w.key_end = std::min(end, (b.t_first + t_end) * kTileKeys);
        w.part_row = -1;
        w.n = b.n;
        w.k = b.k;
        w.cu_q = b.cu_q;
        items.push_back(w);
        owners.push_back(o);
      }
      if (parts > 1) {
        MergeSeg m{b.req, g, part_rows, parts, b.k, b.cu_q};
        merges.push_back(m);
        for (int s = 0; s < parts; ++s) items[first_item + s].part_row = part_rows + s * R;
        part_rows += parts * R;
      }
      c0 += b.ovh + b.t_count * b.cpt;
    }
  }
  // cta_first[c] = first item owned by a CTA >= c
  size_t at = 0;
  for (int c = 0; c <= P; ++c) {
    while (at < items.size() && owners[at] < c) ++at;
    cta_first[c] = (int32_t)at;
  }
}

// Row blocks a request can have at most under this plan (1 unless the keys-on-M kernel serves more than 128 rows).
int max_row_blocks(const as_plan_s* p) {
  if (p->D != 128) return 1;
  int v = 1;
  for (int k = 0; k <= p->max_draft; ++k) {
    const int pb = plan_block_positions(true, false, p->G, k);
    v = std::max(v, (k + pb) / pb);
  }
  return v;
}

// Most query rows a launch item of a request with k drafts has (the request's own, or its widest row block's).
int item_rows(const as_plan_s* p, int impl, int k) {
  const bool tc = impl == AS_ATTN_TC;
  return p->G * std::min(k + 1, plan_block_positions(tc, tc && attn_rows_on_m(p->D, p->G * (k + 1)), p->G, k));
}
// ... of any request with up to kmax drafts: what picks the kernel instance of a launch.
int launch_rows(const as_plan_s* p, int impl, int kmax) {
  int rows = 0;
  for (int k = 0; k <= kmax; ++k) rows = std::max(rows, item_rows(p, impl, k));
  return rows;
}

}  // namespace

extern "C" {

const char* as_status_string(int status) {
  switch (status) {
    case AS_OK: return "ok";
    case AS_ERR_INVALID_ARG: return "invalid argument";
    case AS_ERR_UNSUPPORTED: return "unsupported shape";
    case AS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case AS_ERR_CUDA: return "CUDA call failed";
    case AS_ERR_DEVICE_FLAG: return "a kernel recorded a fault";
    case AS_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    default: return "unknown status";
  }
}

const char* as_last_error(void) { return g_last_error.c_str(); }

int as_plan_create(as_plan_t** out, const as_layer_desc* kinds, int num_kinds, int max_batch, int max_draft,
                   int max_blocks_per_req, int num_blocks, int device) {
  if (!out || !kinds) return fail(AS_ERR_INVALID_ARG, "as_plan_create: null pointer");
  *out = nullptr;
  if (num_kinds < 1 || num_kinds > kMaxKinds) return fail(AS_ERR_UNSUPPORTED, "as_plan_create: num_kinds must be 1..4");
  if (max_batch < 1 || max_draft < 0 || max_blocks_per_req < 1 || num_blocks < 1 || device < 0)
    return fail(AS_ERR_INVALID_ARG, "as_plan_create: sizes must be positive");
  const as_layer_desc& k0 = kinds[0];
  for (int i = 0; i < num_kinds; ++i) {
    const as_layer_desc& k = kinds[i];
    if (k.num_q_heads != k0.num_q_heads || k.num_kv_heads != k0.num_kv_heads || k.head_dim != k0.head_dim ||
        k.block_size != k0.block_size)
      return fail(AS_ERR_UNSUPPORTED, "as_plan_create: all layer kinds must share heads, head_dim and block_size");
    if (k.window < 0 || !(k.sm_scale >= 0.f)) return fail(AS_ERR_INVALID_ARG, "as_plan_create: bad window or sm_scale");
  }
  if (k0.num_kv_heads < 1 || k0.num_q_heads < 1 || k0.num_q_heads % k0.num_kv_heads != 0)
    return fail(AS_ERR_INVALID_ARG, "as_plan_create: num_q_heads must be a positive multiple of num_kv_heads");
  if (k0.head_dim != 64 && k0.head_dim != 128) return fail(AS_ERR_UNSUPPORTED, "as_plan_create: head_dim must be 64 or 128");
  if (k0.block_size != 16 && k0.block_size != 32 && k0.block_size != 64 && k0.block_size != 128)
    return fail(AS_ERR_UNSUPPORTED, "as_plan_create: block_size must be 16, 32, 64 or 128");
  const int G = k0.num_q_heads / k0.num_kv_heads;
  if ((int64_t)G * (max_draft + 1) > kMaxRows)
    return fail(AS_ERR_UNSUPPORTED, "as_plan_create: G * (max_draft + 1) must be <= 256");
  if ((int64_t)max_batch * (max_draft + 1) > (1 << 24)) return fail(AS_ERR_INVALID_ARG, "as_plan_create: batch too large");

  as_plan_s* p = new (std::nothrow) as_plan_s();
  if (!p) return fail(AS_ERR_INVALID_ARG, "as_plan_create: out of host memory");
  p->device = device;
  p->num_kinds = num_kinds;
  for (int i = 0; i < num_kinds; ++i) p->kinds[i] = kinds[i];
  p->max_batch = max_batch;
  p->max_draft = max_draft;
  p->max_blocks = max_blocks_per_req;
  p->num_blocks = num_blocks;
  p->Hq = k0.num_q_heads;
  p->Hkv = k0.num_kv_heads;
  p->D = k0.head_dim;
  p->bs = k0.block_size;
  p->G = G;
  p->rows_max = G * (max_draft + 1);
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms <= 0) {
    cudaGetLastError();
    sms = 148;                 // no device visible (host-only use): size for a B200
  }
  p->num_sms = sms;
  const size_t simt_smem = attn_simt_smem_bytes(p->rows_max, p->D);
  if (simt_smem > 227 * 1024) {
    delete p;
    return fail(AS_ERR_UNSUPPORTED, "as_plan_create: rows x head_dim too large for shared memory");
  }
  p->simt_ctas_per_sm = (int)std::max<size_t>(1, std::min<size_t>(4, (227 * 1024) / (simt_smem + 1024)));
  p->max_ctas = sms * 4;
  p->max_part_rows = 2 * kMaxSub * p->max_ctas * p->rows_max;
  p->max_total_q = max_batch * (max_draft + 1);
  p->max_free = max_batch * ((max_draft + 1 + p->bs - 1) / p->bs + 1);

  // workspace: [status | per-step metadata | commit counts | split partials | accept scratch]
  size_t off = 0;
  p->off_status = off;
  off += 256;
  p->off_meta = off;
  size_t meta = 0;
  meta += align_up(sizeof(StepHeader), 16);
  meta += align_up(sizeof(ReqMeta) * max_batch, 16);
  meta += align_up(sizeof(int2) * p->max_total_q, 16);
  meta += align_up(sizeof(int32_t) * (max_batch + 1), 16);
  meta += align_up(sizeof(int32_t) * p->max_free, 16);
  const size_t max_items = (size_t)max_batch * p->Hkv * max_row_blocks(p) + kMaxSub * p->max_ctas;
  for (int i = 0; i < num_kinds; ++i) {
    meta += align_up(sizeof(WorkItem) * max_items, 16);
    meta += kMaxSub * align_up(sizeof(int32_t) * (p->max_ctas + 1), 16);
    meta += kMaxSub * align_up(sizeof(MergeSeg) * p->max_ctas, 16);
  }
  p->meta_capacity = meta;
  off += align_up(meta, 256);
  p->off_commit_counts = off;
  off += align_up(sizeof(int32_t) * (max_batch + 1), 256);
  p->off_part_o = off;
  off += align_up(sizeof(float) * (size_t)p->max_part_rows * p->D, 256);
  p->off_part_ml = off;
  off += align_up(sizeof(float2) * (size_t)p->max_part_rows, 256);
  p->off_row_part = off;
  off += align_up(sizeof(float4) * (size_t)p->max_total_q * p->accept_chunks_max, 256);
  p->off_row_final = off;
  off += align_up(sizeof(float4) * (size_t)p->max_total_q, 256);
  p->off_row_ticket = off;
  off += align_up(sizeof(int32_t) * (size_t)p->max_total_q, 256);
  p->off_recover = off;
  off += align_up(sizeof(int32_t) * max_batch, 256);
  p->off_rec_cells = off;
  off += align_up(sizeof(double) * 2 * (size_t)max_batch * p->accept_cells_max, 256);
  p->total_bytes = off;
  p->host_meta.resize(meta);
  *out = p;
  return AS_OK;
}

int as_plan_destroy(as_plan_t* plan) {
  if (!plan) return AS_OK;
  delete plan;
  return AS_OK;
}

size_t as_plan_workspace_bytes(const as_plan_t* plan) { return plan ? plan->total_bytes : 0; }

int as_plan_bind(as_plan_t* plan, void* dev_workspace, size_t bytes) {
  if (!plan) return fail(AS_ERR_INVALID_ARG, "as_plan_bind: null plan");
  if (!dev_workspace || (reinterpret_cast<uintptr_t>(dev_workspace) & 255) != 0 || bytes < plan->total_bytes)
    return fail(AS_ERR_WORKSPACE, "as_plan_bind: workspace null, not 256-byte aligned, or too small");
  DeviceGuard guard(plan->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_plan_bind: cannot select the plan's device");
  AS_CUDA(cudaMemset(dev_workspace, 0, 256));
  AS_CUDA(cudaMemset(static_cast<char*>(dev_workspace) + plan->off_row_ticket, 0, sizeof(int32_t) * (size_t)plan->max_total_q));
  AS_CUDA(cudaDeviceSynchronize());
  plan->ws = static_cast<char*>(dev_workspace);
  plan->ws_bytes = bytes;
  plan->planned = false;
  return AS_OK;
}

int as_plan_set_attn_impl(as_plan_t* plan, int impl) {
  if (!plan || impl < AS_ATTN_AUTO || impl > AS_ATTN_TC) return fail(AS_ERR_INVALID_ARG, "as_plan_set_attn_impl: bad argument");
  plan->impl_request = impl;
  plan->planned = false;
  return AS_OK;
}

int as_plan_set_fixed_launch(as_plan_t* plan, int on) {
  if (!plan) return fail(AS_ERR_INVALID_ARG, "as_plan_set_fixed_launch: null plan");
  plan->fixed_launch = on != 0;
  plan->planned = false;
  return AS_OK;
}

int as_plan(as_plan_t* p, int batch, const int32_t* seq_lens, const int32_t* draft_lens, int32_t* block_table,
            const int32_t* free_blocks, int num_free, int* num_taken, void* stream) {
  if (!p || !seq_lens || !draft_lens || !block_table) return fail(AS_ERR_INVALID_ARG, "as_plan: null pointer");
  if (!p->ws) return fail(AS_ERR_WORKSPACE, "as_plan: no workspace bound");
  if (batch < 0 || batch > p->max_batch) return fail(AS_ERR_INVALID_ARG, "as_plan: batch outside [0, max_batch]");
  if (num_free < 0 || (num_free > 0 && !free_blocks)) return fail(AS_ERR_INVALID_ARG, "as_plan: bad free list");
  p->planned = false;
  int64_t tq = 0, td = 0, need_free = 0;
  for (int i = 0; i < batch; ++i) {
    if (seq_lens[i] < 0 || draft_lens[i] < 0 || draft_lens[i] > p->max_draft)
      return fail(AS_ERR_INVALID_ARG, "as_plan: seq_len < 0 or draft_len outside [0, max_draft]");
    const int64_t need = ((int64_t)seq_lens[i] + draft_lens[i] + 1 + p->bs - 1) / p->bs;
    if (need > p->max_blocks) return fail(AS_ERR_INVALID_ARG, "as_plan: a request needs more pages than max_blocks_per_req");
    need_free += need - ((int64_t)seq_lens[i] + p->bs - 1) / p->bs;
    tq += draft_lens[i] + 1;
    td += draft_lens[i];
  }
  const bool assign = free_blocks != nullptr;
  if (assign && need_free > num_free) return fail(AS_ERR_INVALID_ARG, "as_plan: free list too short for this step");
  if (assign)
    for (int64_t x = 0; x < need_free; ++x)
      if (free_blocks[x] < 0 || free_blocks[x] >= p->num_blocks) return fail(AS_ERR_INVALID_ARG, "as_plan: free page id out of range");
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_plan: cannot select the plan's device");

  p->batch = batch;
  p->total_q = (int)tq;
  p->total_d = (int)td;
  int kmax_step = 0;
  for (int i = 0; i < batch; ++i) kmax_step = std::max(kmax_step, (int)draft_lens[i]);
  char* hm = p->host_meta.data();
  size_t off = 0;
  // every array takes what this step needs, or - with fixed launches - its full capacity, so that its
  // device address is the same in every step
  auto take = [&](size_t bytes, size_t capacity) {
    const size_t at = off;
    off += align_up(p->fixed_launch ? capacity : bytes, 16);
    return at;
  };
  const size_t max_items = (size_t)p->max_batch * p->Hkv * max_row_blocks(p) + kMaxSub * p->max_ctas;
  const size_t o_hdr = take(sizeof(StepHeader), sizeof(StepHeader));
  const size_t o_req = take(sizeof(ReqMeta) * batch, sizeof(ReqMeta) * p->max_batch);
  const size_t o_map = take(sizeof(int2) * tq, sizeof(int2) * p->max_total_q);
  const size_t o_ff = take(sizeof(int32_t) * (batch + 1), sizeof(int32_t) * (p->max_batch + 1));
  const size_t o_fi = take(sizeof(int32_t) * (assign ? need_free : 0), sizeof(int32_t) * p->max_free);
  StepHeader* hdr = reinterpret_cast<StepHeader*>(hm + o_hdr);
  *hdr = StepHeader{};
  hdr->batch = batch;
  hdr->total_q = (int32_t)tq;
  hdr->total_d = (int32_t)td;
  ReqMeta* rm = reinterpret_cast<ReqMeta*>(hm + o_req);
  int2* map = reinterpret_cast<int2*>(hm + o_map);
  int32_t* ff = reinterpret_cast<int32_t*>(hm + o_ff);
  int cq = 0, cd = 0, cf = 0;
  for (int i = 0; i < batch; ++i) {
    rm[i] = ReqMeta{seq_lens[i], draft_lens[i], cq, cd};
    for (int j = 0; j <= draft_lens[i]; ++j) map[cq + j] = make_int2(i, j);
    ff[i] = cf;
    cf += (seq_lens[i] + draft_lens[i] + 1 + p->bs - 1) / p->bs - (seq_lens[i] + p->bs - 1) / p->bs;
    cq += draft_lens[i] + 1;
    cd += draft_lens[i];
  }
  ff[batch] = cf;
  if (assign && need_free) std::memcpy(hm + o_fi, free_blocks, sizeof(int32_t) * need_free);
  if (num_taken) *num_taken = assign ? (int)need_free : 0;

  std::vector<WorkItem> items;
  std::vector<int32_t> cta_first;
  std::vector<MergeSeg> merges;
  for (int kd = 0; kd < p->num_kinds; ++kd) {
    KindStep& st = p->step[kd];
    st.impl = pick_impl(p, kd);
    if (st.impl < 0) return fail(AS_ERR_UNSUPPORTED, "as_plan: the tensor-core attention kernel does not cover this shape");
    st.num_ctas = st.impl == AS_ATTN_TC ? p->num_sms : p->num_sms * p->simt_ctas_per_sm;
    // Requests are bucketed by row count when the step mixes short and long drafts: a launch runs the kernel
    // instance of its widest request, and narrow requests run markedly faster in a narrow instance (and a
    // launch of like requests balances better).  Two classes at most; one when launches must be fixed, when
    // the step is small, or when a class would be nearly empty.
    std::vector<uint8_t> member[kMaxSub];
    const int rows_kind = launch_rows(p, st.impl, p->fixed_launch ? p->max_draft : kmax_step);
    int rows_of[kMaxSub] = {rows_kind};
    st.num_sub = 1;
    // (the rows-on-M kernel's tile cost does not depend on the row count: nothing to gain there)
    if (st.impl == AS_ATTN_TC && !p->fixed_launch && rows_kind > kRowClassCut && !attn_rows_on_m(p->D, rows_kind)) {
      int cuts[kMaxSub - 1];
      for (int c = 0; c < kMaxSub - 1; ++c) cuts[c] = 1 << 30;
      cuts[0] = kRowClassCut;
      int64_t tiles[kMaxSub] = {};
      int rows_max_of[kMaxSub] = {};
      std::vector<uint8_t> cls(batch);
      for (int i = 0; i < batch; ++i) {
        const int R = item_rows(p, st.impl, draft_lens[i]);      // (a wide request counts by its row blocks)
        int c = 0;
        while (c < kMaxSub - 1 && R > cuts[c]) ++c;
        cls[i] = (uint8_t)c;
        const int W = p->kinds[kd].window;
        const int lo = W > 0 ? std::max(0, seq_lens[i] - W + 1) : 0;
        tiles[c] += (seq_lens[i] + draft_lens[i] + kTileKeys) / kTileKeys - lo / kTileKeys;   // visible tiles
        rows_max_of[c] = std::max(rows_max_of[c], R);
      }
      int64_t all = 0;
      for (int c = 0; c < kMaxSub; ++c) all += tiles[c];
      if (all * p->Hkv >= 64 * (int64_t)st.num_ctas) {
        // a class with less than an eighth of the work joins the next wider one (the widest joins the one below)
        int to[kMaxSub];
        for (int c = 0; c < kMaxSub; ++c) to[c] = c;
        for (int c = 0; c < kMaxSub - 1; ++c)
          if (tiles[c] * 8 < all) {
            to[c] = c + 1;
            tiles[c + 1] += tiles[c];
            rows_max_of[c + 1] = std::max(rows_max_of[c + 1], rows_max_of[c]);
            tiles[c] = 0;
          }
        if (tiles[kMaxSub - 1] * 8 < all) {
          int below = kMaxSub - 2;
          while (below > 0 && tiles[below] == 0) --below;
          if (tiles[below] > 0) {
            to[kMaxSub - 1] = below;
            tiles[below] += tiles[kMaxSub - 1];
            rows_max_of[below] = std::max(rows_max_of[below], rows_max_of[kMaxSub - 1]);
            tiles[kMaxSub - 1] = 0;
          }
        }
        int slot_of[kMaxSub], n = 0;
        for (int c = 0; c < kMaxSub; ++c) slot_of[c] = -1;
        for (int c = 0; c < kMaxSub; ++c)
          if (tiles[c] > 0) {
            slot_of[c] = n;
            rows_of[n] = rows_max_of[c];
            member[n].assign(batch, 0);
            ++n;
          }
        if (n > 1) {
          st.num_sub = n;
          for (int i = 0; i < batch; ++i) {
            int c = cls[i];
            while (slot_of[c] < 0 || to[c] != c) {         // follow the joins to a class that kept its own launch
              if (to[c] == c) break;
              c = to[c];
            }
            member[slot_of[c]][i] = 1;
          }
        } else {
          rows_of[0] = rows_kind;
        }
      }
    }
    st.num_items = 0;
    st.num_merges = 0;
    int part_rows = 0;
    for (int sb = 0; sb < st.num_sub; ++sb) {
      SubLaunch& sl = st.sub[sb];
      sl.rows_inst = rows_of[sb];
      build_work(p, kd, st.impl, st.num_ctas, sl.rows_inst, seq_lens, draft_lens, batch,
                 st.num_sub > 1 ? member[sb].data() : nullptr, part_rows, items, cta_first, merges);
      sl.num_items = (int)items.size();
      sl.num_merges = (int)merges.size();
      st.num_items += sl.num_items;
      st.num_merges += sl.num_merges;
      if (st.num_items > (int)max_items || merges.size() > (size_t)p->max_ctas || cta_first.size() > (size_t)p->max_ctas + 1 ||
          part_rows > p->max_part_rows)
        return fail(AS_ERR_WORKSPACE, "as_plan: work list exceeds the planned capacity");
      hdr->num_merges[kd * kMaxSub + sb] = sl.num_merges;
      // (with fixed launches there is one sub-launch, which takes the kind's full capacity)
      sl.off_items = take(sizeof(WorkItem) * items.size(), sizeof(WorkItem) * max_items);
      sl.off_cta_first = take(sizeof(int32_t) * cta_first.size(), sizeof(int32_t) * (p->max_ctas + 1));
      sl.off_merges = take(sizeof(MergeSeg) * merges.size(), sizeof(MergeSeg) * p->max_ctas);
      if (off > p->meta_capacity) return fail(AS_ERR_WORKSPACE, "as_plan: metadata exceeds the planned capacity");
      if (!items.empty()) std::memcpy(hm + sl.off_items, items.data(), sizeof(WorkItem) * items.size());
      std::memcpy(hm + sl.off_cta_first, cta_first.data(), sizeof(int32_t) * cta_first.size());
      if (!merges.empty()) std::memcpy(hm + sl.off_merges, merges.data(), sizeof(MergeSeg) * merges.size());
      sl.off_items += p->off_meta;
      sl.off_cta_first += p->off_meta;
      sl.off_merges += p->off_meta;
    }
  }
  p->off_req = p->off_meta + o_req;
  p->off_row_map = p->off_meta + o_map;
  p->off_free_first = p->off_meta + o_ff;
  p->off_free_ids = p->off_meta + o_fi;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (off) AS_CUDA(cudaMemcpyAsync(p->ws + p->off_meta, hm, off, cudaMemcpyHostToDevice, s));
  if (assign && need_free) {
    const DevPlan d = dev_plan(p);
    AS_CUDA(launch_assign_pages(d, block_table, reinterpret_cast<const int32_t*>(p->ws + p->off_free_ids),
                                reinterpret_cast<const int32_t*>(p->ws + p->off_free_first), s));
    p->launches += 1;
  }
  p->planned = true;
  return AS_OK;
}

int as_plan_device(as_plan_t* p, int batch, const int32_t* seq_lens, const int32_t* draft_lens, int32_t* block_table,
                   const int32_t* free_blocks, int num_free, void* stream) {
  if (!p || !seq_lens || !draft_lens || !block_table) return fail(AS_ERR_INVALID_ARG, "as_plan_device: null pointer");
  if (!p->ws) return fail(AS_ERR_WORKSPACE, "as_plan_device: no workspace bound");
  if (!p->fixed_launch) return fail(AS_ERR_INVALID_ARG, "as_plan_device: needs fixed launches (as_plan_set_fixed_launch)");
  if (batch < 0 || batch > p->max_batch) return fail(AS_ERR_INVALID_ARG, "as_plan_device: batch outside [0, max_batch]");
  if (num_free < 0 || (num_free > 0 && !free_blocks)) return fail(AS_ERR_INVALID_ARG, "as_plan_device: bad free list");
  p->planned = false;
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_plan_device: cannot select the plan's device");
  // the host knows the number of requests only; every grid is sized for the plan's maxima (fixed launches)
  p->batch = batch;
  p->total_q = p->max_total_q;
  p->total_d = p->max_draft > 0 ? p->max_total_q : 0;   // (what as_accept's null check goes by: drafts are possible)
  // the same fixed layout as_plan() uses with fixed launches: every array at its full capacity
  size_t off = 0;
  auto take = [&](size_t capacity) {
    const size_t at = off;
    off += align_up(capacity, 16);
    return at;
  };
  const size_t max_items = (size_t)p->max_batch * p->Hkv * max_row_blocks(p) + kMaxSub * p->max_ctas;
  const size_t o_hdr = take(sizeof(StepHeader));
  const size_t o_req = take(sizeof(ReqMeta) * p->max_batch);
  const size_t o_map = take(sizeof(int2) * p->max_total_q);
  const size_t o_ff = take(sizeof(int32_t) * (p->max_batch + 1));
  take(sizeof(int32_t) * p->max_free);               // (the host planner's copy of the free list: unused here)
  PlanDevArgs a{};
  a.seq_lens = seq_lens;
  a.draft_lens = draft_lens;
  a.batch = batch;
  char* meta = p->ws + p->off_meta;
  a.hdr = reinterpret_cast<StepHeader*>(meta + o_hdr);
  a.req = reinterpret_cast<ReqMeta*>(meta + o_req);
  a.row_map = reinterpret_cast<int2*>(meta + o_map);
  a.free_first = reinterpret_cast<int32_t*>(meta + o_ff);
  a.status = reinterpret_cast<uint32_t*>(p->ws + p->off_status);
  a.num_kinds = p->num_kinds;
  for (int kd = 0; kd < p->num_kinds; ++kd) {
    KindStep& st = p->step[kd];
    st.impl = pick_impl(p, kd);
    if (st.impl < 0) return fail(AS_ERR_UNSUPPORTED, "as_plan_device: the tensor-core attention kernel does not cover this shape");
    st.num_ctas = st.impl == AS_ATTN_TC ? p->num_sms : p->num_sms * p->simt_ctas_per_sm;
    st.num_sub = 1;
    SubLaunch& sl = st.sub[0];
    sl.rows_inst = launch_rows(p, st.impl, p->max_draft);
    // counts stay on the device: the merge grid covers the capacity, the kernels read the step's counts
    sl.num_items = st.num_items = -1;
    sl.num_merges = st.num_merges = p->max_ctas;
    sl.off_items = p->off_meta + take(sizeof(WorkItem) * max_items);
    sl.off_cta_first = p->off_meta + take(sizeof(int32_t) * (p->max_ctas + 1));
    sl.off_merges = p->off_meta + take(sizeof(MergeSeg) * p->max_ctas);
    PlanDevKind& K = a.kind[kd];
    K.items = reinterpret_cast<WorkItem*>(p->ws + sl.off_items);
    K.cta_first = reinterpret_cast<int32_t*>(p->ws + sl.off_cta_first);
    K.merges = reinterpret_cast<MergeSeg*>(p->ws + sl.off_merges);
    K.window = p->kinds[kd].window;
    K.num_ctas = st.num_ctas;
    K.rows_inst = sl.rows_inst;
    K.tensor_core = st.impl == AS_ATTN_TC;
    K.rows_on_m = K.tensor_core && attn_rows_on_m(p->D, sl.rows_inst);
    K.row_blocks = K.tensor_core && !K.rows_on_m ? max_row_blocks(p) : 1;
  }
  if (off > p->meta_capacity) return fail(AS_ERR_WORKSPACE, "as_plan_device: metadata exceeds the planned capacity");
  a.G = p->G;
  a.Hkv = p->Hkv;
  a.bs = p->bs;
  a.max_blocks = p->max_blocks;
  a.max_draft = p->max_draft;
  a.max_total_q = p->max_total_q;
  a.max_items = (int64_t)max_items;
  a.max_merges = p->max_ctas;
  a.max_part_rows = p->max_part_rows;
  a.assign = free_blocks != nullptr;
  a.num_free = num_free;
  p->off_req = p->off_meta + o_req;
  p->off_row_map = p->off_meta + o_map;
  p->off_free_first = p->off_meta + o_ff;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  AS_CUDA(launch_plan_device(a, p->max_batch, s));
  p->launches += 1;
  if (a.assign && batch > 0) {
    const DevPlan d = dev_plan(p);
    AS_CUDA(launch_assign_pages(d, block_table, free_blocks, a.free_first, s));
    p->launches += 1;
  }
  p->planned = true;
  return AS_OK;
}

int as_verify_attn(as_plan_t* p, int kind, const void* q, const void* k_new, const void* v_new, void* k_pool,
                   void* v_pool, const int32_t* block_table, void* out, float* lse, void* stream) {
  if (!p || !q || !k_new || !v_new || !k_pool || !v_pool || !block_table || !out)
    return fail(AS_ERR_INVALID_ARG, "as_verify_attn: null pointer");
  if (!p->planned) return fail(AS_ERR_INVALID_ARG, "as_verify_attn: as_plan() has not been called for this step");
  if (kind < 0 || kind >= p->num_kinds) return fail(AS_ERR_INVALID_ARG, "as_verify_attn: kind out of range");
  if ((reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool) | reinterpret_cast<uintptr_t>(q) |
       reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(out)) & 15)
    return fail(AS_ERR_INVALID_ARG, "as_verify_attn: tensors must be 16-byte aligned");
  if (p->batch == 0) return AS_OK;
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_verify_attn: cannot select the plan's device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const DevPlan d = dev_plan(p);
  const KindStep& st = p->step[kind];
  const as_layer_desc& L = p->kinds[kind];
  AS_CUDA(launch_append(d, static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                        static_cast<__nv_bfloat16*>(k_pool), static_cast<__nv_bfloat16*>(v_pool), block_table, s));
  AttnArgs A;
  A.q = static_cast<const __nv_bfloat16*>(q);
  A.k_pool = static_cast<const __nv_bfloat16*>(k_pool);
  A.v_pool = static_cast<const __nv_bfloat16*>(v_pool);
  A.block_table = block_table;
  A.out = static_cast<__nv_bfloat16*>(out);
  A.lse = lse;
  A.sinks = L.sinks;
  A.window = L.window;
  const float scale = L.sm_scale > 0.f ? L.sm_scale : 1.0f / std::sqrt((float)p->D);
  A.scale_log2 = scale * 1.4426950408889634f;
  A.part_o = reinterpret_cast<float*>(p->ws + p->off_part_o);
  A.part_ml = reinterpret_cast<float2*>(p->ws + p->off_part_ml);
  A.num_ctas = st.num_ctas;
  A.wait_limit_ns = p->test_wait_limit_ns;
  A.stall_after_loads = p->test_stall_after_loads;
  if (p->prof_begin && p->prof_end) AS_CUDA(cudaEventRecord(p->prof_begin, s));
  for (int sb = 0; sb < st.num_sub; ++sb) {
    const SubLaunch& sl = st.sub[sb];
    A.items = reinterpret_cast<const WorkItem*>(p->ws + sl.off_items);
    A.cta_first = reinterpret_cast<const int32_t*>(p->ws + sl.off_cta_first);
    A.rows_step = sl.rows_inst;
    if (sl.num_items == 0 && !p->fixed_launch) continue;
    if (st.impl == AS_ATTN_TC) {
      std::string err;
      const int rc = launch_attn_tc(d, A, p->tc, s, err);
      if (rc != AS_OK) return fail(rc, "as_verify_attn: " + err);
    } else {
      AS_CUDA(launch_attn_simt(d, A, s));
    }
    p->launches += 1;
  }
  if (p->prof_begin && p->prof_end) AS_CUDA(cudaEventRecord(p->prof_end, s));
  for (int sb = 0; sb < st.num_sub; ++sb) {
    const SubLaunch& sl = st.sub[sb];
    A.merges = reinterpret_cast<const MergeSeg*>(p->ws + sl.off_merges);
    A.num_merges = p->fixed_launch ? p->max_ctas : sl.num_merges;
    A.num_merges_dev = &d.hdr->num_merges[kind * kMaxSub + sb];
    AS_CUDA(launch_attn_merge(d, A, s));
    if (A.num_merges > 0) p->launches += 1;
  }
  p->launches += 1;                                   // the append kernel
  return AS_OK;
}

namespace {
int accept_impl(as_plan_t* p, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
                const float* draft_probs, const float* temperature, const float* u, const float* w,
                const uint64_t* rng, int32_t* accept_len, int32_t* out_tokens, void* stream);
}

int as_accept(as_plan_t* p, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
              const float* draft_probs, const float* temperature, const float* u, const float* w,
              int32_t* accept_len, int32_t* out_tokens, void* stream) {
  if (temperature && (!u || !w)) return fail(AS_ERR_INVALID_ARG, "as_accept: sampling needs u and w");
  return accept_impl(p, logits, ld, vocab, draft_tokens, draft_probs, temperature, u, w, nullptr, accept_len, out_tokens,
                     stream);
}

int as_accept_lm_head(as_plan_t* p, const void* hidden, const void* weight, int hidden_dim, int vocab,
                      const int32_t* draft_tokens, int32_t* accept_len, int32_t* out_tokens, void* stream) {
  if (!p || !hidden || !weight || !accept_len || !out_tokens) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head: null pointer");
  if (!p->planned) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head: as_plan() has not been called for this step");
  if (vocab < 1 || hidden_dim < 64 || hidden_dim % 64 != 0)
    return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head: need vocab >= 1 and hidden_dim a positive multiple of 64");
  if ((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(weight)) & 15)
    return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head: hidden and weight must be 16-byte aligned");
  if (p->total_d > 0 && !draft_tokens) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head: draft_tokens is null");
  if (p->batch == 0) return AS_OK;
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_accept_lm_head: cannot select the plan's device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const DevPlan d = dev_plan(p);
  AcceptArgs A{};
  A.vocab = vocab;
  A.draft_tokens = draft_tokens;
  A.accept_len = accept_len;
  A.out_tokens = out_tokens;
  A.row_final = reinterpret_cast<float4*>(p->ws + p->off_row_final);
  A.recover_row = reinterpret_cast<int32_t*>(p->ws + p->off_recover);
  // (the per-chunk row statistics of as_accept are not needed here: their space holds the packed maxima)
  std::string err;
  const int rc = launch_lm_head_argmax(d, p->lm, hidden, weight, hidden_dim, vocab, d.total_q, p->num_sms,
                                       reinterpret_cast<unsigned long long*>(p->ws + p->off_row_part), A.row_final, s, err);
  if (rc != 0) return fail(rc, "as_accept_lm_head: " + err);
  AS_CUDA(launch_decide(d, A, s));
  p->launches += 3;
  return AS_OK;
}

size_t as_accept_lm_head_scratch_bytes(const as_plan_t* p, int hidden_dim, int vocab) {
  if (!p || hidden_dim < 1 || vocab < 1) return 0;
  const size_t ld = align_up((size_t)vocab, 4);
  const size_t logits = sizeof(float) * (size_t)p->max_batch * ld;
  const size_t parts = sizeof(float2) * (size_t)p->max_total_q * lm_head_vocab_tiles(vocab);
  return align_up(std::max(logits, parts), 256) + align_up(sizeof(uint16_t) * (size_t)p->max_batch * hidden_dim, 256) +
         align_up(sizeof(float) * (size_t)p->max_total_q, 256);
}

int as_accept_lm_head_sampled(as_plan_t* p, const void* hidden, const void* weight, int hidden_dim, int vocab,
                              const int32_t* draft_tokens, const float* draft_probs, int64_t ld, const float* temperature,
                              const float* u, const float* w, const uint64_t* rng_state, void* scratch, size_t scratch_bytes,
                              int32_t* accept_len, int32_t* out_tokens, void* stream) {
  if (!p || !hidden || !weight || !accept_len || !out_tokens || !temperature || !scratch)
    return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: null pointer");
  if (!p->planned) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: as_plan() has not been called for this step");
  if (vocab < 1 || hidden_dim < 64 || hidden_dim % 64 != 0)
    return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: need vocab >= 1 and hidden_dim a positive multiple of 64");
  if (!rng_state && (!u || !w)) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: sampling needs u and w, or rng_state");
  if (draft_probs && ld < vocab) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: need ld >= vocab for draft_probs");
  if ((reinterpret_cast<uintptr_t>(hidden) | reinterpret_cast<uintptr_t>(weight)) & 15)
    return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: hidden and weight must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(scratch) & 255) || scratch_bytes < as_accept_lm_head_scratch_bytes(p, hidden_dim, vocab))
    return fail(AS_ERR_WORKSPACE, "as_accept_lm_head_sampled: scratch not 256-byte aligned or smaller than as_accept_lm_head_scratch_bytes()");
  if (p->total_d > 0 && !draft_tokens) return fail(AS_ERR_INVALID_ARG, "as_accept_lm_head_sampled: draft_tokens is null");
  if (p->batch == 0) return AS_OK;
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_accept_lm_head_sampled: cannot select the plan's device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const DevPlan d = dev_plan(p);
  // scratch: [logits of the recovery rows | tile partials of the first pass (dead before the logits are written)]
  // [hidden states of the recovery rows] [logit of every row's draft token]
  const size_t rec_ld = align_up((size_t)vocab, 4);
  char* sc = static_cast<char*>(scratch);
  const size_t logits_bytes = sizeof(float) * (size_t)p->max_batch * rec_ld;
  const size_t parts_bytes = sizeof(float2) * (size_t)p->max_total_q * lm_head_vocab_tiles(vocab);
  float* rec_logits = reinterpret_cast<float*>(sc);
  float2* tile_part = reinterpret_cast<float2*>(sc);
  char* hidden_rows = sc + align_up(std::max(logits_bytes, parts_bytes), 256);
  float* zd = reinterpret_cast<float*>(hidden_rows + align_up(sizeof(uint16_t) * (size_t)p->max_batch * hidden_dim, 256));
  AcceptArgs A{};
  A.ld = draft_probs ? ld : vocab;
  A.vocab = vocab;
  A.draft_tokens = draft_tokens;
  A.draft_probs = draft_probs;
  A.temperature = temperature;
  A.u = u;
  A.w = w;
  A.rng = rng_state;
  A.accept_len = accept_len;
  A.out_tokens = out_tokens;
  A.row_final = reinterpret_cast<float4*>(p->ws + p->off_row_final);
  A.recover_row = reinterpret_cast<int32_t*>(p->ws + p->off_recover);
  A.rec_cells = reinterpret_cast<double*>(p->ws + p->off_rec_cells);
  A.zd = zd;
  A.rec_logits = rec_logits;
  A.rec_ld = (int64_t)rec_ld;
  int chunk = 16384;
  while ((vocab + chunk - 1) / chunk > p->accept_chunks_max) chunk *= 2;
  A.chunk_elems = chunk;
  A.chunks = (vocab + chunk - 1) / chunk;
  int cell = 512;                            // (a cell costs its warp two fp64 reductions: few, large cells)
  while ((vocab + cell - 1) / cell > p->accept_cells_max) cell *= 2;
  A.cell_elems = cell;
  A.cells = (vocab + cell - 1) / cell;
  std::string err;
  // pass 1 over the weights: argmax, softmax statistics per row, the logit of each draft token
  int rc = launch_lm_head_stats(d, p->lm, hidden, weight, hidden_dim, vocab, d.total_q, p->num_sms,
                                reinterpret_cast<unsigned long long*>(p->ws + p->off_row_part), tile_part, zd, draft_tokens,
                                temperature, A.row_final, s, err);
  if (rc != 0) return fail(rc, "as_accept_lm_head_sampled: " + err);
  AS_CUDA(launch_decide(d, A, s));
  // pass 2, over the one row per request whose recovery distribution is sampled
  rc = launch_lm_head_recover_rows(d, p->lm_rec, A.recover_row, hidden, hidden_rows, weight, hidden_dim, vocab, d.batch, p->num_sms,
                                   rec_logits, (long long)rec_ld, s, err);
  if (rc != 0) return fail(rc, "as_accept_lm_head_sampled: " + err);
  AS_CUDA(launch_recover(d, A, s));
  p->launches += 8;
  return AS_OK;
}

int as_accept_seeded(as_plan_t* p, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
                     const float* draft_probs, const float* temperature, const uint64_t* rng_state,
                     int32_t* accept_len, int32_t* out_tokens, void* stream) {
  if (!temperature || !rng_state) return fail(AS_ERR_INVALID_ARG, "as_accept_seeded: temperature and rng_state are required");
  return accept_impl(p, logits, ld, vocab, draft_tokens, draft_probs, temperature, nullptr, nullptr, rng_state, accept_len,
                     out_tokens, stream);
}

}  // extern "C"

namespace {
int accept_impl(as_plan_t* p, const float* logits, int64_t ld, int vocab, const int32_t* draft_tokens,
                const float* draft_probs, const float* temperature, const float* u, const float* w,
                const uint64_t* rng, int32_t* accept_len, int32_t* out_tokens, void* stream) {
  if (!p || !logits || !accept_len || !out_tokens) return fail(AS_ERR_INVALID_ARG, "as_accept: null pointer");
  if (!p->planned) return fail(AS_ERR_INVALID_ARG, "as_accept: as_plan() has not been called for this step");
  if (vocab < 1 || ld < vocab) return fail(AS_ERR_INVALID_ARG, "as_accept: need 1 <= vocab <= ld");
  if (p->total_d > 0 && !draft_tokens) return fail(AS_ERR_INVALID_ARG, "as_accept: draft_tokens is null");
  if (p->batch == 0) return AS_OK;
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_accept: cannot select the plan's device");
  AcceptArgs A;
  A.logits = logits;
  A.ld = ld;
  A.vocab = vocab;
  A.draft_tokens = draft_tokens;
  A.draft_probs = draft_probs;
  A.temperature = temperature;
  A.u = u;
  A.w = w;
  A.rng = rng;
  A.accept_len = accept_len;
  A.out_tokens = out_tokens;
  A.row_part = reinterpret_cast<float4*>(p->ws + p->off_row_part);
  A.row_final = reinterpret_cast<float4*>(p->ws + p->off_row_final);
  A.row_ticket = reinterpret_cast<int32_t*>(p->ws + p->off_row_ticket);
  int chunk = 16384;                         // 64 KB of logits per CTA
  while ((vocab + chunk - 1) / chunk > p->accept_chunks_max) chunk *= 2;
  A.chunk_elems = chunk;
  A.chunks = (vocab + chunk - 1) / chunk;
  A.recover_row = reinterpret_cast<int32_t*>(p->ws + p->off_recover);
  A.rec_cells = reinterpret_cast<double*>(p->ws + p->off_rec_cells);
  int cell = 512;                            // (a cell costs its warp two fp64 reductions: few, large cells)
  while ((vocab + cell - 1) / cell > p->accept_cells_max) cell *= 2;
  A.cell_elems = cell;                       // a power of two below the chunk size, so it divides it
  A.cells = (vocab + cell - 1) / cell;
  AS_CUDA(launch_accept(dev_plan(p), A, static_cast<cudaStream_t>(stream)));
  p->launches += temperature ? 4 : 2;
  return AS_OK;
}
}  // namespace

extern "C" {

int as_kv_commit(as_plan_t* p, const int32_t* accept_len, int32_t* seq_lens, int32_t* block_table, int32_t* freed,
                 int32_t* freed_count, int flags, void* k_pool, void* v_pool, void* stream) {
  if (!p || !accept_len || !seq_lens || !block_table || !freed || !freed_count)
    return fail(AS_ERR_INVALID_ARG, "as_kv_commit: null pointer");
  if (!p->planned) return fail(AS_ERR_INVALID_ARG, "as_kv_commit: as_plan() has not been called for this step");
  if ((flags & ~AS_COMMIT_SCRUB) != 0) return fail(AS_ERR_INVALID_ARG, "as_kv_commit: unknown flag");
  if ((flags & AS_COMMIT_SCRUB) && (!k_pool || !v_pool)) return fail(AS_ERR_INVALID_ARG, "as_kv_commit: scrub needs the pools");
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_kv_commit: cannot select the plan's device");
  AS_CUDA(launch_commit(dev_plan(p), accept_len, seq_lens, block_table, freed, freed_count, flags & AS_COMMIT_SCRUB,
                        static_cast<__nv_bfloat16*>(k_pool), static_cast<__nv_bfloat16*>(v_pool),
                        reinterpret_cast<int32_t*>(p->ws + p->off_commit_counts), static_cast<cudaStream_t>(stream)));
  p->planned = false;          // lengths and tables changed: the next step needs a new plan
  p->launches += 1;
  return AS_OK;
}

int as_plan_check(as_plan_t* p, uint32_t* flags, void* stream) {
  if (!p) return fail(AS_ERR_INVALID_ARG, "as_plan_check: null plan");
  if (!p->ws) return fail(AS_ERR_WORKSPACE, "as_plan_check: no workspace bound");
  DeviceGuard guard(p->device);
  if (!guard.ok) return fail(AS_ERR_CUDA, "as_plan_check: cannot select the plan's device");
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint32_t word = 0;
  AS_CUDA(cudaMemcpyAsync(&word, p->ws + p->off_status, sizeof word, cudaMemcpyDeviceToHost, s));
  AS_CUDA(cudaMemsetAsync(p->ws + p->off_status, 0, sizeof word, s));
  AS_CUDA(cudaStreamSynchronize(s));
  if (flags) *flags = word;
  if (word & kFlagWaitCap) return fail(AS_ERR_TIMEOUT, "as_plan_check: a bounded device-side wait ran out");
  if (word) return fail(AS_ERR_DEVICE_FLAG, "as_plan_check: device status word is non-zero");
  return AS_OK;
}

int as_plan_stats(const as_plan_t* p, int kind, int* num_ctas, int* num_items, int* num_merges, int* impl) {
  if (!p || kind < 0 || kind >= p->num_kinds) return fail(AS_ERR_INVALID_ARG, "as_plan_stats: bad argument");
  if (num_ctas) *num_ctas = p->step[kind].num_ctas;
  if (num_items) *num_items = p->step[kind].num_items;
  if (num_merges) *num_merges = p->step[kind].num_merges;
  if (impl) *impl = p->step[kind].impl;
  return AS_OK;
}

int as_plan_set_profile_events(as_plan_t* p, void* begin, void* end) {
  if (!p || ((begin == nullptr) != (end == nullptr))) return fail(AS_ERR_INVALID_ARG, "as_plan_set_profile_events: bad argument");
  p->prof_begin = static_cast<cudaEvent_t>(begin);
  p->prof_end = static_cast<cudaEvent_t>(end);
  return AS_OK;
}

int64_t as_plan_launch_count(const as_plan_t* p) { return p ? p->launches : 0; }

int as_plan_set_test_stall(as_plan_t* p, uint64_t wait_limit_ns, int stall_after_loads) {
  if (!p || stall_after_loads < -1) return fail(AS_ERR_INVALID_ARG, "as_plan_set_test_stall: bad argument");
  p->test_wait_limit_ns = wait_limit_ns;
  p->test_stall_after_loads = stall_after_loads;
  return AS_OK;
}

int as_plan_preview(const as_plan_t* p, int kind, int num_ctas, int batch, const int32_t* seq_lens,
                    const int32_t* draft_lens, int32_t* items_out, int cap_items, int32_t* cta_first_out,
                    int* num_items, int* num_ctas_out) {
  if (!p || kind < 0 || kind >= p->num_kinds || !seq_lens || !draft_lens || batch < 0 || batch > p->max_batch)
    return fail(AS_ERR_INVALID_ARG, "as_plan_preview: bad argument");
  for (int i = 0; i < batch; ++i)
    if (seq_lens[i] < 0 || draft_lens[i] < 0 || draft_lens[i] > p->max_draft)
      return fail(AS_ERR_INVALID_ARG, "as_plan_preview: seq_len < 0 or draft_len outside [0, max_draft]");
  const int impl = pick_impl(p, kind);
  if (impl < 0) return fail(AS_ERR_UNSUPPORTED, "as_plan_preview: shape not covered by the requested kernel");
  if (num_ctas <= 0) num_ctas = impl == AS_ATTN_TC ? p->num_sms : p->num_sms * p->simt_ctas_per_sm;
  std::vector<WorkItem> items;
  std::vector<int32_t> cta_first;
  std::vector<MergeSeg> merges;
  int kmax_step = 0;
  for (int i = 0; i < batch; ++i) kmax_step = std::max(kmax_step, (int)draft_lens[i]);
  int part_rows = 0;
  build_work(p, kind, impl, num_ctas, launch_rows(p, impl, p->fixed_launch ? p->max_draft : kmax_step), seq_lens, draft_lens, batch,
             nullptr, part_rows, items, cta_first, merges);
  if (items_out)
    for (size_t x = 0; x < items.size() && (int)x < cap_items; ++x) {
      const WorkItem& w = items[x];
      int32_t* o = items_out + 5 * x;
      o[0] = w.req; o[1] = w.kv_head; o[2] = w.key_begin; o[3] = w.key_end; o[4] = w.part_row;
    }
  if (cta_first_out) std::memcpy(cta_first_out, cta_first.data(), sizeof(int32_t) * cta_first.size());
  if (num_items) *num_items = (int)items.size();
  if (num_ctas_out) *num_ctas_out = num_ctas;
  return AS_OK;
}

}  // extern "C"
