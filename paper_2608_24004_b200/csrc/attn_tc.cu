// Verify attention on the 5th-generation tensor cores (tcgen05 + TMEM) with TMA-staged KV pages.
// Two kernels: this file's "keys on M" kernel for head_dim 128, and the "rows on M" kernel of attn_rows.inl
// (included below, sharing the helpers, the work items and the tensor maps) for head_dim 64.
//
// Shape of the problem: per (request, kv-head) pair there are only R = G * (k + 1) query rows (up to 128
// here) but thousands of keys, and every K/V byte is read exactly once.
// So the tile is laid out "keys on M": for a tile of 128 keys
//     S^T [128 keys x R]  = K_tile [128 x D] . Q^T [D x R]      (A = K from smem, B = Q from smem)
//     O^T [D x R]        += V_tile^T [D x 128] . P^T [128 x R]   (A = V from smem, MN-major; B = P^T)
// All 128 TMEM lanes carry real keys (no padding of the short row dimension up to M = 128), the
// page tile that TMA drops into shared memory is directly the A operand of both products, and a
// softmax thread owns one key (one TMEM lane) and walks the R columns.
//
// Online softmax without a per-tile row maximum: all 128 key-threads of a row use one shared
// reference m_ref[row]; it is raised (and O^T / the partial sums rescaled) only when some score
// exceeds it by more than 2^8, which the threads detect with one warp-wide OR, one shared-memory
// atomic and one rendezvous of their warpgroup per tile.  Row sums are per-thread partials over the
// bf16-rounded weights (exactly what enters the PV product), 16 registers per thread and slab,
// reduced in a fixed order once per work item.
//
// Warp roles (64 threads + 128 per softmax warpgroup, one CTA per SM, persistent over the plan's share of items):
//   warp 0      TMA producer: block-table lookup, one 5-d tensor-map copy per (page, kv-head, K|V) into a
//               ring of 128-key slots, completion on mbarriers
//   warp 1      allocates TMEM; one lane issues every tcgen05.mma and tcgen05.commit
//   warps 2..   softmax warpgroups (lane = key): one per 16-row slab of the query rows, at most five, each
//               walking up to two slabs per tile; they also stage Q and run the epilogue (lane =
//               head-dim index); a warpgroup owns its slabs' references outright
// Every mbarrier wait is bounded; on a timeout the CTA raises the status word, all roles leave
// their loops, in-flight copies are given time to land, TMEM is freed and the kernel returns.
#include <cuda.h>

#include <cstring>
#include <type_traits>

#include "attn_tc.cuh"
#include "tc_ptx.cuh"

namespace asv {
namespace {

constexpr int kTile = kTileKeys;                 // 128 keys per tile
constexpr float kRescaleThreshold = 8.f;         // log2 units
constexpr int kItemCache = 48;                   // work items of a CTA mirrored in shared memory

template <int D, int NPAD>
struct Smem {
  static constexpr int kSlabs = NPAD / 16;                    // 16-row slabs of the query-row dimension
  static constexpr int kGroups = kSlabs < 7 ? kSlabs : 7;     // softmax warpgroups: one per slab up to seven (960 threads)
  static constexpr int kSlabsPerGroup = (kSlabs + kGroups - 1) / kGroups;
  static constexpr int kThreads = 64 + 128 * kGroups + 32;      // K producer, issuer, softmax warpgroups, V producer
  static constexpr int kWarpProd2 = 2 + 4 * kGroups;
  // one ring slot: a 128-key K or V tile
  static constexpr int kSlotBytes = kTile * D * 2;
  static constexpr int kQBytes = NPAD * D * 2;
  static constexpr int kPBytes = NPAD * kTile * 2;
  // barriers (for the deepest ring), per-row tables, control block, item mirror: see the offsets below
  static constexpr int kSmallBytes = (2 * 8 + 14 + kGroups + 1) / 2 * 2 * 8 + NPAD * (4 + 4 + 4 + 16 + 4 + 8) + 64 + 256 + kItemCache * 32;
  // Q staging is double-buffered while it is small.  P staging is double-buffered whenever that still
  // leaves four K/V slots: with one P buffer the softmax of tile g+1 has to wait for the PV product of tile g.
  static constexpr int kQBufs = NPAD <= 64 ? 2 : 1;
  static constexpr int kFree = 232448 - 1024 - kQBufs * kQBytes - kSmallBytes;
  static constexpr int kPBufs = (kFree - 2 * kPBytes) / kSlotBytes >= 4 ? 2 : 1;
  static constexpr int kSlotsFit = (kFree - kPBufs * kPBytes) / kSlotBytes;
  static constexpr int kSlots = kSlotsFit > 8 ? 8 : kSlotsFit;   // ring of K / V slots (alternating K(g), V(g))
  static_assert(kSlots >= 3, "the K/V ring needs at least three slots");
  static constexpr int kOffQ = kSlots * kSlotBytes;
  static constexpr int kOffP = kOffQ + kQBufs * kQBytes;
  static constexpr int kOffBars = kOffP + kPBufs * kPBytes;
  static constexpr int kNumBars = (2 * kSlots + 14 + kGroups + 1) / 2 * 2;   // even, so the tables after the barriers stay 16-byte aligned
  static_assert((kNumBars * 8) % 16 == 0, "tables after the barriers must stay 16-byte aligned");
  static constexpr int kOffMref = kOffBars + kNumBars * 8;
  static constexpr int kOffAlpha = kOffMref + NPAD * 4;
  static constexpr int kOffWmax = kOffAlpha + NPAD * 4;       // per-row tile maxima (order-preserving ints)
  static constexpr int kOffLsum = kOffWmax + NPAD * 4;        // per slab [4 warps][16 rows] row-sum partials
  static constexpr int kOffInv = kOffLsum + 4 * NPAD * 4;     // per row: output scale
  static constexpr int kOffOff = kOffInv + NPAD * 4;          // per row: destination offset (8 bytes, -1 = none)
  static constexpr int kOffUnseen = kOffOff + NPAD * 8;
  static constexpr int kOffCtl = kOffUnseen + 64;
  static constexpr int kOffItems = kOffCtl + 256;             // this CTA's first kItemCache work items
  static constexpr int kTotal = kOffItems + kItemCache * 32;
  static_assert(kTotal - kOffBars <= kSmallBytes, "small tables outgrew their reservation");
  static constexpr uint32_t kTmemCols = 3 * NPAD <= 256 ? 256 : 512;   // S double buffer + O
  static_assert(3 * NPAD <= 512, "S double buffer and O must fit in TMEM");
};

struct ItemView {            // what each role needs to know about one work item
  int req, kv_head, key_begin, key_end, part_row, n, k, cu_q, tiles;
};
// Work item `it` of this CTA: from the shared-memory mirror when it is one of the first kItemCache
// (every role walks the same list, so none of them pays a global-memory round trip per item).
__device__ __forceinline__ ItemView view(const AttnArgs& A, const WorkItem* cache, int it_begin, int it) {
  const WorkItem w = (it - it_begin < kItemCache) ? cache[it - it_begin] : A.items[it];
  return ItemView{w.req, w.kv_head, w.key_begin, w.key_end, w.part_row, w.n, w.k, w.cu_q,
                  (w.key_end - w.key_begin + kTile - 1) / kTile};
}

template <int D, int NPAD>
__global__ void __launch_bounds__(Smem<D, NPAD>::kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, DevPlan P, AttnArgs A) {
  using L = Smem<D, NPAD>;
  constexpr int kSlots = L::kSlots;
  constexpr int NWG = L::kGroups;
  constexpr int SPW = L::kSlabsPerGroup;
  constexpr int kThreads = L::kThreads;
  constexpr int NQ = L::kQBufs, NP = L::kPBufs;
  constexpr int KSTEPS_S = D / 16;                      // tcgen05.mma K = 16 for bf16
  constexpr int KSTEPS_PV = kTile / 16;
  constexpr uint32_t SBO_KV = 2048;                     // 8-key group stride inside a slot
  // byte offset of the K / V atoms inside a slot: separate slots (0), or interleaved per 8-row group
  constexpr uint32_t TMEM_COLS = L::kTmemCols;
  static_assert(D == 128, "head_dim 128 (head_dim 64 runs the rows-on-M kernel)");

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + L::kOffBars;
  auto bar_slot_full = [&](int s) { return bars + 8u * s; };
  auto bar_slot_empty = [&](int s) { return bars + 8u * (kSlots + s); };
  const uint32_t b0 = bars + 8u * 2 * kSlots;
  auto bar_s_full = [&](int b) { return b0 + 8u * b; };
  auto bar_s_free = [&](int b) { return b0 + 8u * (2 + b); };
  auto bar_p_full = [&](int b) { return b0 + 8u * (4 + b); };
  auto bar_p_free = [&](int b) { return b0 + 8u * (6 + b); };
  auto bar_q_full = [&](int b) { return b0 + 8u * (8 + b); };
  auto bar_q_free = [&](int b) { return b0 + 8u * (10 + b); };
  const uint32_t bar_o_full = b0 + 8u * 12, bar_o_free = b0 + 8u * 13;
  auto bar_wg = [&](int w) { return b0 + 8u * (14 + w); };       // warpgroup-local rendezvous (bounded, unlike bar.sync)
  float* m_ref = reinterpret_cast<float*>(smem + L::kOffMref);
  float* alpha = reinterpret_cast<float*>(smem + L::kOffAlpha);
  int* wmax = reinterpret_cast<int*>(smem + L::kOffWmax);
  uint32_t* unseen = reinterpret_cast<uint32_t*>(smem + L::kOffUnseen);   // per slab: rows without a finite reference
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + L::kOffCtl);
  const WorkItem* item_cache = reinterpret_cast<const WorkItem*>(smem + L::kOffItems);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = P.Hq / P.Hkv;
  const int it_begin = A.cta_first[blockIdx.x], it_end = A.cta_first[blockIdx.x + 1];

  if (tid == 0) {
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(bar_slot_full(s), 1);
      mbar_init(bar_slot_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_s_full(b), 1);
      mbar_init(bar_s_free(b), 128 * NWG);
      mbar_init(bar_p_full(b), 128 * NWG);
      mbar_init(bar_p_free(b), 1);
      mbar_init(bar_q_full(b), 128 * NWG);
      mbar_init(bar_q_free(b), 1);
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, 128 * NWG);
    for (int w = 0; w < NWG; ++w) mbar_init(bar_wg(w), 128);
    ctl->abort = 0;
    ctl->tmem_base = 0;
    ctl->limit_ns = A.wait_limit_ns ? A.wait_limit_ns : kWaitLimitNs;
    for (int x = 0; x < 32; ++x) (&ctl->flags[0][0])[x] = 0;
    for (int x = 0; x < NPAD; ++x) wmax[x] = (int)0x807fffff;      // order-preserving image of -inf
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int x = tid; x < min(it_end - it_begin, kItemCache) * 2; x += kThreads)
    reinterpret_cast<uint4*>(smem + L::kOffItems)[x] = reinterpret_cast<const uint4*>(A.items + it_begin)[x];
  // Q and P staging start out as zeros so that padded rows / columns hold finite values
  for (int x = tid; x < (NQ * L::kQBytes + NP * L::kPBytes) / 16; x += kThreads)
    reinterpret_cast<uint4*>(smem + L::kOffQ)[x] = make_uint4(0, 0, 0, 0);
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctl->tmem_base;
  const uint32_t tmem_s0 = tmem, tmem_o = tmem + 2 * NPAD;

  if (warp == 0 || warp == L::kWarpProd2) {
    // ------------------------------------------------------------------ TMA producers
    // Two warps share the ring: warp 0 copies the K tiles (even slots of the running sequence K(0), V(0), K(1), ...),
    // the last warp the V tiles.  One warp issuing all sixteen copies of a tile pair, one lane after the other, reaches
    // 6.5 TB/s over the device with nothing else to do; two reach 6.9.  Page ids come 32 at a time (one coalesced
    // load of the request's block-table row: four tiles' worth at 16 keys a page), a chunk ahead of their use, so that
    // no pass of the loop waits for a global-memory round trip.
    const int which = warp == 0 ? 0 : 1;
    const CUtensorMap* map = which == 0 ? &kmap : &vmap;
    const int pages_per_tile = kTile / P.bs;
    const int tiles_per_chunk = 32 / pages_per_tile;
    const uint32_t page_bytes = (uint32_t)P.bs * D * 2;
    auto chunk_load = [&](const ItemView& v, int c) -> int {
      const int idx = c * 32 + lane;                       // page of the item's key range
      const int np_item = (v.key_end - v.key_begin + P.bs - 1) / P.bs;
      return idx < np_item ? __ldg(A.block_table + (size_t)v.req * P.max_blocks + v.key_begin / P.bs + idx) : -1;
    };
    uint32_t tile_idx = 0;                                 // running tile number of this CTA
    bool ok = it_begin < it_end;
    int it = it_begin;
    ItemView v = ok ? view(A, item_cache, it_begin, it_begin) : ItemView{};
    int ids = ok ? chunk_load(v, 0) : -1;
    while (ok) {
      const int nit = it + 1;
      const ItemView nv = nit < it_end ? view(A, item_cache, it_begin, nit) : ItemView{};
      const int nch = (v.tiles + tiles_per_chunk - 1) / tiles_per_chunk;
      for (int c = 0; c < nch && ok; ++c) {
        const int ids_next = c + 1 < nch ? chunk_load(v, c + 1) : (nit < it_end ? chunk_load(nv, 0) : -1);
        const int t_end = min(v.tiles, (c + 1) * tiles_per_chunk);
        for (int tile = c * tiles_per_chunk; tile < t_end; ++tile, ++tile_idx) {
          if (A.stall_after_loads >= 0 && (int)tile_idx >= A.stall_after_loads) { ok = false; break; }   // (test hook: the copies stop coming)
          const int kbase = v.key_begin + tile * kTile;
          const int npages = min(pages_per_tile, (v.key_end - kbase + P.bs - 1) / P.bs);
          int page = __shfl_sync(0xffffffffu, ids, ((tile - c * tiles_per_chunk) * pages_per_tile + lane) & 31);
          if (lane >= npages) page = -1;
          if (lane < npages && (unsigned)page >= (unsigned)P.num_blocks) {
            atomicOr(P.status, kFlagBadPage);
            page = -1;
          }
          const int nvalid = __popc(__ballot_sync(0xffffffffu, page >= 0));
          const uint32_t load_idx = 2 * tile_idx + which;
          const int slot = load_idx % kSlots;
          const uint32_t par = ((load_idx / kSlots) & 1u) ^ 1u;
          int good = 1;
          if (lane == 0) good = mbar_wait_c(bar_slot_empty(slot), par, ctl, P.status, 0) ? 1 : 0;
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
          if (lane == 0) mbar_arrive_expect_tx(bar_slot_full(slot), (uint32_t)nvalid * page_bytes);
          __syncwarp();
          if (page >= 0)
            tma_load_5d(sbase + slot * L::kSlotBytes + lane * page_bytes, map, bar_slot_full(slot), 0, 0, 0, 0,
                        page * P.Hkv + v.kv_head);
        }
        ids = ids_next;
      }
      if (nit >= it_end) break;
      it = nit;
      v = nv;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      // N of both products is the instance's NPAD for every item (an N fitted to the item's own row count
      // was measured 2-3 % slower).  S^T: M = 128 keys;  O^T: M = head_dim (128, or 64 on half the lanes)
      constexpr uint32_t idesc_s = instr_desc(kTile, NPAD, false, false);
      constexpr uint32_t idesc_pv = instr_desc(D, NPAD, true, true);
      uint32_t g = 0;                          // global tile counter of this CTA
      bool ok = true;
      bool have_prev = false, prev_first = false, prev_last = false;
      uint32_t prev_item = 0;
      auto issue_pv = [&](uint32_t h, bool first, bool last, uint32_t item_idx) -> bool {
        const uint32_t li = 2 * h + 1;
        const int vslot = li % kSlots;
        if (!mbar_wait_c(bar_slot_full(vslot), (li / kSlots) & 1u, ctl, P.status, 1)) return false;
        const int pbuf = h % NP;
        if (!mbar_wait_c(bar_p_full(pbuf), (h / NP) & 1u, ctl, P.status, 2)) return false;
        if (first && !mbar_wait_c(bar_o_free, (item_idx & 1u) ^ 1u, ctl, P.status, 3)) return false;
        tc_fence_after();
        const uint32_t vaddr = sbase + vslot * L::kSlotBytes;
        const uint32_t paddr = sbase + L::kOffP + pbuf * L::kPBytes;
        // A = V^T (MN-major, 128-byte swizzle): 16 keys per step = two 8-key groups; B = P^T (MN-major, no swizzle)
        const uint32_t v_lo = desc_lo(vaddr, 1024), p_lo = desc_lo(paddr, 128);
#pragma unroll
        for (int kk = 0; kk < KSTEPS_PV; ++kk)
          umma_bf16(tmem_o, v_lo + kk * (2 * SBO_KV / 16), desc_hi(SBO_KV, 2), p_lo + kk * (256 / 16), desc_hi(kTile * 16, 0),
                    idesc_pv, !(first && kk == 0));
        umma_commit(bar_slot_empty(vslot));
        umma_commit(bar_p_free(pbuf));
        if (last) umma_commit(bar_o_full);
        return true;
      };
      uint32_t item_idx = 0;
      for (int it = it_begin; it < it_end && ok; ++it, ++item_idx) {
        const ItemView v = view(A, item_cache, it_begin, it);
        const int qbuf = item_idx % NQ;
        if (!mbar_wait_c(bar_q_full(qbuf), (item_idx / NQ) & 1u, ctl, P.status, 4)) { ok = false; break; }
        const uint32_t q_lo = desc_lo(sbase + L::kOffQ + qbuf * L::kQBytes, 16);
        for (int tile = 0; tile < v.tiles; ++tile, ++g) {
          const uint32_t li = 2 * g;
          const int kslot = li % kSlots;
          if (!mbar_wait_c(bar_slot_full(kslot), (li / kSlots) & 1u, ctl, P.status, 5)) { ok = false; break; }
          const int sbuf = g & 1;
          if (!mbar_wait_c(bar_s_free(sbuf), ((g >> 1) & 1u) ^ 1u, ctl, P.status, 6)) { ok = false; break; }
          tc_fence_after();
          const uint32_t kaddr = sbase + kslot * L::kSlotBytes;
          // A = K tile, B = Q (both K-major, 128-byte swizzle): 32 bytes per step inside a 64-element atom
          const uint32_t k_lo = desc_lo(kaddr, 16);
#pragma unroll
          for (int kk = 0; kk < KSTEPS_S; ++kk)
            umma_bf16(tmem_s0 + sbuf * NPAD, k_lo + ((kk / 4) * 1024 + (kk % 4) * 32) / 16, desc_hi(SBO_KV, 2),
                      q_lo + ((kk / 4) * (NPAD * 128) + (kk % 4) * 32) / 16, desc_hi(1024, 2), idesc_s, kk > 0);
          umma_commit(bar_slot_empty(kslot));
          umma_commit(bar_s_full(sbuf));
          if (tile == v.tiles - 1) umma_commit(bar_q_free(qbuf));
          if (have_prev && !issue_pv(g - 1, prev_first, prev_last, prev_item)) { ok = false; break; }
          have_prev = true;
          prev_first = (tile == 0);
          prev_last = (tile == v.tiles - 1);
          prev_item = item_idx;
        }
      }
      if (ok && have_prev) issue_pv(g - 1, prev_first, prev_last, prev_item);
    }
  } else if (warp < L::kWarpProd2) {
    // ------------------------------------------------------------------ softmax + epilogue
    // Warpgroup wg owns the 16-row slabs wg, wg + NWG, ... (rows = TMEM columns): their references,
    // their weights, their slice of O^T and of the output.  Warpgroups never synchronise with each other.
    const int wg = (warp - 2) >> 2;                       // 0..NWG-1
    const int st = (tid - 64) & 127;                      // thread within the warpgroup
    const int quarter = warp & 3;                         // TMEM lanes this warp may touch
    const int kt = quarter * 32 + lane;                   // key within the tile
    // head-dim index of this thread's TMEM lane in O^T: lane itself for M = 128; for M = 64 rows
    // 16q..16q+15 sit in the first 16 lanes of quarter q and the other lanes hold nothing
    const int dd = kt;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const float scale = A.scale_log2;
    const int W = A.window;
    float* lsum_all = reinterpret_cast<float*>(smem + L::kOffLsum);
    float* inv_all = reinterpret_cast<float*>(smem + L::kOffInv);
    long long* off_all = reinterpret_cast<long long*>(smem + L::kOffOff);
    uint32_t wg_phase = 0;
    // rendezvous of the 128 threads of this warpgroup; false if the wait ran out or the CTA is aborting
    auto wg_bar = [&]() -> bool {
      mbar_arrive(bar_wg(wg));
      const bool r = mbar_wait_c(bar_wg(wg), wg_phase, ctl, P.status, 7);
      wg_phase ^= 1u;
      return r;
    };
    bool ok = true;
    uint32_t g = 0;

    auto load_q = [&](const ItemView& v, uint32_t item_idx) -> bool {
      const int qbuf = item_idx % NQ;
      if (!mbar_wait_c(bar_q_free(qbuf), ((item_idx / NQ) & 1u) ^ 1u, ctl, P.status, 8)) return false;
      unsigned char* qs = smem + L::kOffQ + qbuf * L::kQBytes;
      const int R = G * (v.k + 1);
      constexpr int CPR = D / 8;                          // 16-byte chunks per row
#pragma unroll
      for (int i = 0; i < SPW; ++i) {                     // every warpgroup stages the rows of its own slabs
        const int col0 = (wg + i * NWG) * 16;
        // (a slab that the item fills only in part gets zeros for the rest: what an earlier, wider item left there
        // would otherwise vote on the references with scores that depend on bytes past the request's last key)
        const int rows_here = col0 < R ? 16 : 0;
        for (int x = st; x < rows_here * CPR; x += 128) {
          const int row = col0 + x / CPR, ch = x % CPR;
          const uint4 val = row < R ? *reinterpret_cast<const uint4*>(
              A.q + ((size_t)(v.cu_q + row / G) * P.Hq + v.kv_head * G + row % G) * D + ch * 8) : make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(qs + (ch / 8) * (NPAD * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) = val;
        }
      }
      fence_proxy_async();
      mbar_arrive(bar_q_full(qbuf));
      return true;
    };

    // The same staging without waiting for the data: asynchronous 16-byte copies now, completion and the
    // arrival on q_full one tile later (the queries of the next item are not needed before this item's last
    // tiles, and a synchronous copy cost every item a global-memory round trip on the softmax threads).
    auto load_q_issue = [&](const ItemView& v, uint32_t item_idx) -> bool {
      const int qbuf = item_idx % NQ;
      if (!mbar_wait_c(bar_q_free(qbuf), ((item_idx / NQ) & 1u) ^ 1u, ctl, P.status, 8)) return false;
      const uint32_t qs = sbase + L::kOffQ + qbuf * L::kQBytes;
      const int R = G * (v.k + 1);
      constexpr int CPR = D / 8;
#pragma unroll
      for (int i = 0; i < SPW; ++i) {
        const int col0 = (wg + i * NWG) * 16;
        const int rows_here = col0 < R ? 16 : 0;            // (zeros behind the item's last row: see load_q)
        for (int x = st; x < rows_here * CPR; x += 128) {
          const int row = col0 + x / CPR, ch = x % CPR;
          const uint32_t dst = qs + (ch / 8) * (NPAD * 128) + row * 128 + (((ch & 7) ^ (row & 7)) << 4);
          if (row < R) {
            const __nv_bfloat16* src = A.q + ((size_t)(v.cu_q + row / G) * P.Hq + v.kv_head * G + row % G) * D + ch * 8;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
          } else {
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
          }
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      return true;
    };
    auto load_q_finish = [&](uint32_t item_idx) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async();
      mbar_arrive(bar_q_full(item_idx % NQ));
    };
    // (measured: with a single softmax warpgroup the asynchronous form is 8 % slower on short ragged contexts and
    // no faster elsewhere, with two or more it is 5-18 % faster on short contexts)
    constexpr bool ASYNC_Q = NWG >= 2;
    bool q_pending = false;                               // copies of the next item's queries are in flight

    if (it_begin < it_end) ok = load_q(view(A, item_cache, it_begin, it_begin), 0);
    uint32_t item_idx = 0;
    for (int it = it_begin; it < it_end && ok; ++it, ++item_idx) {
      const ItemView v = view(A, item_cache, it_begin, it);
      const int R = G * (v.k + 1);
      float l_part[SPW][16];                              // this thread's share of its slabs' row sums
#pragma unroll
      for (int i = 0; i < SPW; ++i)
#pragma unroll
        for (int e = 0; e < 16; ++e) l_part[i][e] = 0.f;
      // first position whose keys some row of the item cannot see from below (sliding window)
      const int lo_edge = W > 0 ? v.n + v.k - W + 1 : 0;

      for (int tile = 0; tile < v.tiles && ok; ++tile, ++g) {
        const int kbase = v.key_begin + tile * kTile;
        const int t = kbase + kt;
        const int sbuf = g & 1, pbuf = g % NP;
        if (!mbar_wait_c(bar_s_full(sbuf), (g >> 1) & 1u, ctl, P.status, 9)) { ok = false; break; }
        tc_fence_after();
        const bool mask_hi = kbase + kTile - 1 > v.n;      // tile holds keys that some row must not see yet
        const bool mask_lo = W > 0 && kbase < lo_edge;     // ... or no longer sees
        // raw scores q.k of this thread's key for the 16 rows of a slab, -inf where a row may not see the key
        auto scores = [&](int col0, float* y) {
          tmem_ld16(tmem_s0 + sbuf * NPAD + lane_addr + col0, y);
          tmem_wait_ld();
          if (mask_hi || mask_lo) {
            // row col0 + e belongs to draft position (col0 + e) / G and sees keys n + pos - W + 1 .. n + pos
            int jj = col0 / G, rem = col0 - jj * G;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              if (t > v.n + jj || (W > 0 && t < v.n + jj - W + 1) || t >= v.key_end) y[e] = -INFINITY;
              if (++rem == G) {
                rem = 0;
                ++jj;
              }
            }
          }
        };
        // weights P^T[key][row] = 2^(score - reference) in bf16 (the B operand of the PV product) for one slab.
        // sign = +1: write them and add them to the row-sum partials; sign = -1: take the same weights out of the
        // partials again (their references are about to move).  Returns the rows whose score outgrew the reference.
        auto weights = [&](int col0, const float* y, float* lp, float sign) -> uint32_t {
          unsigned char* ps = smem + L::kOffP + pbuf * L::kPBytes + (kt >> 3) * 128 + (kt & 7) * 16 + (col0 >> 3) * (kTile * 16);
          const bool careful = unseen[col0 >> 4] != 0;     // some row of the slab has no finite reference yet
          float dmax = -INFINITY;
          uint32_t fb = 0;
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const float4 ma = *reinterpret_cast<const float4*>(m_ref + col0 + h * 8);
            const float4 mb = *reinterpret_cast<const float4*>(m_ref + col0 + h * 8 + 4);
            const float mr[8] = {ma.x, ma.y, ma.z, ma.w, mb.x, mb.y, mb.z, mb.w};
            uint32_t packed[4];
#pragma unroll
            for (int e = 0; e < 8; e += 2) {
              float p0, p1;
              if (!careful) {
                // one FMA gives score * scale - reference; exp2(-inf) = 0 takes care of masked keys
                const float d0 = fmaf(y[h * 8 + e], scale, -mr[e]), d1 = fmaf(y[h * 8 + e + 1], scale, -mr[e + 1]);
                dmax = fmaxf(dmax, fmaxf(d0, d1));
                p0 = exp2f(d0);
                p1 = exp2f(d1);
              } else {
                // a row that has seen no key yet (reference -inf) gets weight 0 and is flagged as soon as it sees
                // one; the redo pass then computes its weights against a finite reference
                const float y0 = y[h * 8 + e] * scale, y1 = y[h * 8 + e + 1] * scale;
                if (y0 > mr[e] + kRescaleThreshold || y1 > mr[e + 1] + kRescaleThreshold) fb = 1;
                p0 = (y0 == -INFINITY || mr[e] == -INFINITY) ? 0.f : exp2f(y0 - mr[e]);
                p1 = (y1 == -INFINITY || mr[e + 1] == -INFINITY) ? 0.f : exp2f(y1 - mr[e + 1]);
              }
              lp[h * 8 + e] = fmaf(sign, p0, lp[h * 8 + e]);
              lp[h * 8 + e + 1] = fmaf(sign, p1, lp[h * 8 + e + 1]);
              if (sign < 0.f) {
                // a weight that overflowed cannot be taken back out (inf - inf); its reference is about to rise by
                // 2^120 or more, which leaves nothing of the old partial sum anyway
                if (!(fabsf(lp[h * 8 + e]) < INFINITY)) lp[h * 8 + e] = 0.f;
                if (!(fabsf(lp[h * 8 + e + 1]) < INFINITY)) lp[h * 8 + e + 1] = 0.f;
              }
              const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
              packed[e >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
            }
            if (sign > 0.f)
              *reinterpret_cast<uint4*>(ps + h * (kTile * 16)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
          }
          return fb | (dmax > kRescaleThreshold ? 1u : 0u);
        };
        // tile maxima of one slab's rows into wmax (order-preserving ints, one atomic per row and warp)
        auto maxima = [&](int col0, const float* y) {
          int mykey = (int)0x807fffff;
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const int bits = __float_as_int(y[e] * scale);
            const int key = __reduce_max_sync(0xffffffffu, bits ^ ((bits >> 31) & 0x7fffffff));
            if (lane == e) mykey = key;
          }
          if (lane < 16) atomicMax(&wmax[col0 + lane], mykey);
        };
        // new references for the slabs in `mask` (bit i = this group's i-th slab): thread st handles row st
        auto raise_refs = [&](uint32_t mask) {
          if (st < 16 * SPW && ((mask >> (st >> 4)) & 1u)) {
            const int slab = wg + (st >> 4) * NWG, col = slab * 16 + (st & 15);
            const int key = wmax[col];
            const float mx = __int_as_float(key ^ ((key >> 31) & 0x7fffffff));
            const float mo = tile == 0 ? -INFINITY : m_ref[col];
            const float mnew = fmaxf(mo, mx);
            alpha[col] = mo == -INFINITY ? 0.f : exp2f(mo - mnew);
            m_ref[col] = mnew;
            wmax[col] = (int)0x807fffff;
            // rows of the slab that still have no finite reference (bit per row); the 16 threads of a
            // slab are the lower or upper half of one warp
            const unsigned half = __ballot_sync(0xffffu << (st & 16), mnew == -INFINITY) >> (st & 16) & 0xffffu;
            if ((st & 15) == 0) unseen[slab] = half;
          }
        };

        // the P buffer of this tile becomes writable when the PV product that last read it is done; the
        // first slab's scores are fetched before waiting for that
        bool p_writable = false;
        auto wait_p = [&]() -> bool {
          if (p_writable) return true;
          p_writable = true;
          return mbar_wait_c(bar_p_free(pbuf), ((g / NP) & 1u) ^ 1u, ctl, P.status, 10);
        };
        uint32_t redo = 0;                                  // slabs (bit i) whose references must move
        if (tile == 0) {
          // an item's first tile defines the references: maxima first, then the weights
#pragma unroll
          for (int i = 0; i < SPW; ++i) {
            const int col0 = (wg + i * NWG) * 16;
            if (col0 < R) {
              float y[16];
              scores(col0, y);
              maxima(col0, y);
              redo |= 1u << i;
            }
          }
        } else {
          // weights against the current references; flag the slabs in which a score outgrew its reference
          uint32_t mine = 0;
#pragma unroll
          for (int i = 0; i < SPW; ++i) {
            const int col0 = (wg + i * NWG) * 16;
            if (col0 < R) {
              float y[16];
              scores(col0, y);
              if (!wait_p()) ok = false;
              if (weights(col0, y, l_part[i], 1.f)) mine |= 1u << i;
            }
          }
          if (wg * 16 < R) {                                // groups without rows have nothing to agree on
            mine = __reduce_or_sync(0xffffffffu, mine);
            uint32_t* fl = &ctl->flags[wg][0];
            const int fs = g % 3;
            if (lane == 0 && mine) atomicOr(&fl[fs], mine);
            if (st == 0) fl[(g + 1) % 3] = 0;
            if (!wg_bar()) { ok = false; break; }
            redo = fl[fs];
            if (redo) {
              // rare: take the optimistic weights back out and collect the tile maxima of those slabs
#pragma unroll
              for (int i = 0; i < SPW; ++i) {
                if ((redo >> i) & 1u) {
                  const int col0 = (wg + i * NWG) * 16;
                  float y[16];
                  scores(col0, y);
                  weights(col0, y, l_part[i], -1.f);
                  maxima(col0, y);
                }
              }
            }
          }
        }
        if (!ok) break;
        if (redo) {
          if (!wait_p()) { ok = false; break; }
          if (!wg_bar()) { ok = false; break; }
          raise_refs(redo);
          if (!wg_bar()) { ok = false; break; }
          if (tile > 0) {
            // O^T holds the products up to the previous tile: wait for them, rescale it and the row sums
            if (!mbar_wait_c(bar_p_free((g - 1) % NP), ((g - 1) / NP) & 1u, ctl, P.status, 11)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int i = 0; i < SPW; ++i) {
              if ((redo >> i) & 1u) {
                const int col0 = (wg + i * NWG) * 16;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                  float o[8];
                  tmem_ld8(tmem_o + lane_addr + col0 + c * 8, o);
                  tmem_wait_ld();
#pragma unroll
                  for (int e = 0; e < 8; ++e) {
                    const float a = alpha[col0 + c * 8 + e];
                    o[e] *= a;
                    l_part[i][c * 8 + e] *= a;
                  }
                  tmem_st8(tmem_o + lane_addr + col0 + c * 8, o);
                }
              }
            }
            tmem_wait_st();
          }
#pragma unroll
          for (int i = 0; i < SPW; ++i) {
            if ((redo >> i) & 1u) {
              const int col0 = (wg + i * NWG) * 16;
              float y[16];
              scores(col0, y);
              weights(col0, y, l_part[i], 1.f);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(bar_s_free(sbuf));
        if (wg == 0 && mask_hi && t >= v.key_end) {
          // keys past the end of the request: their V rows (page tail or a slot row that no copy
          // touched) may hold anything, and 0 * NaN would poison O^T.  Zero them before the product.
          const uint32_t li = 2 * g + 1;
          const int vslot = li % kSlots;
          if (mbar_wait_c(bar_slot_full(vslot), (li / kSlots) & 1u, ctl, P.status, 12)) {
            unsigned char* vr = smem + vslot * L::kSlotBytes + (kt >> 3) * SBO_KV + (kt & 7) * 128;
#pragma unroll
            for (int h = 0; h < D / 64; ++h)
#pragma unroll
              for (int x = 0; x < 8; ++x) *reinterpret_cast<uint4*>(vr + h * 1024 + x * 16) = make_uint4(0, 0, 0, 0);
          }
        }
        // every thread, also one whose warpgroup has no rows in this item, may only announce P(g) once the
        // product that last read the buffer is done: otherwise its arrival could land in the previous phase
        if (!wait_p()) { ok = false; break; }
        fence_proxy_async();
        mbar_arrive(bar_p_full(pbuf));
        // with two Q buffers the next item's queries are staged early, so its first QK product never waits
        if (NQ == 2 && !ASYNC_Q) {
          if (tile == 0 && it + 1 < it_end && !load_q(view(A, item_cache, it_begin, it + 1), item_idx + 1)) { ok = false; break; }
        } else if (NQ == 2) {
          if (q_pending) {
            load_q_finish(item_idx + 1);
            q_pending = false;
          }
          if (tile == 0 && it + 1 < it_end) {
            if (!load_q_issue(view(A, item_cache, it_begin, it + 1), item_idx + 1)) { ok = false; break; }
            q_pending = true;
          }
        }
      }
      if (!ok) break;
      if (q_pending) {                                    // an item of a single tile
        load_q_finish(item_idx + 1);
        q_pending = false;
      }
      // with one Q buffer they can only follow the item's last QK product
      // (synchronously: the issuing thread needs them for the next item's first QK product, which it issues
      // before this item's last PV product, and the epilogue below waits for that product)
      if (NQ == 1 && it + 1 < it_end && !load_q(view(A, item_cache, it_begin, it + 1), item_idx + 1)) { ok = false; break; }

      // ---- epilogue: O^T (lane = head-dim index) to the output or the partial buffers ----
      if (!mbar_wait_c(bar_o_full, item_idx & 1u, ctl, P.status, 13)) { ok = false; break; }
      tc_fence_after();
      if (wg * 16 < R) {
        // row sums: a fixed-order butterfly leaves the warp total of row r of a slab in lanes 2r and 2r + 1
#pragma unroll
        for (int i = 0; i < SPW; ++i) {
          const int slab = wg + i * NWG;
          if (slab * 16 < R) {
            float v8[8], v4[4], v2[2], v1;
            {
              const bool hi = lane & 16;
#pragma unroll
              for (int x = 0; x < 8; ++x) {
                const float give = hi ? l_part[i][x] : l_part[i][x + 8], mine = hi ? l_part[i][x + 8] : l_part[i][x];
                v8[x] = mine + __shfl_xor_sync(0xffffffffu, give, 16);
              }
            }
            {
              const bool hi = lane & 8;
#pragma unroll
              for (int x = 0; x < 4; ++x) {
                const float give = hi ? v8[x] : v8[x + 4], mine = hi ? v8[x + 4] : v8[x];
                v4[x] = mine + __shfl_xor_sync(0xffffffffu, give, 8);
              }
            }
            {
              const bool hi = lane & 4;
#pragma unroll
              for (int x = 0; x < 2; ++x) {
                const float give = hi ? v4[x] : v4[x + 2], mine = hi ? v4[x + 2] : v4[x];
                v2[x] = mine + __shfl_xor_sync(0xffffffffu, give, 4);
              }
            }
            {
              const bool hi = lane & 2;
              const float give = hi ? v2[0] : v2[1], mine = hi ? v2[1] : v2[0];
              v1 = mine + __shfl_xor_sync(0xffffffffu, give, 2);
            }
            v1 += __shfl_xor_sync(0xffffffffu, v1, 1);
            if (!(lane & 1)) lsum_all[slab * 64 + quarter * 16 + (lane >> 1)] = v1;
          }
        }
        if (!wg_bar()) { ok = false; break; }
        // a few threads turn the sums into what the stores need: per row a scale and a destination
        if (st < 16 * SPW) {
          const int slab = wg + (st >> 4) * NWG, e = st & 15, j = slab * 16 + e;
          if (slab * 16 < R) {
            long long off = -1;
            float inv = 0.f;
            if (j < R) {
              const float* ls = lsum_all + slab * 64;
              float l = (ls[e] + ls[16 + e]) + (ls[32 + e] + ls[48 + e]);
              float m = m_ref[j];
              if (v.part_row >= 0) {
                off = (long long)(v.part_row + j) * D;
                inv = 1.f;                                       // partials stay unnormalised
                A.part_ml[v.part_row + j] = make_float2(m, l);
              } else {
                const int pos = j / G, h = v.kv_head * G + (j - pos * G);
                float sc = 1.f;
                if (A.sinks) {
                  const float sk = A.sinks[h] * 1.4426950408889634f;
                  const float m2 = fmaxf(m, sk);
                  sc = exp2f(m - m2);
                  l = l * sc + exp2f(sk - m2);
                  m = m2;
                }
                const long long row = (long long)(v.cu_q + pos) * P.Hq + h;
                off = row * D;
                inv = sc / l;
                if (A.lse) A.lse[row] = (m + log2f(l)) * 0.6931471805599453f;
              }
            }
            inv_all[j] = inv;
            off_all[j] = off;
          }
        }
        if (!wg_bar()) { ok = false; break; }
        // (rolled loops: this runs once per item, and its size counts against the instruction cache)
#pragma unroll 1
        for (int i = 0; i < SPW; ++i) {
          const int col0 = (wg + i * NWG) * 16;
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
            if (col0 + c * 8 < R) {
              float o[8];
              tmem_ld8(tmem_o + lane_addr + col0 + c * 8, o);
              tmem_wait_ld();
              if (dd >= 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                  const long long off = off_all[col0 + c * 8 + e];
                  if (off >= 0) {
                    const float val = o[e] * inv_all[col0 + c * 8 + e];
                    if (v.part_row >= 0) A.part_o[off + dd] = val;
                    else A.out[off + dd] = __float2bfloat16_rn(val);
                  }
                }
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar_o_free);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (ctl->abort) {
    // a role gave up: let copies that are still in flight land before shared memory goes away
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

#include "attn_rows.inl"

// The pool [num_blocks, Hkv, bs, D] bf16 seen as a 5-d tensor (fastest first):
//   64 elements of a row | 8 rows of a group | D/64 halves of the row | bs/8 row groups | page*Hkv + head
// so that one box = one (page, head) tile, delivered as 1024-byte atoms (8 rows x 128 bytes,
// 128-byte swizzled) ordered [row group][row half]: the canonical shared-memory layout of a
// tcgen05 operand with an 8-row-group stride of (D/64)*1024 bytes.
bool encode_pool_map(void* map, const void* pool, int num_blocks, int Hkv, int bs, int D, std::string& err) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    err = "cuTensorMapEncodeTiled is not available from the driver";
    return false;
  }
  const cuuint64_t halves = (cuuint64_t)(D / 64);
  const cuuint64_t dims[5] = {64, 8, halves, (cuuint64_t)(bs / 8), (cuuint64_t)num_blocks * Hkv};
  const cuuint64_t strides[4] = {(cuuint64_t)D * 2, 128, (cuuint64_t)8 * D * 2, (cuuint64_t)bs * D * 2};
  const cuuint32_t box[5] = {64, 8, (cuuint32_t)halves, (cuuint32_t)(bs / 8), 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  const CUresult r = fn(reinterpret_cast<CUtensorMap*>(map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5,
                        const_cast<void*>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
    return false;
  }
  return true;
}

template <int D, int NPAD>
cudaError_t launch_instance(const CUtensorMap& km, const CUtensorMap& vm, const DevPlan& P, const AttnArgs& A,
                            cudaStream_t s) {
  const int smem = Smem<D, NPAD>::kTotal + 1024;
  // the opt-in to large dynamic shared memory is per device and costs a few microseconds: once is enough
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !opted_in[dev]) {
    e = cudaFuncSetAttribute(attn_tc_kernel<D, NPAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  attn_tc_kernel<D, NPAD><<<A.num_ctas, Smem<D, NPAD>::kThreads, smem, s>>>(km, vm, P, A);
  return cudaGetLastError();
}

// padded row counts the kernel is instantiated for
template <int D>
cudaError_t launch_for_rows(int rows, const CUtensorMap& km, const CUtensorMap& vm, const DevPlan& P, const AttnArgs& A,
                            cudaStream_t s) {
  if (rows <= 16) return launch_instance<D, 16>(km, vm, P, A, s);
  if (rows <= 32) return launch_instance<D, 32>(km, vm, P, A, s);
  if (rows <= 48) return launch_instance<D, 48>(km, vm, P, A, s);
  // (49..64 rows run the 80-row instance: five warpgroups of one slab each measured 12 % faster than four)
  if (rows <= 80) return launch_instance<D, 80>(km, vm, P, A, s);
  if (rows <= 96) return launch_instance<D, 96>(km, vm, P, A, s);
  if (rows <= 112) return launch_instance<D, 112>(km, vm, P, A, s);
  // (wider requests reach this kernel as row blocks of at most 96 rows: see plan_block_positions)
  return cudaErrorInvalidValue;
}

}  // namespace

// Which orientation runs a launch: head_dim 64 always takes the rows-on-M kernel (faster there at every row count,
// and its tile cost does not depend on the row count), head_dim 128 the keys-on-M instances.
bool attn_rows_on_m(int D, int rows) { return D == 64 && rows <= kMaxRows; }

bool attn_tc_supported(int Hq, int Hkv, int D, int bs, int max_draft, int window) {
  const int rows = (Hq / Hkv) * (max_draft + 1);
  (void)window;                                       // full attention and sliding windows are both covered
  if (bs != 16 && bs != 32 && bs != 64 && bs != 128) return false;
  // (head_dim 128: up to 128 rows per launch item; the planner cuts wider requests into row blocks by draft position)
  return (D == 128 && rows <= kMaxRows && Hq / Hkv <= kKeysOnMRows) || (D == 64 && rows <= kMaxRows);
}

int launch_attn_tc(const DevPlan& P, const AttnArgs& A, TcState& st, cudaStream_t s, std::string& err) {
  if (A.num_ctas == 0) return 0;
  AttnArgs B = A;
  TcState::Entry* en = nullptr;
  for (int x = 0; x < TcState::kEntries && !en; ++x)
    if (st.entry[x].k_pool == A.k_pool && st.entry[x].v_pool == A.v_pool) en = &st.entry[x];
  if (!en) {
    en = &st.entry[st.next];
    st.next = (st.next + 1) % TcState::kEntries;
    en->k_pool = en->v_pool = nullptr;
    if (!encode_pool_map(en->k_map, A.k_pool, P.num_blocks, P.Hkv, P.bs, P.D, err)) return 4;
    if (!encode_pool_map(en->v_map, A.v_pool, P.num_blocks, P.Hkv, P.bs, P.D, err)) return 4;
    en->k_pool = A.k_pool;
    en->v_pool = A.v_pool;
  }
  const CUtensorMap& km = *reinterpret_cast<const CUtensorMap*>(en->k_map);
  const CUtensorMap& vm = *reinterpret_cast<const CUtensorMap*>(en->v_map);
  // the instance is as wide as this step's longest draft needs, not as the plan's maximum allows
  const int rows = A.rows_step > 0 ? A.rows_step : (P.Hq / P.Hkv) * (P.max_draft + 1);
  const cudaError_t e = attn_rows_on_m(P.D, rows) ? launch_rows_instance(km, vm, P, B, s) : launch_for_rows<128>(rows, km, vm, P, B, s);
  if (e != cudaSuccess) {
    err = std::string("tensor-core attention launch: ") + cudaGetErrorString(e);
    return 4;
  }
  return 0;
}

}  // namespace asv
