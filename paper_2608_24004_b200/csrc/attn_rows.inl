// Verify attention with the query rows on M, for head_dim 64 (up to 256 rows per KV head, in blocks of 128).
// Included by attn_tc.cu after its PTX helpers; shares the planner's work items, the merge kernel and the status
// word with the keys-on-M kernel there.
//
// Why a second orientation.  With the keys on M a softmax thread owns one key and the rows of a tile are spread
// over warpgroups, which have to agree on every row's reference (a vote and a rendezvous per tile) and, beyond
// 80 rows, walk two or three 16-row slabs one after the other; at 136 rows a 128-key tile took about 4600
// cycles.  With the rows on M
//     S [128 rows x 128 keys] = Q [128 x D] . K_tile^T          (A = Q, B = K tile, both K-major)
//     O [128 rows x D]       += P [128 x 128 keys] . V_tile      (A = P from TMEM, written there by the row's own thread; B = V tile, MN-major)
// a softmax thread owns one query row (one TMEM lane): its running maximum, its row sum, its rescaling of O are
// its own business, nothing is voted on and nothing is reduced across threads.  Rows beyond the item's own count
// are computed and thrown away, so the cost of a tile depends on the row count only through the number of warps
// (blocks of 32 rows) that have rows at all.
//
// A tile's softmax is a serial chain (scores out of tensor memory, maximum, 128 exponentials, weights back in), and
// one warp per scheduler hides none of its latencies, so the tiles of an item are dealt to NS = 2 independent
// streams: warpgroup s takes the tiles whose running number is s modulo 2, with its own reference and row sum per
// row, its own S and P buffer and its OWN accumulator O_s in TMEM.  The streams never talk to each other during an
// item; the epilogue merges the (m, l, O_s) triples of a row like split-KV partials.
//
// Softmax of a tile, per thread: the weights 2^(score - reference) are computed against the row's reference as it
// stands, with no pass for the maximum.  A row whose weights of the tile add up to more than 2^9 keeps them (bf16 keeps
// their relative precision, O_s and the sum are fp32) and moves its reference afterwards: the sum at once, its row of
// O_s when the tile's PV product has completed.  Weights that may have overflowed (a score 2^96 above its reference)
// are recomputed from the queries and keys in global memory.  Only a stream's first tile of an item, a row that has
// seen no key yet and the masked edge tiles take the row maximum first.  The scores have left tensor memory for good
// a quarter of the way before the weights are finished; from then on the stream's S buffer is free (s_free) and the
// QK product of the stream's next tile runs under the rest of this tile's weights.
//
// K and V tiles travel in separate rings (3 + 8 slots of 16 KB), each filled by its own producer warp: a K tile is
// dead as soon as its QK product has completed, a V tile has to wait for the whole softmax of its tile, and in one
// ring of fused K+V slots the K halves would hold their shared memory for all that time; the depth of the prefetch,
// not the arithmetic, bounded the kernel then (five fused slots: 1590 cycles a tile, four: 1820).
//
// Warps (352 threads, one CTA per SM, persistent): 0..7 softmax (stream = warp / 4, TMEM lane quarter = warp % 4),
// 8 K producer, 9 V producer, 10 issues every tcgen05.mma from one lane.  That lane's own instructions are what bounds
// the kernel (measured: cycles added to it show one to one in the time of a tile, the softmax arithmetic taken out
// shows nothing): a product costs it 50 cycles when it has its scheduler to itself and more when softmax warps compete
// for the issue slots, a commit about a hundred, a turn of its loop a few hundred.  A warp's scheduler is its index modulo 4, and so is its TMEM lane
// quarter: warp 10 shares scheduler 2 with the softmax warps of lanes 64..95, and the block's rows 96..127, the ones
// that most items do not have, are mapped to those lanes (rows 64..95 to lanes 96..127).
// Every wait is bounded as in the other kernel.

template <int D, int NS>
struct RowsSmem {
  static_assert(D == 64, "rows-on-M kernel: head_dim 64");
  static constexpr int kRows = 128;
  static constexpr int kTileBytes = kTile * D * 2;             // one K or V tile
  static constexpr int kQBytes = kRows * D * 2;
  static constexpr int kPBufs = 2;                             // P buffers, in TMEM
  static constexpr int kMlBytes = 2 * NS * kRows * 8;          // per item parity, stream and row: (m, l)
  static constexpr int kSmallBytes = 40 * 8 + 256 + kMlBytes + kItemCache * 32;
  static constexpr int kQBufs = 2;                             // the next item's queries are staged during this one
  static constexpr int kFree = 232448 - 1024 - kQBufs * kQBytes - kSmallBytes;
  static constexpr int kKSlots = 3;
  static constexpr int kVSlots = kFree / kTileBytes - kKSlots > 8 ? 8 : kFree / kTileBytes - kKSlots;
  static_assert(kKSlots >= 2 && kVSlots >= 3, "rings too shallow");
  static_assert((kKSlots + kVSlots) * kTileBytes <= kFree, "rings do not fit");
  static constexpr int kOffK = 0;
  static constexpr int kOffV = kKSlots * kTileBytes;
  static constexpr int kOffQ = (kKSlots + kVSlots) * kTileBytes;
  static constexpr int kOffBars = kOffQ + kQBufs * kQBytes;
  static constexpr int kNumBars = 2 * (kKSlots + kVSlots) + 15;
  static_assert(kNumBars <= 40, "barrier reservation");
  static constexpr int kOffCtl = kOffBars + 40 * 8;
  static constexpr int kOffMl = kOffCtl + 256;
  static constexpr int kOffItems = kOffMl + kMlBytes;
  static constexpr int kTotal = kOffItems + kItemCache * 32;
  static constexpr int kWarpProdK = 4 * NS, kWarpProdV = 4 * NS + 1, kWarpMma = 4 * NS + 2, kWarps = 4 * NS + 3;
  static constexpr int kThreads = 32 * kWarps;
  // TMEM columns: S0, S1 (128 each), O_0 .. O_{NS-1} (D each), P0, P1 (64 each: 128 bf16 weights per row, two to a column)
  static constexpr uint32_t kTmemCols = 512;
  static_assert(2 * kTile + NS * D + kPBufs * (kTile / 2) <= 512, "S, O and P must fit in TMEM");
};

// packed pairs of floats in a 64-bit register, for fma / add .f32x2
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
constexpr float kRescaleStep = 8.f;              // a row's reference moves when a tile's maximum exceeds it by more than this (log2 units)
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

// tcgen05.mma with the A operand in tensor memory (row = lane, two bf16 per 32-bit column)
__device__ __forceinline__ void umma_bf16_ta(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                             bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"((uint32_t)accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16u(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(r[0])), "r"(__float_as_uint(r[1])), "r"(__float_as_uint(r[2])), "r"(__float_as_uint(r[3])),
      "r"(__float_as_uint(r[4])), "r"(__float_as_uint(r[5])), "r"(__float_as_uint(r[6])), "r"(__float_as_uint(r[7])),
      "r"(__float_as_uint(r[8])), "r"(__float_as_uint(r[9])), "r"(__float_as_uint(r[10])), "r"(__float_as_uint(r[11])),
      "r"(__float_as_uint(r[12])), "r"(__float_as_uint(r[13])), "r"(__float_as_uint(r[14])), "r"(__float_as_uint(r[15])),
      "r"(__float_as_uint(r[16])), "r"(__float_as_uint(r[17])), "r"(__float_as_uint(r[18])), "r"(__float_as_uint(r[19])),
      "r"(__float_as_uint(r[20])), "r"(__float_as_uint(r[21])), "r"(__float_as_uint(r[22])), "r"(__float_as_uint(r[23])),
      "r"(__float_as_uint(r[24])), "r"(__float_as_uint(r[25])), "r"(__float_as_uint(r[26])), "r"(__float_as_uint(r[27])),
      "r"(__float_as_uint(r[28])), "r"(__float_as_uint(r[29])), "r"(__float_as_uint(r[30])), "r"(__float_as_uint(r[31]))
      : "memory");
}

// Non-blocking look at four mbarriers: bit i = phase `parity i` of barrier i is complete.
__device__ __forceinline__ uint32_t mbar_test4(uint32_t bar0, uint32_t par0, uint32_t bar1, uint32_t par1, uint32_t bar2,
                                               uint32_t par2, uint32_t bar3, uint32_t par3) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p0, p1, p2, p3;\n\t.reg .u32 a, b, c, d;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p0, [%1], %2;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p1, [%3], %4;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p2, [%5], %6;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p3, [%7], %8;\n\t"
      "selp.u32 a, 1, 0, p0;\n\t"
      "selp.u32 b, 2, 0, p1;\n\t"
      "selp.u32 c, 4, 0, p2;\n\t"
      "selp.u32 d, 8, 0, p3;\n\t"
      "or.b32 a, a, b;\n\t"
      "or.b32 c, c, d;\n\t"
      "or.b32 %0, a, c;\n\t}"
      : "=r"(r)
      : "r"(bar0), "r"(par0), "r"(bar1), "r"(par1), "r"(bar2), "r"(par2), "r"(bar3), "r"(par3)
      : "memory");
  return r;
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

// An item with more than 128 query rows is walked once per block of 128 rows: the same keys again, the next rows.
// Every role derives the number of blocks from the item itself (G = query heads per kv head).
__device__ __forceinline__ int row_blocks_of(int G, const ItemView& v) { return (G * (v.k + 1) + 127) / 128; }

constexpr float kGrowSum = 512.f;                // a tile's weights of one row may add up to this before its reference moves
constexpr float kHugeSum = 7.9e28f;              // 2^96: beyond it (or NaN) the weights may have overflowed

// The softmax of one tile for one warp's rows WITHOUT the scores in tensor memory: every thread recomputes its row's
// 128 scores from the queries and keys in global memory (fp32 sums of the exact bf16 products), takes their maximum as
// the row's new reference, rescales its row of O_s and its sum, and writes the weights.  Slow (two passes of 128 dot
// products per thread) and rare: the optimistic pass of the kernel calls it when a row's weights overflowed, which
// takes a score more than 2^96 above the row's reference, long after the scores were released.  All 32 lanes call it.
template <int D>
__device__ __noinline__ void rows_tile_from_memory(const __nv_bfloat16* qrow, const __nv_bfloat16* k_pool, const int32_t* bt_row,
                                                   int bs, int Hkv, int head, int num_blocks, int kbase, int key_end, int hi_r,
                                                   int lo_r, float scale, uint32_t p_addr, uint32_t os_addr, bool own_first, float& m,
                                                   float& l) {
  float q[D];
  if (qrow) {
#pragma unroll
    for (int x = 0; x < D / 8; ++x) {
      const uint4 u = __ldg(reinterpret_cast<const uint4*>(qrow) + x);
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        q[8 * x + 2 * y] = __uint_as_float(w[y] << 16);
        q[8 * x + 2 * y + 1] = __uint_as_float(w[y] & 0xffff0000u);
      }
    }
  } else {
#pragma unroll
    for (int d = 0; d < D; ++d) q[d] = 0.f;
  }
  auto score = [&](int t) -> float {
    const int tt = kbase + t;
    if (tt >= key_end || tt > hi_r || tt < lo_r) return -INFINITY;
    const int page = __ldg(bt_row + tt / bs);
    if ((unsigned)page >= (unsigned)num_blocks) return -INFINITY;
    const uint4* kr = reinterpret_cast<const uint4*>(k_pool + ((size_t)(page * Hkv + head) * bs + tt % bs) * D);
    float acc = 0.f;
#pragma unroll
    for (int x = 0; x < D / 8; ++x) {
      const uint4 u = __ldg(kr + x);
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        acc = fmaf(q[8 * x + 2 * y], __uint_as_float(w[y] << 16), acc);
        acc = fmaf(q[8 * x + 2 * y + 1], __uint_as_float(w[y] & 0xffff0000u), acc);
      }
    }
    return acc;
  };
  float mx = -INFINITY;
#pragma unroll 1
  for (int t = 0; t < kTile; ++t) mx = fmaxf(mx, score(t));
  const float mnew = fmaxf(m, mx * scale);
  const float alpha = m == -INFINITY ? 0.f : exp2f(m - mnew);
  if (!own_first) {
    tc_fence_after();
#pragma unroll 1
    for (int c = 0; c < D / 32; ++c) {
      float o[32];
      tmem_ld32(os_addr + c * 32, o);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) o[e] *= alpha;
      tmem_st32(os_addr + c * 32, o);
    }
    tmem_wait_st();
  }
  l *= alpha;
  m = mnew;
  const float mref = m == -INFINITY ? 0.f : m;
  float lt = 0.f;
#pragma unroll 1
  for (int c = 0; c < kTile / 32; ++c) {
    uint32_t pk[16];
#pragma unroll 1
    for (int e = 0; e < 32; e += 2) {
      const float p0 = exp2f(fmaf(score(c * 32 + e), scale, -mref)), p1 = exp2f(fmaf(score(c * 32 + e + 1), scale, -mref));
      lt += p0 + p1;
      const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
      const uint32_t word = *reinterpret_cast<const uint32_t*>(&pb);
      // (pk is filled through a constant-index switch so that it stays in registers under the rolled loop)
#pragma unroll
      for (int x = 0; x < 16; ++x)
        if (x == (e >> 1)) pk[x] = word;
    }
    tmem_st16u(p_addr + c * 16, pk);
  }
  tmem_wait_st();
  l += lt;
}

template <int D, int NS>
__global__ void __launch_bounds__(RowsSmem<D, NS>::kThreads, 1)
attn_rows_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, DevPlan P, AttnArgs A) {
  using L = RowsSmem<D, NS>;
  constexpr int KS = L::kKSlots, VS = L::kVSlots;
  constexpr int kThreads = L::kThreads;
  constexpr int NP = L::kPBufs;
  constexpr int KSTEPS_S = D / 16;
  constexpr int KSTEPS_PV = kTile / 16;
  constexpr uint32_t SBO_KV = 1024;                     // 8-key group stride inside a K or V tile
  constexpr uint32_t TMEM_COLS = L::kTmemCols;

  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + L::kOffBars;
  auto bar_k_full = [&](int s) { return bars + 8u * s; };
  // the K slot of tile g is released by the stream that has seen the tile's scores complete
  auto bar_k_empty = [&](int s) { return bars + 8u * (KS + s); };
  auto bar_v_full = [&](int s) { return bars + 8u * (2 * KS + s); };
  // completion of the PV product of tile h, on barrier h % VS: frees the tile's V slot for the producer and
  // its P buffer for the softmax threads, and tells them that O holds the products up to tile h (one commit
  // for all three: every commit costs the issuing thread about as much as a product)
  auto bar_v_empty = [&](int s) { return bars + 8u * (2 * KS + VS + s); };
  static_assert(VS >= NP + 1, "a P buffer is reused before its tile's slot");
  const uint32_t b0 = bars + 8u * 2 * (KS + VS);
  auto bar_s_full = [&](int b) { return b0 + 8u * b; };
  auto bar_s_free = [&](int b) { return b0 + 8u * (2 + b); };
  auto bar_p_full = [&](int b) { return b0 + 8u * (4 + b); };
  auto bar_q_full = [&](int b) { return b0 + 8u * (8 + b); };
  auto bar_q_free = [&](int b) { return b0 + 8u * (10 + b); };
  const uint32_t bar_o_full = b0 + 8u * 12, bar_o_free = b0 + 8u * 13;
  const uint32_t bar_ml = b0 + 8u * 14;                 // the streams' (m, l) of an item are all in shared memory
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + L::kOffCtl);
  const WorkItem* item_cache = reinterpret_cast<const WorkItem*>(smem + L::kOffItems);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = P.Hq / P.Hkv;
  const int it_begin = A.cta_first[blockIdx.x], it_end = A.cta_first[blockIdx.x + 1];

  if (tid == 0) {
    for (int s = 0; s < KS; ++s) {
      mbar_init(bar_k_full(s), 1);
      mbar_init(bar_k_empty(s), 1);
    }
    for (int s = 0; s < VS; ++s) {
      mbar_init(bar_v_full(s), 1);
      mbar_init(bar_v_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_s_full(b), 1);
      mbar_init(bar_s_free(b), 4);                        // one arrival per warp of the stream that owns the buffer
      mbar_init(bar_p_full(b), 4);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_q_full(b), 4 * NS);
      mbar_init(bar_q_free(b), 1);
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, 4 * NS);
    mbar_init(bar_ml, 4 * NS);
    ctl->abort = 0;
    ctl->tmem_base = 0;
    ctl->limit_ns = A.wait_limit_ns ? A.wait_limit_ns : kWaitLimitNs;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int x = tid; x < min(it_end - it_begin, kItemCache) * 2; x += kThreads)
    reinterpret_cast<uint4*>(smem + L::kOffItems)[x] = reinterpret_cast<const uint4*>(A.items + it_begin)[x];
  // Q staging starts out as zeros: rows that no item uses stay finite
  for (int x = tid; x < L::kQBufs * L::kQBytes / 16; x += kThreads)
    reinterpret_cast<uint4*>(smem + L::kOffQ)[x] = make_uint4(0, 0, 0, 0);
  if (warp == L::kWarpMma) {
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
  const uint32_t tmem_s0 = tmem, tmem_o = tmem + 2 * kTile, tmem_p0 = tmem_o + NS * D;

  if (warp == L::kWarpProdK || warp == L::kWarpProdV) {
    // ------------------------------------------------------------------ TMA producers: one ring each, one copy per page
    const bool is_k = warp == L::kWarpProdK;
    const CUtensorMap* map = is_k ? &kmap : &vmap;
    const int NSLOT = is_k ? KS : VS;
    const uint32_t ring = sbase + (is_k ? L::kOffK : L::kOffV);
    const int pages_per_tile = kTile / P.bs;
    const uint32_t page_bytes = (uint32_t)P.bs * D * 2;
    // Page ids come 32 at a time (one coalesced load of the request's block-table row: four tiles' worth at 16 keys a
    // page), a chunk ahead of their use: a load per tile, even issued a tile early, put a global-memory round trip
    // into every pass of this loop and held a producer to one tile per ~1500 cycles.
    const int tiles_per_chunk = 32 / pages_per_tile;
    auto chunk_load = [&](const ItemView& v, int c) -> int {
      const int idx = c * 32 + lane;                       // page of the item's key range
      const int np_item = (v.key_end - v.key_begin + P.bs - 1) / P.bs;
      return idx < np_item ? __ldg(A.block_table + (size_t)v.req * P.max_blocks + v.key_begin / P.bs + idx) : -1;
    };
    uint32_t load_idx = 0;                                 // running tile number
    bool ok = it_begin < it_end;
    int it = it_begin, rb = 0;
    ItemView v = ok ? view(A, item_cache, it_begin, it_begin) : ItemView{};
    int ids = ok ? chunk_load(v, 0) : -1;
    while (ok) {
      // the (item, row block) that follows this one: the same keys again for the item's next 128 rows, or the next item
      int nit = it, nrb = rb + 1;
      ItemView nv = v;
      if (nrb == row_blocks_of(G, v)) {
        nrb = 0;
        nit = it + 1;
        if (nit < it_end) nv = view(A, item_cache, it_begin, nit);
      }
      const int nch = (v.tiles + tiles_per_chunk - 1) / tiles_per_chunk;
      for (int c = 0; c < nch && ok; ++c) {
        const int ids_next = c + 1 < nch ? chunk_load(v, c + 1) : (nit < it_end ? chunk_load(nv, 0) : -1);
        const int t_end = min(v.tiles, (c + 1) * tiles_per_chunk);
        for (int tile = c * tiles_per_chunk; tile < t_end; ++tile) {
          if (A.stall_after_loads >= 0 && (int)load_idx >= A.stall_after_loads) { ok = false; break; }   // (test hook: the copies stop coming)
          const int kbase = v.key_begin + tile * kTile;
          const int npages = min(pages_per_tile, (v.key_end - kbase + P.bs - 1) / P.bs);
          int page = __shfl_sync(0xffffffffu, ids, ((tile - c * tiles_per_chunk) * pages_per_tile + lane) & 31);
          if (lane >= npages) page = -1;
          if (lane < npages && (unsigned)page >= (unsigned)P.num_blocks) {
            atomicOr(P.status, kFlagBadPage);
            page = -1;
          }
          const int nvalid = __popc(__ballot_sync(0xffffffffu, page >= 0));
          const int slot = load_idx % NSLOT;
          const uint32_t par = ((load_idx / NSLOT) & 1u) ^ 1u;
          const uint32_t full = is_k ? bar_k_full(slot) : bar_v_full(slot);
          int good = 1;
          if (lane == 0) good = mbar_wait_c(is_k ? bar_k_empty(slot) : bar_v_empty(slot), par, ctl, P.status, is_k ? 0 : 1) ? 1 : 0;
          good = __shfl_sync(0xffffffffu, good, 0);
          if (!good) { ok = false; break; }
          if (lane == 0) mbar_arrive_expect_tx(full, (uint32_t)nvalid * page_bytes);
          __syncwarp();
          if (page >= 0)
            tma_load_5d(ring + slot * L::kTileBytes + lane * page_bytes, map, full, 0, 0, 0, 0, page * P.Hkv + v.kv_head);
          ++load_idx;
        }
        ids = ids_next;
      }
      if (nit >= it_end) break;
      it = nit;
      rb = nrb;
      v = nv;
    }
  } else if (warp == L::kWarpMma) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t idesc_s = instr_desc(L::kRows, kTile, false, false);   // S: M = 128 rows, N = 128 keys
      constexpr uint32_t idesc_pv = instr_desc(L::kRows, D, false, true);       // O: M = 128 rows, N = head_dim, B = V MN-major
      // Two cursors over this CTA's tiles: cs for the QK products, cp for the PV products.  Every operation of this
      // thread that touches the tensor unit or a barrier costs it 50-140 cycles, so a pass of the loop below looks at
      // all the barriers it may need at once.  QK(g) needs the tile's K slot and the stream's S buffer (s_free: the
      // stream has taken the scores of its previous tile out of tensor memory); PV(g) needs the weights P(g) and the
      // tile's V slot.  Whichever is ready goes, in any order: nothing here can wait for something it has yet to issue.
      struct Cursor {
        int it, rb;
        int tile;
        uint32_t g, item_idx;                               // running tile number; running (item, row block) number
        ItemView v;
      };
      Cursor cs{it_begin, 0, 0, 0, 0, it_begin < it_end ? view(A, item_cache, it_begin, it_begin) : ItemView{}};
      Cursor cp = cs;
      auto advance = [&](Cursor& c) {
        ++c.g;
        if (++c.tile == c.v.tiles) {
          c.tile = 0;
          ++c.item_idx;
          if (++c.rb == row_blocks_of(G, c.v)) {
            c.rb = 0;
            if (++c.it < it_end) c.v = view(A, item_cache, it_begin, c.it);
          }
        }
      };
      unsigned long long idle_since = 0;
      uint32_t spins = 0;
      while (cp.it < it_end) {
        const bool s_cand = cs.it < it_end;
        const bool p_cand = cp.g < cs.g;
        const int kslot = cs.g % KS, sbuf = cs.g & 1;
        const int vslot = cp.g % VS, pbuf = cp.g % NP;
        const uint32_t rdy = mbar_test4(bar_k_full(kslot), (cs.g / KS) & 1u, bar_s_free(sbuf), ((cs.g >> 1) & 1u) ^ 1u,
                                        bar_p_full(pbuf), (cp.g / NP) & 1u, bar_v_full(vslot), (cp.g / VS) & 1u);
        const bool p_first = cp.tile < NS;                 // the first tile of its stream in this item
        bool p_ok = p_cand && (rdy & 12u) == 12u;
        if (p_ok && p_first) p_ok = mbar_test(bar_o_free, (cp.item_idx & 1u) ^ 1u);   // the last item's O has been read
        bool s_ok = s_cand && (rdy & 3u) == 3u;
        if (s_ok && cs.tile == 0) s_ok = mbar_test(bar_q_full(cs.item_idx & 1u), (cs.item_idx >> 1) & 1u);
        if (s_ok || p_ok) tc_fence_after();
        if (s_ok) {
          // A = Q, B = K tile (both K-major, 128-byte swizzle): 32 bytes per step inside the 64-element atom
          const uint32_t k_lo = desc_lo(sbase + L::kOffK + kslot * L::kTileBytes, 16);
          const uint32_t q_lo = desc_lo(sbase + L::kOffQ + (cs.item_idx & 1u) * L::kQBytes, 16);
#pragma unroll
          for (int kk = 0; kk < KSTEPS_S; ++kk)
            umma_bf16(tmem_s0 + sbuf * kTile, q_lo + (kk * 32) / 16, desc_hi(1024, 2), k_lo + (kk * 32) / 16, desc_hi(SBO_KV, 2),
                      idesc_s, kk > 0);
          umma_commit(bar_s_full(sbuf));
          if (cs.tile == cs.v.tiles - 1) umma_commit(bar_q_free(cs.item_idx & 1u));
          advance(cs);
        }
        if (p_ok) {
          // A = P from TMEM (row = lane, 16 keys of a step = 8 columns); B = V (MN-major, 128-byte swizzle):
          // 16 keys per step = two 8-key groups
          const uint32_t p_t = tmem_p0 + pbuf * (kTile / 2);
          const uint32_t v_lo = desc_lo(sbase + L::kOffV + vslot * L::kTileBytes, 1024);
#pragma unroll
          for (int kk = 0; kk < KSTEPS_PV; ++kk)          // tile g belongs to stream g % NS and accumulates into its O
            umma_bf16_ta(tmem_o + (cp.g % NS) * D, p_t + kk * 8, v_lo + kk * (2 * SBO_KV / 16), desc_hi(SBO_KV, 2), idesc_pv,
                         !(p_first && kk == 0));
          umma_commit(bar_v_empty(vslot));
          if (cp.tile == cp.v.tiles - 1) umma_commit(bar_o_full);
          advance(cp);
        }
        if (s_ok || p_ok) {
          idle_since = 0;
          spins = 0;
        } else if ((++spins & 63u) == 0) {
          // nothing was ready: bounded like every other wait of the kernel
          if (ctl->abort) break;
          const unsigned long long now = global_ns();
          if (idle_since == 0) {
            idle_since = now;
          } else if (now - idle_since > ctl->limit_ns) {
            ctl->abort = 1;
            atomicOr(P.status, kFlagWaitCap | (1u << (8 + 2)));
            break;
          }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (thread = query row)
    const int stream = warp >> 2;                         // which tiles: those whose running number is `stream` modulo NS
    const int quarter = warp & 3;                         // TMEM lanes this warp may touch: 32 * quarter ..
    const int rp = quarter * 32 + lane;                   // this thread's TMEM lane = row of the Q operand
    // ... and which 32 rows of a block live there: rows 96..127 on the lanes of the issuing warp's scheduler
    const int lq = quarter == 2 ? 3 : (quarter == 3 ? 2 : quarter);
    const int r = lq * 32 + lane;                         // this thread's query row of the block
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    constexpr int CK = kTile;
    constexpr int NCH = CK / 32;                          // a tile's keys in chunks of 32
    const uint32_t tmem_os = tmem_o + stream * D;         // this stream's accumulator
    const float scale = A.scale_log2;
    const int W = A.window;
    float2* const ml_all = reinterpret_cast<float2*>(smem + L::kOffMl);
    bool ok = true;
    uint32_t g_run = 0;                                   // running number of the current (item, row block)'s first tile
    // One arrival per warp, after every lane has done its part (each lane fences its own accesses first): 128 * NS
    // arrivals on one barrier word are 128 * NS serialised shared-memory atomics per tile.
    auto warp_arrive = [&](uint32_t bar) {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar);
    };

    // Q of one (item, row block): row r = (draft position j / G, query head j % G of the group), 128 bytes; the
    // streams' threads of a row stage D / 8 / NS 16-byte chunks each, rows beyond the item's own are zeroed.  The
    // copies are asynchronous (cp.async) into the buffer the previous-but-one block used: issued when a block begins,
    // completed and announced after the stream's first tile of it, so the queries of the next block are in place long
    // before its first QK product and the global round trip is off the softmax threads' path.
    auto load_q_issue = [&](const ItemView& v, int rb, uint32_t item_idx) -> bool {
      const int qb = item_idx & 1u;
      if (!mbar_wait_c(bar_q_free(qb), ((item_idx >> 1) & 1u) ^ 1u, ctl, P.status, 8)) return false;
      constexpr int CPT = D / 8 / NS;
      const uint32_t qrow = sbase + L::kOffQ + qb * L::kQBytes + rp * 128;
      const int j = rb * L::kRows + r;                      // row of the item
      if (j < G * (v.k + 1)) {
        const __nv_bfloat16* src = A.q + ((size_t)(v.cu_q + j / G) * P.Hq + v.kv_head * G + j % G) * D;
#pragma unroll
        for (int x = 0; x < CPT; ++x)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(qrow + (((stream * CPT + x) ^ (rp & 7)) << 4)),
                       "l"(src + (stream * CPT + x) * 8)
                       : "memory");
      } else {
#pragma unroll
        for (int x = 0; x < CPT; ++x)
          *reinterpret_cast<uint4*>(smem + L::kOffQ + qb * L::kQBytes + rp * 128 + (((stream * CPT + x) ^ (rp & 7)) << 4)) =
              make_uint4(0, 0, 0, 0);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      return true;
    };
    auto load_q_finish = [&](uint32_t item_idx) {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      fence_proxy_async();
      warp_arrive(bar_q_full(item_idx & 1u));
    };

    if (it_begin < it_end) {
      ok = load_q_issue(view(A, item_cache, it_begin, it_begin), 0, 0);
      if (ok) load_q_finish(0);
    }
    uint32_t item_idx = 0;                                // running (item, row block) number
    for (int it = it_begin; it < it_end && ok; ++it)
    for (int rb = 0; ok; ++rb, ++item_idx) {
      const ItemView v = view(A, item_cache, it_begin, it);
      if (rb == row_blocks_of(G, v)) break;
      const int R = G * (v.k + 1) - rb * L::kRows;        // rows of the item from this block's first on
      const int j = rb * L::kRows + r;                    // this thread's row of the item
      const bool warp_active = lq * 32 < R;               // some row of this warp belongs to the item
      // keys this row may see: lo_r .. hi_r.  A row beyond the item's own (its queries are zeros) sees everything:
      // it costs its warp no masking, and what it computes is never stored.
      const int hi_r = r < R ? v.n + j / G : 0x7fffffff;
      const int lo_r = (r < R && W > 0) ? max(0, hi_r - W + 1) : 0;
      float m = -INFINITY, l = 0.f;                       // this stream's running reference (log2 units) and row sum
      float o_alpha = 1.f;                                // factor this row of O_s is still owed (see the optimistic pass)
      bool o_owed = false;                                // ... for some row of the warp
      bool own_first = true;                              // the stream has not had a tile of this item yet
      // the queries of the next (item, row block) start their way into the other Q buffer now
      bool q_pending = false;
      if (rb + 1 < row_blocks_of(G, v)) {
        if (!load_q_issue(v, rb + 1, item_idx + 1)) { ok = false; break; }
        q_pending = true;
      } else if (it + 1 < it_end) {
        if (!load_q_issue(view(A, item_cache, it_begin, it + 1), 0, item_idx + 1)) { ok = false; break; }
        q_pending = true;
      }

      // (only this stream's tiles are visited: a turn of this loop for the other stream's tile is a taken branch back over
      // the whole softmax, which costs about 200 cycles of instruction fetch)
      static_assert(NS == 2, "tile parity");
      for (int tile = (int)((stream ^ g_run) & 1u); tile < v.tiles && ok; tile += NS) {
        const uint32_t g = g_run + tile;
        const int kbase = v.key_begin + tile * kTile;
        const int sbuf = g & 1, pbuf = g % NP;
        if (!mbar_wait_c(bar_s_full(sbuf), (g >> 1) & 1u, ctl, P.status, 9)) { ok = false; break; }
        // the tile's scores are complete, so its K slot has served its purpose
        if (quarter == 0 && lane == 0) mbar_arrive(bar_k_empty(g % KS));
        tc_fence_after();
        // the P buffer of this tile becomes writable when the PV product that last read it (tile g - NP) is done: not
        // needed before the row maxima are known.  (That product is also the last that O_s was waiting for.)
        static_assert(NP == NS, "the P buffer's last reader is the stream's previous tile");
        auto wait_p = [&]() -> bool {
          return g < (uint32_t)NP || mbar_wait_c(bar_v_empty((g - NP) % VS), ((g - NP) / VS) & 1u, ctl, P.status, 10);
        };
        // All of a tile's scores have left tensor memory some way before its weights are finished: from then on the
        // issuing thread may compute the stream's next scores into the same buffer (arrival on s_free).
        bool s_released = false;
        auto release_s = [&]() {
          tc_fence_before();
          warp_arrive(bar_s_free(sbuf));
          s_released = true;
        };
        if (warp_active) {
          const uint32_t s_addr = tmem_s0 + sbuf * kTile + lane_addr;
          const uint32_t p_addr = tmem_p0 + pbuf * (kTile / 2) + lane_addr;
          const int t_first = kbase;
          // every row of the warp sees every key of the tile: the common case, which then
          // carries no masking code at all (a per-thread test is compiled into selects that every tile pays for)
          const bool interior = __all_sync(0xffffffffu, t_first >= lo_r && t_first + CK - 1 <= hi_r);
          auto max32 = [&](float mx, const float* y) -> float {      // (four chains: a single one is 16 dependent steps)
            float a = mx, b = y[0], c = y[1], d = y[2];
#pragma unroll
            for (int e = 3; e + 7 < 32; e += 8) {
              a = fmax3(a, y[e], y[e + 1]);
              b = fmax3(b, y[e + 2], y[e + 3]);
              c = fmax3(c, y[e + 4], y[e + 5]);
              d = fmax3(d, y[e + 6], y[e + 7]);
            }
            // (e = 3, 11, 19 covered y[3..26])
            a = fmax3(a, y[27], y[28]);
            b = fmax3(b, y[29], y[30]);
            c = fmaxf(c, y[31]);
            return fmax3(fmaxf(a, b), c, d);
          };
          // weights 2^(score - reference) of 32 keys in bf16 into the P buffer, their sum into acc.  The subtraction and
          // the row sum run on packed pairs (fma / add .f32x2).
          auto chunk_pack = [&](const float* y, uint64_t sc2, uint64_t nm2, uint64_t* acc, uint32_t* pk) {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              float d0, d1;
              unpack2(fma2(pack2(y[e], y[e + 1]), sc2, nm2), d0, d1);
              const float p0 = exp2f(d0), p1 = exp2f(d1);
              acc[(e >> 1) & 3] = add2(acc[(e >> 1) & 3], pack2(p0, p1));
              const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);
              pk[e >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
            }
          };
          auto chunk_weights = [&](int c, const float* y, uint64_t sc2, uint64_t nm2, uint64_t* acc) {
            uint32_t pk[16];
            chunk_pack(y, sc2, nm2, acc, pk);
            tmem_st16u(p_addr + c * 16, pk);              // 32 keys = 16 columns of the row's lane
          };
          // The row's reference follows its running maximum lazily: it moves only when the tile's maximum exceeds it by
          // more than 2^kRescaleStep (weights up to that size are harmless), which after the first tiles is rare.  When
          // it moves for some row of the warp, the warp rescales its rows of O_s (a collective access) and its sums.
          // Only the item's own rows vote: a lane beyond them multiplies zero queries with whatever the slot holds.
          // The P buffer is writable, and O_s holds the products up to the stream's previous tile, once that tile's PV
          // product is done.
          bool p_waited = false;
          if (o_owed || !interior) {
            if (!wait_p()) { ok = false; break; }
            p_waited = true;
          }
          // factor by which this row of O_s is to be multiplied (collective: every lane of the warp takes part)
          auto scale_o = [&](float f) {
            tc_fence_after();
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
              float o[32];
              tmem_ld32(tmem_os + lane_addr + c * 32, o);
              tmem_wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] *= f;
              tmem_st32(tmem_os + lane_addr + c * 32, o);
            }
            tmem_wait_st();
          };
          if (o_owed) {                                     // a reference moved after the previous tile's weights were out
            scale_o(o_alpha);
            o_alpha = 1.f;
            o_owed = false;
          }
          // The row's reference follows its running maximum lazily: it moves only when the tile's maximum exceeds it by
          // more than 2^kRescaleStep (weights up to that size are harmless).  When it moves for some row of the warp, the
          // warp rescales its rows of O_s and its sums.  Only the item's own rows vote: a lane beyond them multiplies
          // zero queries with whatever the slot holds.
          auto new_reference = [&](float mx) {
            const float cand = mx * scale;
            if (!__any_sync(0xffffffffu, r < R && cand > m + kRescaleStep)) return;
            const float mnew = fmaxf(m, cand);
            const float alpha = m == -INFINITY ? 0.f : exp2f(m - mnew);
            if (!own_first) scale_o(alpha);
            l *= alpha;
            m = mnew;
          };
          float lt = 0.f;
          bool from_memory = false;
          if (interior) {
            // The stream's first tile of an item, or a row of the warp that has seen no key so far: references first.
            // Pass 1 takes the row maxima (two chunks of 32 scores at a time) and moves the references.
            const bool careful = own_first || __any_sync(0xffffffffu, r < R && m == -INFINITY);
            float ya[32], yb[32];
            if (careful) {
              if (!p_waited && !wait_p()) { ok = false; break; }      // (the references may move, and O_s with them)
              p_waited = true;
              float mx = -INFINITY;
              tmem_ld32(s_addr + 1 * 32, ya);
              tmem_ld32(s_addr + 2 * 32, yb);
              tmem_wait_ld();
              mx = max32(max32(mx, ya), yb);
              tmem_ld32(s_addr + 3 * 32, ya);
              tmem_ld32(s_addr + 0 * 32, yb);
              tmem_wait_ld();
              mx = max32(max32(mx, ya), yb);
              new_reference(mx);
            }
            // The weights, optimistically against the references as they stand: no maximum is taken.  The scores leave
            // tensor memory for good before the last chunk's weights are computed, and the S buffer is released there.
            // (a row that still sees nothing measures against 0: it has no finite score)
            const float mref = m == -INFINITY ? 0.f : m;
            const uint64_t sc2 = pack2(scale, scale), nm2 = pack2(-mref, -mref);
            uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
            // The first two chunks' weights wait in registers for the P buffer: the PV product that last read it follows
            // this stream's previous tile by the time of eight products, which the stream would otherwise spend idle.
            uint32_t pka[16], pkb[16];
            tmem_ld32(s_addr + 0 * 32, yb);
            tmem_ld32(s_addr + 3 * 32, ya);
            tmem_wait_ld();
            chunk_pack(yb, sc2, nm2, acc, pka);
            tmem_ld32(s_addr + 1 * 32, yb);
            chunk_pack(ya, sc2, nm2, acc, pkb);
            tmem_wait_ld();
            tmem_ld32(s_addr + 2 * 32, ya);
            if (!p_waited && !wait_p()) { ok = false; break; }
            tmem_st16u(p_addr + 0 * 16, pka);
            tmem_st16u(p_addr + 3 * 16, pkb);
            chunk_weights(1, yb, sc2, nm2, acc);
            tmem_wait_ld();
            release_s();
            chunk_weights(2, ya, sc2, nm2, acc);
            tmem_wait_st();
            float s0, s1;
            unpack2(add2(add2(acc[0], acc[1]), add2(acc[2], acc[3])), s0, s1);
            lt = s0 + s1;
            if (!careful) {
              // A score far above its reference shows in the sum of the tile's weights (so does an overflow), and the
              // test on the sum costs nothing per key.  Large but finite weights are as good as any (bf16 keeps their
              // relative precision, O_s and the sum are fp32): the reference moves AFTERWARDS, to within 2^3.5 of the
              // tile's maximum, the sum is rescaled now and the row of O_s at the stream's next tile, when this tile's
              // PV product has completed.  Weights that may have overflowed are computed again from memory.
              if (__any_sync(0xffffffffu, r < R && !(lt <= kGrowSum))) {
                if (__any_sync(0xffffffffu, r < R && !(lt <= kHugeSum))) {
                  from_memory = true;
                } else {
                  const float mnew = lt > kGrowSum ? m + log2f(lt) - 3.5f : m;
                  o_alpha = exp2f(m - mnew);
                  l = (l + lt) * o_alpha;
                  lt = 0.f;
                  m = mnew;
                  o_owed = true;
                }
              }
            }
          } else {
            // An item's last tile, a window's first: chunk by chunk.  A chunk that no row of the warp sees costs
            // nothing (weights 0), one that every row sees in full runs unmasked, and only the chunks cut by some row's
            // first or last key pay for the selects (rows beyond the item's own do not care).
            auto chunk_class = [&](int c) -> int {          // 0: no row sees any key, 1: some row sees some, 2: all see all
              const int t0 = t_first + c * 32;
              if (__all_sync(0xffffffffu, r >= R || t0 > hi_r || t0 + 31 < lo_r)) return 0;
              return __all_sync(0xffffffffu, r >= R || (t0 >= lo_r && t0 + 31 <= hi_r)) ? 2 : 1;
            };
            auto masked_scores = [&](int c, int cls, float* y) {
              tmem_ld32(s_addr + c * 32, y);
              tmem_wait_ld();
              if (cls == 1) {
                const int t0 = t_first + c * 32;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (t0 + e > hi_r || t0 + e < lo_r) y[e] = -INFINITY;
              }
            };
            float mx = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < NCH; ++c) {
              const int cls = chunk_class(c);
              if (cls == 0) continue;
              float y[32];
              masked_scores(c, cls, y);
              mx = max32(mx, y);
            }
            new_reference(mx);
            const float mref = m == -INFINITY ? 0.f : m;
            const uint64_t sc2 = pack2(scale, scale), nm2 = pack2(-mref, -mref);
            uint64_t acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll 1
            for (int c = 0; c < NCH; ++c) {
              const int cls = chunk_class(c);
              if (cls == 0) {
                uint32_t pk[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) pk[e] = 0u;
                tmem_st16u(p_addr + c * 16, pk);
                continue;
              }
              float y[32];
              masked_scores(c, cls, y);
              chunk_weights(c, y, sc2, nm2, acc);
            }
            tmem_wait_st();
            float s0, s1;
            unpack2(add2(add2(acc[0], acc[1]), add2(acc[2], acc[3])), s0, s1);
            lt = s0 + s1;
          }
          if (from_memory) {
            const int jm = r < R ? j : -1;
            rows_tile_from_memory<D>(jm >= 0 ? A.q + ((size_t)(v.cu_q + jm / G) * P.Hq + v.kv_head * G + jm % G) * D : nullptr, A.k_pool,
                                     A.block_table + (size_t)v.req * P.max_blocks, P.bs, P.Hkv, v.kv_head, P.num_blocks, kbase,
                                     v.key_end, hi_r, lo_r, scale, p_addr, tmem_os + lane_addr, own_first, m, l);
            lt = 0.f;
          }
          l += lt;
        } else if (!wait_p()) {
          // (a warp without rows announces P(g) too, and may do so only when the buffer's last reader is done:
          // otherwise its arrival could land in the barrier's previous phase)
          ok = false;
          break;
        }
        own_first = false;
        if (!s_released) release_s();
        tc_fence_before();
        if (kbase + rp >= v.key_end) {
          // keys past the end of the request: their V rows (page tail or a slot row that no copy touched) may
          // hold anything, and 0 * NaN would poison O.  Zero them before the product.  (Thread rp looks after key rp.)
          const int vslot = g % VS;
          if (mbar_wait_c(bar_v_full(vslot), (g / VS) & 1u, ctl, P.status, 12)) {
            unsigned char* vr = smem + L::kOffV + vslot * L::kTileBytes + (rp >> 3) * SBO_KV + (rp & 7) * 128;
#pragma unroll
            for (int x = 0; x < 8; ++x) *reinterpret_cast<uint4*>(vr + x * 16) = make_uint4(0, 0, 0, 0);
            fence_proxy_async();
          }
        }
        warp_arrive(bar_p_full(pbuf));
        if (q_pending) {                                    // after the stream's first tile of the block: they have landed
          load_q_finish(item_idx + 1);
          q_pending = false;
        }
      }
      if (!ok) break;
      g_run += v.tiles;
      if (q_pending) load_q_finish(item_idx + 1);         // (a block in which this stream had no tile)

      // ---- epilogue: merge the streams' (m, l, O_s) of every row; thread (stream, r) finishes D / NS columns of row r ----
      if (!mbar_wait_c(bar_o_full, item_idx & 1u, ctl, P.status, 13)) { ok = false; break; }
      tc_fence_after();
      if (o_owed) {
        // the reference of some row moved after the stream's last tile: its row of O_s has yet to follow
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          float o[32];
          tmem_ld32(tmem_os + lane_addr + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] *= o_alpha;
          tmem_st32(tmem_os + lane_addr + c * 32, o);
        }
        tmem_wait_st();
        tc_fence_before();
      }
      float2* const ml = ml_all + (item_idx & 1u) * (NS * L::kRows);
      ml[stream * L::kRows + rp] = make_float2(m, l);
      warp_arrive(bar_ml);
      if (!mbar_wait_c(bar_ml, item_idx & 1u, ctl, P.status, 14)) { ok = false; break; }
      tc_fence_after();
      if (warp_active) {
        constexpr int DC = D / NS;                          // output columns per thread
        float mt = -INFINITY;
#pragma unroll
        for (int t = 0; t < NS; ++t) mt = fmaxf(mt, ml[t * L::kRows + rp].x);
        float lt = 0.f;
        float o[DC];
#pragma unroll
        for (int e = 0; e < DC; ++e) o[e] = 0.f;
#pragma unroll
        for (int t = 0; t < NS; ++t) {
          const float2 x = ml[t * L::kRows + rp];
          const float wt = x.x == -INFINITY ? 0.f : exp2f(x.x - mt);
          lt = fmaf(wt, x.y, lt);
          float ot[DC];
          if constexpr (DC == 32) tmem_ld32(tmem_o + t * D + lane_addr + stream * DC, ot);
          else if constexpr (DC == 16) tmem_ld16(tmem_o + t * D + lane_addr + stream * DC, ot);
          else {
            tmem_ld32(tmem_o + t * D + lane_addr, ot);
            tmem_ld32(tmem_o + t * D + lane_addr + 32, ot + 32);
          }
          tmem_wait_ld();
          // (a stream that saw no key of the row holds nothing meaningful in O_t: its weight is an exact zero)
#pragma unroll
          for (int e = 0; e < DC; ++e) o[e] = wt == 0.f ? o[e] : fmaf(wt, ot[e], o[e]);
        }
        if (r < R) {
          if (v.part_row >= 0) {
            if (stream == 0) A.part_ml[v.part_row + j] = make_float2(mt, lt);   // partials stay unnormalised
            float4* dst = reinterpret_cast<float4*>(A.part_o + (size_t)(v.part_row + j) * D + stream * DC);
#pragma unroll
            for (int x = 0; x < DC / 4; ++x) dst[x] = make_float4(o[4 * x], o[4 * x + 1], o[4 * x + 2], o[4 * x + 3]);
          } else {
            const int pos = j / G, h = v.kv_head * G + (j - pos * G);
            float sc = 1.f;
            if (A.sinks) {
              const float sk = A.sinks[h] * 1.4426950408889634f;
              const float m2 = fmaxf(mt, sk);
              sc = exp2f(mt - m2);
              lt = lt * sc + exp2f(sk - m2);
              mt = m2;
            }
            const size_t row = (size_t)(v.cu_q + pos) * P.Hq + h;
            const float inv = sc / lt;
            if (stream == 0 && A.lse) A.lse[row] = (mt + log2f(lt)) * 0.6931471805599453f;
            uint4* dst = reinterpret_cast<uint4*>(A.out + row * D + stream * DC);
#pragma unroll
            for (int x = 0; x < DC / 8; ++x) {
              uint32_t w[4];
#pragma unroll
              for (int y = 0; y < 4; ++y) {
                const __nv_bfloat162 b = __floats2bfloat162_rn(o[8 * x + 2 * y] * inv, o[8 * x + 2 * y + 1] * inv);
                w[y] = *reinterpret_cast<const uint32_t*>(&b);
              }
              dst[x] = make_uint4(w[0], w[1], w[2], w[3]);
            }
          }
        }
      }
      tc_fence_before();
      warp_arrive(bar_o_free);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (ctl->abort) {
    const unsigned long long t0 = global_ns();
    while (global_ns() - t0 < 200000ull) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == L::kWarpMma) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

cudaError_t launch_rows_instance(const CUtensorMap& km, const CUtensorMap& vm, const DevPlan& P, const AttnArgs& A, cudaStream_t s) {
  constexpr int D = 64, NS = 2;
  const int smem = RowsSmem<D, NS>::kTotal + 1024;
  // the opt-in to large dynamic shared memory is per device and costs a few microseconds: once is enough
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !opted_in[dev]) {
    e = cudaFuncSetAttribute(attn_rows_kernel<D, NS>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  attn_rows_kernel<D, NS><<<A.num_ctas, RowsSmem<D, NS>::kThreads, smem, s>>>(km, vm, P, A);
  return cudaGetLastError();
}
