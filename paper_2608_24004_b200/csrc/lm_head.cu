// The target model's output projection fused with the greedy acceptance test: logits[r][v] = <hidden[r], weight[v]>
// are computed tile by tile on the tensor cores (tcgen05, accumulators in TMEM, operands staged by TMA) and every
// tile is reduced at once to "largest logit of the row and where", so the [rows, vocab] fp32 logits (0.2 - 1.75 GB
// per step in the workloads here) are never written or read.  A dense contraction: bound by the tensor pipe (and,
// for few rows, by the one pass over the weights).
//
// Tile: 128 rows x 256 vocabulary entries, K in blocks of 64 (one 128-byte swizzle atom per row), four stages of
// A (16 KB) + W (32 KB); two accumulators of 256 TMEM columns, so the reduction of one tile overlaps the products
// of the next.  Warp 0 issues the TMA copies, one lane of warp 1 the tcgen05.mma, warps 2..5 reduce (thread = row
// = TMEM lane).  Units (vocabulary tile, row tile) are dealt round-robin with the row tile fastest, so the CTAs
// that share a weight tile read it at the same time and all but the first find it in L2.  Every wait is bounded.
//
// Three epilogues share the pipeline (template parameter): the row argmax alone (greedy acceptance); the argmax plus
// what rejection sampling needs of a row - per vocabulary tile the online pair (max, sum of 2^((z - max) / T)) and the
// logit of the row's draft token - for as_accept_lm_head_sampled; and plain fp32 logits stored to memory, which that
// call uses for the one row per request whose recovery distribution has to be sampled.
#include <cuda.h>

#include "lm_head.cuh"
#include "tc_ptx.cuh"

namespace asv {

namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64, kStages = 4;
constexpr int kABytes = kBM * kBK * 2, kWBytes = kBN * kBK * 2, kStageBytes = kABytes + kWBytes;
constexpr int kLmThreads = 192;
constexpr int kLmSmem = kStages * kStageBytes + 1024 /* alignment */ + 16 * 8 + 256;

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}

// (value, column) as one integer whose order is "larger value first, then lower column"
__device__ __forceinline__ unsigned long long pack_key(float v, int col) {
  const uint32_t b = __float_as_uint(v);
  const uint32_t ord = b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
  return ((unsigned long long)ord << 32) | (0xffffffffu - (uint32_t)col);
}

constexpr int kEpiArgmax = 0, kEpiStats = 1, kEpiStore = 2;
struct LmEpilogue {
  unsigned long long* keys;         // argmax, stats: packed (largest logit, its column) per row, folded with atomicMax
  float2* tile_part;                // stats: [rows, n_tiles] (max, sum) of 2^(z log2e / T - max) over the tile, log2 units
  float* zd;                        // stats: [rows] logit of the row's draft token
  const int32_t* draft_tokens;      // stats
  const float* temperature;         // stats: per request; <= 0 = greedy (no statistics)
  float* store;                     // store: [rows, store_ld] fp32 logits
  long long store_ld;
  int rows;                         // rows of the A operand that exist (the step's rows, or the batch for the store pass)
};

template <int EPI>
__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap wmap, DevPlan P,
               int H, int V, int m_tiles, int n_tiles, LmEpilogue E) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + kStages * kStageBytes;
  auto bar_full = [&](int s) { return bars + 8u * s; };
  auto bar_empty = [&](int s) { return bars + 8u * (kStages + s); };
  auto bar_acc_full = [&](int b) { return bars + 8u * (2 * kStages + b); };
  auto bar_acc_free = [&](int b) { return bars + 8u * (2 * kStages + 2 + b); };
  Ctl* ctl = reinterpret_cast<Ctl*>(smem + kStages * kStageBytes + 16 * 8);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int total_q = EPI == kEpiStore ? min(E.rows, P.hdr->batch) : P.hdr->total_q;
  const int units = m_tiles * n_tiles;
  const int KB = H / kBK;
  constexpr uint32_t TMEM_COLS = 512;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(bar_full(s), 1);
      mbar_init(bar_empty(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar_acc_full(b), 1);
      mbar_init(bar_acc_free(b), 4);                      // one arrival per reducing warp
    }
    ctl->abort = 0;
    ctl->tmem_base = 0;
    ctl->limit_ns = kWaitLimitNs;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
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

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int n = u / m_tiles, m = u - n * m_tiles;
        if (m * kBM >= total_q) continue;                 // a row tile beyond this step's rows
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kStages;
          if (!mbar_wait(bar_empty(s), ((it / kStages) & 1u) ^ 1u, ctl, P.status, 0)) { ok = false; break; }
          mbar_arrive_expect_tx(bar_full(s), kStageBytes);
          tma_load_2d(sbase + s * kStageBytes, &amap, bar_full(s), kb * kBK, m * kBM);
          tma_load_2d(sbase + s * kStageBytes + kABytes, &wmap, bar_full(s), kb * kBK, n * kBN);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc(kBM, kBN, false, false);
      uint32_t it = 0, ul = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int n = u / m_tiles, m = u - n * m_tiles;
        if (m * kBM >= total_q) continue;
        const int buf = ul & 1;
        if (!mbar_wait(bar_acc_free(buf), ((ul >> 1) & 1u) ^ 1u, ctl, P.status, 1)) break;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kStages;
          if (!mbar_wait(bar_full(s), (it / kStages) & 1u, ctl, P.status, 2)) { ok = false; break; }
          tc_fence_after();
          // both operands K-major with the 128-byte swizzle: 32 bytes per K step of 16 inside the atom
          const uint32_t a_lo = desc_lo(sbase + s * kStageBytes, 16), w_lo = desc_lo(sbase + s * kStageBytes + kABytes, 16);
#pragma unroll
          for (int kk = 0; kk < kBK / 16; ++kk)
            umma_bf16(tmem + buf * kBN, a_lo + kk * 2, desc_hi(1024, 2), w_lo + kk * 2, desc_hi(1024, 2), idesc, (kb | kk) != 0);
          umma_commit(bar_empty(s));
        }
        if (ok) umma_commit(bar_acc_full(buf));
        ++ul;
      }
    }
  } else {
    // ------------------------------------------------------------------ reduction (thread = row = TMEM lane)
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    uint32_t ul = 0;
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
      const int n = u / m_tiles, m = u - n * m_tiles;
      if (m * kBM >= total_q) continue;
      const int buf = ul & 1;
      if (!mbar_wait(bar_acc_full(buf), (ul >> 1) & 1u, ctl, P.status, 3)) break;
      tc_fence_after();
      const int col0 = n * kBN;
      const int r = m * kBM + row;
      if constexpr (EPI == kEpiStore) {
        // the tile's logits as they are, 128 bytes per thread and chunk
        float* dst = E.store + (size_t)r * E.store_ld + col0;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          float y[32];
          tmem_ld32(tmem + buf * kBN + lane_addr + c * 32, y);
          tmem_wait_ld();
          if (r < total_q) {
            if (col0 + c * 32 + 31 < V && (E.store_ld & 3) == 0) {
#pragma unroll
              for (int e = 0; e < 32; e += 4) *reinterpret_cast<float4*>(dst + c * 32 + e) = make_float4(y[e], y[e + 1], y[e + 2], y[e + 3]);
            } else {
#pragma unroll
              for (int e = 0; e < 32; ++e)
                if (col0 + c * 32 + e < V) dst[c * 32 + e] = y[e];
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_free(buf));
      } else {
        float best = -INFINITY;                             // NaN never compares greater: it counts as -inf
        int best_col = col0;
        // what a sampling request's row needs besides: scale of its exponent, its draft token, running (max, sum)
        float cT = 0.f, sm = -INFINITY, ss = 0.f;
        int d = -1;
        if constexpr (EPI == kEpiStats) {
          if (r < total_q) {
            const int2 rj = P.row_map[r];
            const float T = E.temperature[rj.x];
            if (T > 0.f) {
              cT = 1.4426950408889634f / T;
              const ReqMeta rq = P.req[rj.x];
              if (rj.y < rq.k) d = E.draft_tokens[rq.cu_d + rj.y];
            }
          }
        }
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          float y[32];
          tmem_ld32(tmem + buf * kBN + lane_addr + c * 32, y);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float v = y[e] + 0.f;                     // -0 becomes +0: equal logits must tie
            const int col = col0 + c * 32 + e;
            if (col < V && v > best) {                      // strict: the lowest column of a tie stays
              best = v;
              best_col = col;
            }
          }
          if constexpr (EPI == kEpiStats) {
            if (cT > 0.f) {
              // entries past the vocabulary (zero fill of the copy) and NaN count as -inf
              float mx = -INFINITY;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                if (col0 + c * 32 + e >= V || y[e] != y[e]) y[e] = -INFINITY;
                mx = fmaxf(mx, y[e]);
              }
              const float mnew = fmaxf(sm, mx * cT);
              if (mnew > -INFINITY) {
                float add = 0.f;
#pragma unroll
                for (int e = 0; e < 32; ++e) add += exp2f(fmaf(y[e], cT, -mnew));
                ss = ss * exp2f(sm - mnew) + add;           // sm = -inf: ss is 0 and 2^-inf = 0
                sm = mnew;
              }
              const int de = d - (col0 + c * 32);
              if (de >= 0 && de < 32) {
                float zd = -INFINITY;
#pragma unroll
                for (int e = 0; e < 32; ++e)
                  if (e == de) zd = y[e];
                E.zd[r] = zd;
              }
            }
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_acc_free(buf));
        if (r < total_q) {
          atomicMax(E.keys + r, pack_key(best, best_col));
          if constexpr (EPI == kEpiStats) E.tile_part[(size_t)r * n_tiles + n] = make_float2(sm, ss);
        }
      }
      ++ul;
    }
  }

  if (ctl->abort) {
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

// keys -> (largest logit, its column) in the layout the acceptance decision reads
__global__ void lm_head_finish_kernel(DevPlan P, const unsigned long long* __restrict__ keys, float4* __restrict__ row_final) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= P.hdr->total_q) return;
  const unsigned long long k = keys[r];
  const uint32_t ord = (uint32_t)(k >> 32);
  const uint32_t bits = ord ^ ((ord >> 31) ? 0x80000000u : 0xffffffffu);
  const int col = (int)(0xffffffffu - (uint32_t)k);
  row_final[r] = make_float4(__uint_as_float(bits), __int_as_float(col), 0.f, 0.f);
}

// The same for a sampling step: the tile partials of a row folded in tile order by one warp (fixed order: the result
// does not depend on which CTA computed which tile) into (scaled max, sum) beside the argmax.
__global__ void lm_head_finish_stats_kernel(DevPlan P, const unsigned long long* __restrict__ keys,
                                            const float2* __restrict__ tile_part, int n_tiles, float4* __restrict__ row_final) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (r >= P.hdr->total_q) return;
  float m = -INFINITY, s = 0.f;
  for (int t = lane; t < n_tiles; t += 32) {
    const float2 p = tile_part[(size_t)r * n_tiles + t];
    if (p.x == -INFINITY) continue;
    const float mm = fmaxf(m, p.x);
    s = (m == -INFINITY ? 0.f : s * exp2f(m - mm)) + p.y * exp2f(p.x - mm);
    m = mm;
  }
  for (int o = 16; o; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    if (m2 != -INFINITY) {
      const float mm = fmaxf(m, m2);
      s = (m == -INFINITY ? 0.f : s * exp2f(m - mm)) + s2 * exp2f(m2 - mm);
      m = mm;
    }
  }
  if (lane == 0) {
    const unsigned long long k = keys[r];
    const uint32_t ord = (uint32_t)(k >> 32);
    const uint32_t bits = ord ^ ((ord >> 31) ? 0x80000000u : 0xffffffffu);
    const int col = (int)(0xffffffffu - (uint32_t)k);
    row_final[r] = make_float4(__uint_as_float(bits), __int_as_float(col), m, s);
  }
}

// hidden state of the row each sampling request draws its extra token from (row a_i), gathered into [batch, H];
// zeros for requests that do not sample
__global__ void lm_head_gather_rows_kernel(DevPlan P, const int32_t* __restrict__ recover_row, const uint4* __restrict__ hidden,
                                           uint4* __restrict__ out, int H8) {
  const int i = blockIdx.x;
  if (i >= P.hdr->batch) return;
  const int a = recover_row[i];
  const uint4* src = a >= 0 ? hidden + (size_t)(P.req[i].cu_q + a) * H8 : nullptr;
  for (int x = threadIdx.x; x < H8; x += blockDim.x) out[(size_t)i * H8 + x] = src ? src[x] : make_uint4(0, 0, 0, 0);
}

bool encode_2d(void* map, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows, std::string& err) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) {
    err = "cuTensorMapEncodeTiled is not available from the driver";
    return false;
  }
  const cuuint64_t dims[2] = {inner, rows};
  const cuuint64_t strides[1] = {inner * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(reinterpret_cast<CUtensorMap*>(map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                        strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    err = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
    return false;
  }
  return true;
}

}  // namespace

namespace {

bool refresh_maps(LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent, std::string& err) {
  if (st.hidden != hidden || st.weight != weight || st.H != H || st.V != V || st.rows != rows_extent) {
    if (!encode_2d(st.a_map, hidden, (uint64_t)H, (uint64_t)rows_extent, kBM, err)) return false;
    if (!encode_2d(st.w_map, weight, (uint64_t)H, (uint64_t)V, kBN, err)) return false;
    st.hidden = hidden;
    st.weight = weight;
    st.H = H;
    st.V = V;
    st.rows = rows_extent;
  }
  return true;
}

template <int EPI>
cudaError_t launch_epilogue(const LmHeadState& st, const DevPlan& P, int H, int V, int rows_extent, int num_sms, const LmEpilogue& E,
                            cudaStream_t s) {
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess && (dev < 0 || dev >= 64 || !opted_in[dev])) {
    e = cudaFuncSetAttribute(lm_head_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLmSmem);
    if (e == cudaSuccess && dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  if (e != cudaSuccess) return e;
  const int m_tiles = (rows_extent + kBM - 1) / kBM, n_tiles = (V + kBN - 1) / kBN;
  const int grid = m_tiles * n_tiles < num_sms ? m_tiles * n_tiles : num_sms;
  lm_head_kernel<EPI><<<grid, kLmThreads, kLmSmem, s>>>(*reinterpret_cast<const CUtensorMap*>(st.a_map),
                                                         *reinterpret_cast<const CUtensorMap*>(st.w_map), P, H, V, m_tiles, n_tiles, E);
  return cudaGetLastError();
}

}  // namespace

int lm_head_vocab_tiles(int V) { return (V + kBN - 1) / kBN; }

int launch_lm_head_argmax(const DevPlan& P, LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent,
                          int num_sms, unsigned long long* keys, float4* row_final, cudaStream_t s, std::string& err) {
  if (rows_extent <= 0) return 0;
  if (!refresh_maps(st, hidden, weight, H, V, rows_extent, err)) return 4;
  LmEpilogue E{};
  E.keys = keys;
  E.rows = rows_extent;
  cudaError_t e = cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)rows_extent, s);
  if (e == cudaSuccess) e = launch_epilogue<kEpiArgmax>(st, P, H, V, rows_extent, num_sms, E, s);
  if (e == cudaSuccess) {
    lm_head_finish_kernel<<<(rows_extent + 255) / 256, 256, 0, s>>>(P, keys, row_final);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    err = std::string("output projection launch: ") + cudaGetErrorString(e);
    return 4;
  }
  return 0;
}

int launch_lm_head_stats(const DevPlan& P, LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent,
                         int num_sms, unsigned long long* keys, float2* tile_part, float* zd, const int32_t* draft_tokens,
                         const float* temperature, float4* row_final, cudaStream_t s, std::string& err) {
  if (rows_extent <= 0) return 0;
  if (!refresh_maps(st, hidden, weight, H, V, rows_extent, err)) return 4;
  LmEpilogue E{};
  E.keys = keys;
  E.tile_part = tile_part;
  E.zd = zd;
  E.draft_tokens = draft_tokens;
  E.temperature = temperature;
  E.rows = rows_extent;
  cudaError_t e = cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)rows_extent, s);
  if (e == cudaSuccess) e = launch_epilogue<kEpiStats>(st, P, H, V, rows_extent, num_sms, E, s);
  if (e == cudaSuccess) {
    lm_head_finish_stats_kernel<<<(rows_extent + 7) / 8, 256, 0, s>>>(P, keys, tile_part, lm_head_vocab_tiles(V), row_final);
    e = cudaGetLastError();
  }
  if (e != cudaSuccess) {
    err = std::string("output projection launch: ") + cudaGetErrorString(e);
    return 4;
  }
  return 0;
}

int launch_lm_head_recover_rows(const DevPlan& P, LmHeadState& st, const int32_t* recover_row, const void* hidden, void* hidden_rows,
                                const void* weight, int H, int V, int batch_extent, int num_sms, float* logits, long long ld,
                                cudaStream_t s, std::string& err) {
  if (batch_extent <= 0) return 0;
  if (!refresh_maps(st, hidden_rows, weight, H, V, batch_extent, err)) return 4;
  lm_head_gather_rows_kernel<<<batch_extent, 128, 0, s>>>(P, recover_row, static_cast<const uint4*>(hidden),
                                                          static_cast<uint4*>(hidden_rows), H / 8);
  cudaError_t e = cudaGetLastError();
  LmEpilogue E{};
  E.store = logits;
  E.store_ld = ld;
  E.rows = batch_extent;
  if (e == cudaSuccess) e = launch_epilogue<kEpiStore>(st, P, H, V, batch_extent, num_sms, E, s);
  if (e != cudaSuccess) {
    err = std::string("output projection launch: ") + cudaGetErrorString(e);
    return 4;
  }
  return 0;
}

}  // namespace asv
