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

__global__ void __launch_bounds__(kLmThreads, 1)
lm_head_argmax_kernel(const __grid_constant__ CUtensorMap amap, const __grid_constant__ CUtensorMap wmap, DevPlan P,
                      int H, int V, int m_tiles, int n_tiles, unsigned long long* __restrict__ keys) {
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
  const int total_q = P.hdr->total_q;
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
      float best = -INFINITY;                             // NaN never compares greater: it counts as -inf
      int best_col = col0;
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
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_acc_free(buf));
      const int r = m * kBM + row;
      if (r < total_q) atomicMax(keys + r, pack_key(best, best_col));
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

int launch_lm_head_argmax(const DevPlan& P, LmHeadState& st, const void* hidden, const void* weight, int H, int V, int rows_extent,
                          int num_sms, unsigned long long* keys, float4* row_final, cudaStream_t s, std::string& err) {
  if (rows_extent <= 0) return 0;
  if (st.hidden != hidden || st.weight != weight || st.H != H || st.V != V || st.rows != rows_extent) {
    if (!encode_2d(st.a_map, hidden, (uint64_t)H, (uint64_t)rows_extent, kBM, err)) return 4;
    if (!encode_2d(st.w_map, weight, (uint64_t)H, (uint64_t)V, kBN, err)) return 4;
    st.hidden = hidden;
    st.weight = weight;
    st.H = H;
    st.V = V;
    st.rows = rows_extent;
  }
  static bool opted_in[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess && (dev < 0 || dev >= 64 || !opted_in[dev])) {
    e = cudaFuncSetAttribute(lm_head_argmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLmSmem);
    if (e == cudaSuccess && dev >= 0 && dev < 64) opted_in[dev] = true;
  }
  if (e == cudaSuccess) e = cudaMemsetAsync(keys, 0, sizeof(unsigned long long) * (size_t)rows_extent, s);
  if (e == cudaSuccess) {
    const int m_tiles = (rows_extent + kBM - 1) / kBM, n_tiles = (V + kBN - 1) / kBN;
    const int grid = m_tiles * n_tiles < num_sms ? m_tiles * n_tiles : num_sms;
    lm_head_argmax_kernel<<<grid, kLmThreads, kLmSmem, s>>>(*reinterpret_cast<const CUtensorMap*>(st.a_map),
                                                            *reinterpret_cast<const CUtensorMap*>(st.w_map), P, H, V, m_tiles,
                                                            n_tiles, keys);
    e = cudaGetLastError();
  }
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

}  // namespace asv
