// Verify attention, portable SIMT kernel (fp32 FMA), and the split-KV merge.
//
// One CTA walks its share of the work list.  For an item (request, kv-head, key range) the
// R = G * (k + 1) query rows that share the KV head (row r = j * G + g) sit in shared memory;
// keys are staged 32 at a time through the block table; warp w owns rows w, w + 8, ... and runs
// the online softmax of a row with lane = key, reducing max and sum with warp shuffles; the output
// accumulator of a row lives in shared memory with lane = slice of the head dimension.
#include "kernels.cuh"

namespace asv {

namespace {

constexpr int kSimtThreads = 256;
constexpr int kSimtWarps = kSimtThreads / 32;
constexpr int kSimtTile = 32;

__device__ __forceinline__ float warp_max(float v) {
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D>
__global__ void __launch_bounds__(kSimtThreads) attn_simt_kernel(DevPlan P, AttnArgs A) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int KSTRIDE = D + 2;            // padded so that lane = key reads hit distinct banks
  constexpr int DPL = D / 32;               // output columns per lane
  const int G = P.Hq / P.Hkv;
  const int rows_max = G * (P.max_draft + 1);
  __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem_raw);                    // [rows_max][D]
  __nv_bfloat16* Ks = Qs + (size_t)rows_max * D;                                     // [32][D + 2]
  __nv_bfloat16* Vs = Ks + kSimtTile * KSTRIDE;                                      // [32][D]
  float* Os = reinterpret_cast<float*>(Vs + kSimtTile * D);                          // [rows_max][D]
  float* Ms = Os + (size_t)rows_max * D;                                             // [rows_max]
  float* Ls = Ms + rows_max;                                                         // [rows_max]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float NEG_INF = -INFINITY;

  for (int it = A.cta_first[blockIdx.x]; it < A.cta_first[blockIdx.x + 1]; ++it) {
    const WorkItem w = A.items[it];
    const ReqMeta rq{w.n, w.k, w.cu_q, 0};  // (the item's own view of its request: a row block of it, or all of it)
    const int R = G * (rq.k + 1);
    __syncthreads();                        // previous item fully written out before smem is reused
    for (int x = tid; x < R * (D / 8); x += kSimtThreads) {
      const int r = x / (D / 8), c = x % (D / 8);
      const int j = r / G, g = r % G;
      const uint4 v = *reinterpret_cast<const uint4*>(
          A.q + ((size_t)(rq.cu_q + j) * P.Hq + w.kv_head * G + g) * D + c * 8);
      *reinterpret_cast<uint4*>(Qs + (size_t)r * D + c * 8) = v;
    }
    for (int x = tid; x < R * D; x += kSimtThreads) Os[x] = 0.f;
    for (int x = tid; x < R; x += kSimtThreads) {
      Ms[x] = NEG_INF;
      Ls[x] = 0.f;
    }
    const int32_t* bt = A.block_table + (size_t)w.req * P.max_blocks;

    for (int t0 = w.key_begin; t0 < w.key_end; t0 += kSimtTile) {
      __syncthreads();
      for (int x = tid; x < kSimtTile * (D / 8); x += kSimtThreads) {
        const int kk = x / (D / 8), c = x % (D / 8);
        const int t = t0 + kk;
        uint4 kv = make_uint4(0, 0, 0, 0), vv = kv;
        if (t < w.key_end) {
          const int blk = bt[t / P.bs];
          if ((unsigned)blk < (unsigned)P.num_blocks) {
            const size_t src = (((size_t)blk * P.Hkv + w.kv_head) * P.bs + (t % P.bs)) * D + c * 8;
            kv = *reinterpret_cast<const uint4*>(A.k_pool + src);
            vv = *reinterpret_cast<const uint4*>(A.v_pool + src);
          } else {
            atomicOr(P.status, kFlagBadPage);
          }
        }
        uint32_t* kd = reinterpret_cast<uint32_t*>(Ks + kk * KSTRIDE + c * 8);
        kd[0] = kv.x; kd[1] = kv.y; kd[2] = kv.z; kd[3] = kv.w;
        *reinterpret_cast<uint4*>(Vs + kk * D + c * 8) = vv;
      }
      __syncthreads();
      const int t = t0 + lane;
      for (int r = warp; r < R; r += kSimtWarps) {
        const int p = rq.n + r / G;
        const int lo = A.window > 0 ? max(0, p - A.window + 1) : 0;
        if (t0 > p || t0 + kSimtTile <= lo) continue;            // tile wholly invisible to this row
        const bool valid = t < w.key_end && t <= p && t >= lo;
        float acc = 0.f;
        const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(Qs + (size_t)r * D);
        const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(Ks + lane * KSTRIDE);
#pragma unroll 8
        for (int d = 0; d < D / 2; ++d) {
          const float2 a = __bfloat1622float2(q2[d]), b = __bfloat1622float2(k2[d]);
          acc = fmaf(a.x, b.x, acc);
          acc = fmaf(a.y, b.y, acc);
        }
        const float s = valid ? acc * A.scale_log2 : NEG_INF;
        const float m_old = Ms[r];
        const float m_new = fmaxf(m_old, warp_max(s));
        if (m_new == NEG_INF) continue;
        const float pr = valid ? exp2f(s - m_new) : 0.f;
        const float alpha = exp2f(m_old - m_new);                // 0 when m_old = -inf
        const float psum = warp_sum(pr);
        float o[DPL];
#pragma unroll
        for (int c = 0; c < DPL; ++c) o[c] = Os[(size_t)r * D + lane * DPL + c] * alpha;
        for (int kk = 0; kk < kSimtTile; ++kk) {
          const float pk = __shfl_sync(0xffffffffu, pr, kk);
          const __nv_bfloat16* vrow = Vs + kk * D + lane * DPL;
#pragma unroll
          for (int c = 0; c < DPL; c += 2) {
            const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vrow + c));
            o[c] = fmaf(pk, v.x, o[c]);
            o[c + 1] = fmaf(pk, v.y, o[c + 1]);
          }
        }
#pragma unroll
        for (int c = 0; c < DPL; ++c) Os[(size_t)r * D + lane * DPL + c] = o[c];
        if (lane == 0) {
          Ms[r] = m_new;
          Ls[r] = Ls[r] * alpha + psum;
        }
        __syncwarp();
      }
    }
    __syncthreads();
    // epilogue: final output (with the sink term) or the unnormalised partial
    for (int r = warp; r < R; r += kSimtWarps) {
      const int j = r / G, g = r % G, h = w.kv_head * G + g;
      float m = Ms[r], l = Ls[r];
      if (w.part_row >= 0) {
        for (int c = 0; c < DPL; ++c)
          A.part_o[(size_t)(w.part_row + r) * D + lane * DPL + c] = Os[(size_t)r * D + lane * DPL + c];
        if (lane == 0) A.part_ml[w.part_row + r] = make_float2(m, l);
        continue;
      }
      float scale = 1.f;
      if (A.sinks) {
        const float sk = A.sinks[h] * 1.4426950408889634f;
        const float m2 = fmaxf(m, sk);
        scale = exp2f(m - m2);
        l = l * scale + exp2f(sk - m2);
        m = m2;
      }
      const float inv = scale / l;
      __nv_bfloat16* dst = A.out + ((size_t)(rq.cu_q + j) * P.Hq + h) * D + lane * DPL;
#pragma unroll
      for (int c = 0; c < DPL; c += 2)
        *reinterpret_cast<__nv_bfloat162*>(dst + c) = __floats2bfloat162_rn(
            Os[(size_t)r * D + lane * DPL + c] * inv, Os[(size_t)r * D + lane * DPL + c + 1] * inv);
      if (A.lse && lane == 0) A.lse[(size_t)(rq.cu_q + j) * P.Hq + h] = (m + log2f(l)) * 0.6931471805599453f;
    }
  }
}

// Split-KV merge: one warp per (cut pair, query row); lane = 4 (D = 128) or 2 (D = 64) output columns.
//   out = sum_s 2^(m_s - m) O_s / (sum_s 2^(m_s - m) l_s + sink term), parts in plan order.
template <int DPL>
__global__ void __launch_bounds__(128) attn_merge_kernel(DevPlan P, AttnArgs A) {
  if ((int)blockIdx.x >= *A.num_merges_dev) return;     // the grid may be sized for the plan's maximum
  const MergeSeg sg = A.merges[blockIdx.x];
  const int G = P.Hq / P.Hkv;
  const int R = G * (sg.k + 1);                         // (the pair's own rows: a row block of its request, or all of it)
  const int r = blockIdx.y * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= R) return;
  constexpr int D = DPL * 32;
  const int j = r / G, h = sg.kv_head * G + r % G;
  float m = -INFINITY;
  for (int s = 0; s < sg.num_parts; ++s) m = fmaxf(m, A.part_ml[sg.part_row + s * R + r].x);
  const float sk = A.sinks ? A.sinks[h] * 1.4426950408889634f : -INFINITY;
  m = fmaxf(m, sk);
  float l = 0.f, o[DPL];
#pragma unroll
  for (int c = 0; c < DPL; ++c) o[c] = 0.f;
  for (int s = 0; s < sg.num_parts; ++s) {
    const float2 ml = A.part_ml[sg.part_row + s * R + r];
    const float sc = ml.x == -INFINITY ? 0.f : exp2f(ml.x - m);
    l = fmaf(sc, ml.y, l);
    const float* src = A.part_o + (size_t)(sg.part_row + s * R + r) * D + lane * DPL;
    if (DPL == 4) {
      const float4 v = *reinterpret_cast<const float4*>(src);
      o[0] = fmaf(sc, v.x, o[0]); o[1] = fmaf(sc, v.y, o[1]); o[2] = fmaf(sc, v.z, o[2]); o[3] = fmaf(sc, v.w, o[3]);
    } else {
      const float2 v = *reinterpret_cast<const float2*>(src);
      o[0] = fmaf(sc, v.x, o[0]); o[1] = fmaf(sc, v.y, o[1]);
    }
  }
  if (A.sinks) l += exp2f(sk - m);
  const float inv = 1.f / l;
  __nv_bfloat16* dst = A.out + ((size_t)(sg.cu_q + j) * P.Hq + h) * D + lane * DPL;
#pragma unroll
  for (int c = 0; c < DPL; c += 2) *reinterpret_cast<__nv_bfloat162*>(dst + c) = __floats2bfloat162_rn(o[c] * inv, o[c + 1] * inv);
  if (A.lse && lane == 0) A.lse[(size_t)(sg.cu_q + j) * P.Hq + h] = (m + log2f(l)) * 0.6931471805599453f;
}

}  // namespace

size_t attn_simt_smem_bytes(int rows, int D) {
  return (size_t)rows * D * 2 + kSimtTile * (D + 2) * 2 + kSimtTile * D * 2 + (size_t)rows * D * 4 + rows * 8;
}

cudaError_t launch_attn_simt(const DevPlan& P, const AttnArgs& A, cudaStream_t s) {
  if (A.num_ctas == 0) return cudaSuccess;
  const int rows = (P.Hq / P.Hkv) * (P.max_draft + 1);
  const size_t smem = attn_simt_smem_bytes(rows, P.D);
  cudaError_t e;
  if (P.D == 128) {
    e = cudaFuncSetAttribute(attn_simt_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_simt_kernel<128><<<A.num_ctas, kSimtThreads, smem, s>>>(P, A);
  } else {
    e = cudaFuncSetAttribute(attn_simt_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_simt_kernel<64><<<A.num_ctas, kSimtThreads, smem, s>>>(P, A);
  }
  return cudaGetLastError();
}

cudaError_t launch_attn_merge(const DevPlan& P, const AttnArgs& A, cudaStream_t s) {
  if (A.num_merges == 0) return cudaSuccess;
  const dim3 grid(A.num_merges, ((P.Hq / P.Hkv) * (P.max_draft + 1) + 3) / 4);
  if (P.D == 128) attn_merge_kernel<4><<<grid, 128, 0, s>>>(P, A);
  else attn_merge_kernel<2><<<grid, 128, 0, s>>>(P, A);
  return cudaGetLastError();
}

}  // namespace asv
