// Greedy acceptance with no caller-provided scratch and no allocation: the per-row partial results
// live in a file-scope device array that every GPU loading this library carries until exit.
#include <cstdio>
#include <string>

#include "../../include/as_verify.h"
#include "kernels.cuh"

namespace asv {

namespace {

constexpr int kStaticMaxRows = AS_STATIC_MAX_ROWS;            // query rows (sum of k_i + 1) per call
constexpr int kStaticMaxChunks = 64;                          // vocabulary chunks per row
constexpr int kThreads = 256;

struct Scratch {
  float2 part[kStaticMaxRows * kStaticMaxChunks];                   // (max, index of the lowest maximum) per (row, chunk)
  int32_t row_best[kStaticMaxRows];                           // folded argmax per row
  int32_t ticket[kStaticMaxRows];                             // chunks finished per row; must be zero when a call starts
};

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress; kernels
// receive the device address obtained from it.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(Scratch)];

__device__ __forceinline__ float clean(float x) { return x != x ? -INFINITY : x; }   // NaN never wins
__device__ __forceinline__ bool wins(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// One CTA per (chunk, row): lowest-index maximum of the chunk; the CTA that completes a row folds
// the row's chunks in chunk order.
__global__ void __launch_bounds__(kThreads) static_row_argmax_kernel(Scratch* sc, const float* __restrict__ logits,
                                                                     long long ld, int vocab, int chunk_elems, int chunks) {
  const int row = blockIdx.y, chunk = blockIdx.x;
  const float* z = logits + (size_t)row * ld;
  const int begin = chunk * chunk_elems, end = min(begin + chunk_elems, vocab);
  float bv = -INFINITY;
  int bi = begin;
  for (int i = begin + threadIdx.x; i < end; i += kThreads) {
    const float e = clean(z[i]);
    if (e > bv) {
      bv = e;
      bi = i;
    }
  }
  for (int o = 16; o; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (wins(ov, oi, bv, bi)) {
      bv = ov;
      bi = oi;
    }
  }
  __shared__ float sv[kThreads / 32];
  __shared__ int si[kThreads / 32];
  __shared__ int last;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    sv[warp] = bv;
    si[warp] = bi;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kThreads / 32; ++w)
      if (wins(sv[w], si[w], bv, bi)) {
        bv = sv[w];
        bi = si[w];
      }
    sc->part[(size_t)row * kStaticMaxChunks + chunk] = make_float2(bv, __int_as_float(bi));
    __threadfence();
    last = atomicAdd(&sc->ticket[row], 1) == chunks - 1;
  }
  __syncthreads();
  if (last && threadIdx.x == 0) {
    __threadfence();
    float fv = -INFINITY;
    int fi = 0x7fffffff;
    for (int c = 0; c < chunks; ++c) {
      const float2 p = sc->part[(size_t)row * kStaticMaxChunks + c];
      if (wins(p.x, __float_as_int(p.y), fv, fi)) {
        fv = p.x;
        fi = __float_as_int(p.y);
      }
    }
    sc->row_best[row] = fi;
    sc->ticket[row] = 0;
  }
}

// One warp per request, lane = draft position: longest prefix of drafts that equal their row's argmax.
// cu_q comes from device memory and is not trusted: a request whose entries do not describe 0 <= k <= max_draft rows
// inside [0, total_q) is answered with accept_len 0 and a row of -1 instead of being read.
__global__ void static_decide_kernel(const Scratch* sc, int batch, int total_q, int max_draft, int vocab,
                                     const int32_t* __restrict__ cu_q, const int32_t* __restrict__ draft_tokens,
                                     int32_t* __restrict__ accept_len, int32_t* __restrict__ out_tokens) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= batch) return;
  const int row0 = cu_q[i], k = cu_q[i + 1] - row0 - 1, d0 = row0 - i;   // cu_d[i] = cu_q[i] - i
  int32_t* outs = out_tokens + (size_t)i * (max_draft + 1);
  if (row0 < i || k < 0 || k > max_draft || (long long)row0 + k >= total_q) {
    for (int j = lane; j <= max_draft; j += 32) outs[j] = -1;
    if (lane == 0) accept_len[i] = 0;
    return;
  }
  int a = k;
  for (int j0 = 0; j0 < k && a == k; j0 += 32) {
    const int j = j0 + lane;
    bool ok = true;
    int d = -1;
    if (j < k) {
      d = draft_tokens[d0 + j];
      ok = (unsigned)d < (unsigned)vocab && sc->row_best[row0 + j] == d;
    }
    const unsigned bad = __ballot_sync(0xffffffffu, !ok);
    if (bad) a = j0 + __ffs(bad) - 1;
    if (j < min(a, k)) outs[j] = d;
  }
  for (int j = a + lane; j <= max_draft; j += 32) outs[j] = -1;
  __syncwarp();
  if (lane == 0) {
    outs[a] = sc->row_best[row0 + a];
    accept_len[i] = a;
  }
}

constexpr int kMaxDevices = 64;
Scratch* g_scratch_addr[kMaxDevices];                   // per device, filled on the first call there

}  // namespace

}  // namespace asv

using namespace asv;

extern "C" {

int as_accept_greedy_static(int batch, int total_q, int max_draft, const int32_t* cu_q, const float* logits,
                            int64_t ld, int vocab, const int32_t* draft_tokens, int32_t* accept_len,
                            int32_t* out_tokens, void* stream) {
  auto fail = [](int code, const std::string& msg) { return record_error(code, msg); };   // readable through as_last_error()
  if (batch < 0 || total_q < batch || max_draft < 0 || vocab < 1 || ld < vocab)
    return fail(AS_ERR_INVALID_ARG, "as_accept_greedy_static: need 0 <= batch <= total_q, max_draft >= 0, 1 <= vocab <= ld");
  if (total_q > kStaticMaxRows)
    return fail(AS_ERR_INVALID_ARG, "as_accept_greedy_static: total_q " + std::to_string(total_q) +
                                        " exceeds AS_STATIC_MAX_ROWS " + std::to_string(kStaticMaxRows) +
                                        " (the built-in scratch holds no more rows; use as_accept with a workspace)");
  if (batch == 0) return AS_OK;
  if (!cu_q || !logits || !accept_len || !out_tokens || (total_q > batch && !draft_tokens))
    return fail(AS_ERR_INVALID_ARG, "as_accept_greedy_static: null pointer");
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(AS_ERR_CUDA, std::string("as_accept_greedy_static: cudaGetDevice: ") + cudaGetErrorString(e));
  if (!g_scratch_addr[dev]) {
    // set-up, once per device, with that device current: turn the symbol into a device address
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p)
      return fail(AS_ERR_CUDA, std::string("as_accept_greedy_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    g_scratch_addr[dev] = static_cast<Scratch*>(p);
  }
  Scratch* sc = g_scratch_addr[dev];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left; the tickets are the only part that must start at zero
  e = cudaMemsetAsync(sc->ticket, 0, sizeof(int32_t) * total_q, s);
  if (e != cudaSuccess) return fail(AS_ERR_CUDA, std::string("as_accept_greedy_static: cudaMemsetAsync: ") + cudaGetErrorString(e));
  int chunk = 4096;
  while ((vocab + chunk - 1) / chunk > kStaticMaxChunks) chunk *= 2;
  const int chunks = (vocab + chunk - 1) / chunk;
  static_row_argmax_kernel<<<dim3(chunks, total_q), kThreads, 0, s>>>(sc, logits, ld, vocab, chunk, chunks);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(AS_ERR_CUDA, std::string("as_accept_greedy_static: launch: ") + cudaGetErrorString(e));
  static_decide_kernel<<<(batch + 3) / 4, 128, 0, s>>>(sc, batch, total_q, max_draft, vocab, cu_q, draft_tokens, accept_len, out_tokens);
  e = cudaGetLastError();
  if (e != cudaSuccess) return fail(AS_ERR_CUDA, std::string("as_accept_greedy_static: launch: ") + cudaGetErrorString(e));
  return AS_OK;
}

}  // extern "C"
