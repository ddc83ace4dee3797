// Acceptance over the vocabulary.
//
// Stage 1 (row_stats): the logits are streamed once.  Every CTA takes one chunk of one row and
//   leaves (max, lowest index of the max) and, for a sampling request, the online pair
//   (scaled max, sum of 2^(y - max)) with y = z * log2(e) / T.
//   The CTA that finishes a row last (a ticket counter per row) folds that row's chunk partials in
//   chunk order, so the result does not depend on which CTA that was.
// Stage 2 (decide): one warp per request, lane = draft position: every lane judges its draft against
//   its row's result (greedy: token equality; sampled: u < min(1, p/q)), a ballot finds the first
//   rejection, and greedy requests get their extra token.  Sampling requests record which row must be
//   re-read.
// Stage 3 (recover): a sampling request draws its extra token from max(0, p - q) (or p) by inverse CDF.
//   That row alone is re-read.  Entries are weighed in fp32 (four at a time) and summed in fp64 in index order, so that
//   the chosen index does not depend on how a long fp32 prefix sum would have rounded; the softmax denominator is
//   stage 1's.  Two small launches: the mass of each cell of consecutive entries, spread over the vocabulary chunks
//   so that every SM takes part, then one warp per request walks the cell sums to the cell holding w * S and scans
//   only that.
#include "kernels.cuh"
#include "lm_head.cuh"

namespace asv {

namespace {

constexpr int kStatThreads = 256;
constexpr float kLog2e = 1.4426950408889634f;

struct Best {
  float v;
  int idx;
};
__device__ __forceinline__ Best better(Best a, Best b) {      // greater value wins, ties to the lower index
  return (b.v > a.v || (b.v == a.v && b.idx < a.idx)) ? b : a;
}
__device__ __forceinline__ float clean(float x) { return x != x ? -INFINITY : x; }   // NaN never wins

__device__ __forceinline__ void online(float& m, float& s, float y) {
  if (y > m) {
    s = s * exp2f(m - y) + 1.f;         // m = -inf: s is 0, exp2f(-inf) = 0
    m = y;
  } else if (y > -INFINITY) {
    s += exp2f(y - m);
  }
}
__device__ __forceinline__ void online_merge(float& m, float& s, float m2, float s2) {
  if (m2 == -INFINITY) return;
  if (m == -INFINITY) {
    m = m2;
    s = s2;
    return;
  }
  const float mm = fmaxf(m, m2);
  s = s * exp2f(m - mm) + s2 * exp2f(m2 - mm);
  m = mm;
}

// Folds the chunk partials of one row (all lanes get the result).
__device__ void fold_row(const AcceptArgs& A, int row, int lane, Best& b, float& m, float& s) {
  b = Best{-INFINITY, 0x7fffffff};
  m = -INFINITY;
  s = 0.f;
  for (int ch = lane; ch < A.chunks; ch += 32) {
    const float4 p = A.row_part[(size_t)row * A.chunks + ch];
    b = better(b, Best{p.x, __float_as_int(p.y)});
    online_merge(m, s, p.z, p.w);
  }
  for (int o = 16; o; o >>= 1) {
    Best other{__shfl_xor_sync(0xffffffffu, b.v, o), __shfl_xor_sync(0xffffffffu, b.idx, o)};
    b = better(b, other);
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    online_merge(m, s, m2, s2);
  }
}

__global__ void __launch_bounds__(kStatThreads) row_stats_kernel(DevPlan P, AcceptArgs A) {
  // (one block per (row, chunk), numbered along x: the y dimension of a grid ends at 65535 and a plan may hold more rows)
  const int row = blockIdx.x / A.chunks, chunk = blockIdx.x - row * A.chunks;
  if (row >= P.hdr->total_q) return;                 // the grid may be sized for the plan's maximum
  const int req = P.row_map[row].x;
  const float T = A.temperature ? A.temperature[req] : 0.f;
  const bool sampling = T > 0.f;
  const float c = sampling ? kLog2e / T : 0.f;
  const float* z = A.logits + (size_t)row * A.ld;
  const int begin = chunk * A.chunk_elems;
  const int end = min(begin + A.chunk_elems, A.vocab);
  Best b{-INFINITY, begin};
  float m = -INFINITY, s = 0.f;
  // rows start 16-byte aligned when ld % 4 == 0 and the base is aligned; otherwise scalar loads
  const bool vec = ((reinterpret_cast<uintptr_t>(z + begin) & 15) == 0);
  if (vec) {
    const int n4 = (end - begin) / 4;
    const float4* z4 = reinterpret_cast<const float4*>(z + begin);
    for (int i0 = 0; i0 < n4; i0 += 4 * kStatThreads) {
      float4 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {                    // four independent 16-byte loads in flight per thread
        const int i = i0 + u * kStatThreads + threadIdx.x;
        x[u] = i < n4 ? __ldcs(z4 + i) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
      float e[16];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int at = begin + (i0 + u * kStatThreads + threadIdx.x) * 4;
        e[4 * u] = clean(x[u].x); e[4 * u + 1] = clean(x[u].y); e[4 * u + 2] = clean(x[u].z); e[4 * u + 3] = clean(x[u].w);
#pragma unroll
        for (int v = 0; v < 4; ++v)
          if (e[4 * u + v] > b.v) { b.v = e[4 * u + v]; b.idx = at + v; }
      }
      if (sampling) {
        // the sixteen values join the running (maximum, sum) in one step: their own maximum first, then one
        // 2^x each against the new reference - no branch and no rescaling per element
        float mx = e[0];
#pragma unroll
        for (int v = 1; v < 16; ++v) mx = fmaxf(mx, e[v]);
        const float mnew = fmaxf(m, mx * c);              // c > 0
        if (mnew > -INFINITY) {
          float add = 0.f;
#pragma unroll
          for (int v = 0; v < 16; ++v) add += exp2f(fmaf(e[v], c, -mnew));   // 2^-inf = 0 for absent entries
          s = s * exp2f(m - mnew) + add;                  // m = -inf: s is 0 and 2^-inf = 0
          m = mnew;
        }
      }
    }
    for (int i = begin + n4 * 4 + threadIdx.x; i < end; i += kStatThreads) {
      const float e = clean(z[i]);
      if (e > b.v) { b.v = e; b.idx = i; }
      if (sampling) online(m, s, e * c);
    }
  } else {
    for (int i = begin + threadIdx.x; i < end; i += kStatThreads) {
      const float e = clean(z[i]);
      if (e > b.v) { b.v = e; b.idx = i; }
      if (sampling) online(m, s, e * c);
    }
  }
  // a thread visits ascending indices, so strict '>' already keeps its lowest maximum
  for (int o = 16; o; o >>= 1) {
    Best other{__shfl_xor_sync(0xffffffffu, b.v, o), __shfl_xor_sync(0xffffffffu, b.idx, o)};
    b = better(b, other);
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
    online_merge(m, s, m2, s2);
  }
  __shared__ Best sb[kStatThreads / 32];
  __shared__ float sm[kStatThreads / 32], ss[kStatThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) {
    sb[warp] = b;
    sm[warp] = m;
    ss[warp] = s;
  }
  __syncthreads();
  __shared__ int last;
  if (threadIdx.x == 0) {
    for (int wv = 1; wv < kStatThreads / 32; ++wv) {
      b = better(b, sb[wv]);
      online_merge(m, s, sm[wv], ss[wv]);
    }
    A.row_part[(size_t)row * A.chunks + chunk] = make_float4(b.v, __int_as_float(b.idx), m, s);
    __threadfence();
    last = atomicAdd(&A.row_ticket[row], 1) == A.chunks - 1;
  }
  __syncthreads();
  if (last && warp == 0) {                       // this CTA completed the row: fold its chunks in chunk order
    __threadfence();
    fold_row(A, row, lane, b, m, s);
    if (lane == 0) {
      A.row_final[row] = make_float4(b.v, __int_as_float(b.idx), m, s);
      A.row_ticket[row] = 0;                     // ready for the next call
    }
  }
}

// Philox4x32-10 (Salmon et al., SC 2011): ten rounds of two 32 x 32 -> 64 bit multiplications on a 128-bit
// counter, the key bumped by the Weyl constants each round.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += 0x9E3779B9u;
    k.y += 0xBB67AE85u;
  }
  return c;
}
// The uniforms of a seeded call.  Block (i, b) has counter (i, b, step) and key seed; draft j of request i takes
// word j mod 4 of block (i, j / 4), the request's extra token word 0 of block (i, 2^31); a word x becomes
// (x >> 8) * 2^-24 in [0, 1).
__device__ __forceinline__ float rng_uniform(const uint64_t* rng, int request, uint32_t block, int word) {
  const uint64_t seed = rng[0], step = rng[1];
  const uint4 r = philox4x32_10(make_uint4((uint32_t)request, block, (uint32_t)step, (uint32_t)(step >> 32)),
                                make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
  const uint32_t x = word == 0 ? r.x : word == 1 ? r.y : word == 2 ? r.z : r.w;
  return (float)(x >> 8) * (1.0f / 16777216.0f);
}

__global__ void decide_kernel(DevPlan P, AcceptArgs A) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= P.hdr->batch) return;
  const ReqMeta rq = P.req[i];
  const float T = A.temperature ? A.temperature[i] : 0.f;
  const bool sampling = T > 0.f;
  int32_t* outs = A.out_tokens + (size_t)i * (P.max_draft + 1);
  int a = rq.k;                                        // first rejected position, k if none
  for (int j0 = 0; j0 < rq.k && a == rq.k; j0 += 32) {
    const int j = j0 + lane;
    bool ok = true;
    int d = -1;
    if (j < rq.k) {
      d = A.draft_tokens[rq.cu_d + j];
      const float4 rf = A.row_final[rq.cu_q + j];
      if ((unsigned)d >= (unsigned)A.vocab) {
        atomicOr(P.status, kFlagBadToken);
        ok = false;
      } else if (!sampling) {
        ok = (__float_as_int(rf.y) == d);
      } else {
        const float zd = clean(A.zd ? A.zd[rq.cu_q + j] : A.logits[(size_t)(rq.cu_q + j) * A.ld + d]);
        const float pd = exp2f(zd * (kLog2e / T) - rf.z) / rf.w;
        const float qd = A.draft_probs ? A.draft_probs[(size_t)(rq.cu_d + j) * A.ld + d] : 1.f;
        float ratio;
        if (!(pd > 0.f)) ratio = 0.f;
        else if (!(qd > 0.f)) ratio = 1.f;
        else ratio = fminf(1.f, pd / qd);
        const float uj = A.rng ? rng_uniform(A.rng, i, (uint32_t)j >> 2, j & 3) : A.u[rq.cu_d + j];
        ok = uj < ratio;
      }
    }
    const unsigned bad = __ballot_sync(0xffffffffu, !ok);
    if (bad) a = j0 + __ffs(bad) - 1;
    if (j < min(a, rq.k)) outs[j] = d;                // accepted drafts of this group of 32
  }
  for (int j = a + lane; j <= P.max_draft; j += 32) outs[j] = -1;
  __syncwarp();
  if (lane == 0) {
    if (!sampling) outs[a] = __float_as_int(A.row_final[rq.cu_q + a].y);
    A.accept_len[i] = a;
    A.recover_row[i] = sampling ? a : -1;
  }
}

__device__ __forceinline__ double warp_sum_f64(double v) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
constexpr int kRecThreads = 256;

// What a sampling request needs to know about the row its extra token is drawn from.
struct RecRow {
  const float* z;        // logits row a_i
  const float* q;        // draft distribution to subtract, or nullptr
  int onehot;            // ... or the drafted token when the draft distribution is one-hot, else -1
  float c, mxc;          // log2(e) / T and the row maximum of z times it: 2^(z c - mxc) = exp(z / T - max)
  bool bonus;            // all drafts accepted: draw from p itself
  double den;            // softmax denominator of the row against mxc
};
__device__ __forceinline__ RecRow rec_row(const DevPlan& P, const AcceptArgs& A, int i, int a) {
  const ReqMeta rq = P.req[i];
  RecRow r;
  const int row = rq.cu_q + a;
  r.z = A.rec_logits ? A.rec_logits + (size_t)i * A.rec_ld : A.logits + (size_t)row * A.ld;
  r.bonus = (a == rq.k);
  r.q = (!r.bonus && A.draft_probs) ? A.draft_probs + (size_t)(rq.cu_d + a) * A.ld : nullptr;
  r.onehot = (!r.bonus && !A.draft_probs) ? A.draft_tokens[rq.cu_d + a] : -1;
  // the largest logit of the row is known from the first pass (NaN never wins there either)
  const double c = 1.4426950408889634 / (double)A.temperature[i];
  r.c = (float)c;
  const float4 rf = A.row_final[row];
  r.mxc = (float)((double)rf.x * c);
  // The denominator is the first pass's: the online (reference, sum of 2^(z c - reference)) of the row, moved to this
  // reference (the two references differ by a rounding at most).  An fp32 sum, like the ratio the drafts were judged by.
  r.den = (double)rf.w * (double)exp2f(rf.z - r.mxc);
  return r;
}
// exp(z_v / T - max); 0 for NaN.  One fp32 FMA and the transcendental unit (about 2^-22 relative; the rounding of mxc is
// a common factor of the whole row and cancels in the normalisation): far inside what the fp64 sums and the comparison
// against w * S can resolve.  An fp64 exponential (the library's, then a table and a degree-5 polynomial) and then fp64
// arguments around ex2 kept these kernels bound by fp64 instructions.
__device__ __forceinline__ float rec_exp_f32(const RecRow& r, float x) { return x == x ? exp2f(fmaf(x, r.c, -r.mxc)) : 0.f; }
// p_v and the recovery weight max(0, p_v - q_v) from the logit and the draft probability
__device__ __forceinline__ void rec_weights_val(const RecRow& r, float x, double qv, double inv_den, double& p, double& res) {
  // (fp32 per entry, as in the cell sums this is compared with)
  const float pf = rec_exp_f32(r, x) * (float)inv_den;
  p = (double)pf;
  res = (double)fmaxf(0.f, pf - (float)qv);
}
__device__ __forceinline__ void rec_weights(const RecRow& r, int v, double inv_den, double& p, double& res) {
  const double qv = r.q ? (double)r.q[v] : (v == r.onehot ? 1.0 : 0.0);
  rec_weights_val(r, r.z[v], qv, inv_den, p, res);
}
// Four consecutive entries of a row starting at v (a multiple of 4): one 16-byte load where the address
// allows it, guarded scalar loads otherwise; entries past the vocabulary read as `fill`.
__device__ __forceinline__ float4 load4(const float* row, int v, int V, bool vec, float fill) {
  if (vec && v + 3 < V) return __ldg(reinterpret_cast<const float4*>(row + v));
  float4 o;
  o.x = v < V ? row[v] : fill;
  o.y = v + 1 < V ? row[v + 1] : fill;
  o.z = v + 2 < V ? row[v + 2] : fill;
  o.w = v + 3 < V ? row[v + 3] : fill;
  return o;
}
__device__ __forceinline__ bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
// Recovery, step 1: per cell (cell_elems consecutive vocabulary entries, a multiple of 128) the mass of p and
// of max(0, p - q).  A warp owns whole cells and walks them in strips of 128 entries, four entries per lane,
// four strips' loads in flight; the sums do not depend on the launch shape.
__global__ void __launch_bounds__(kRecThreads) recover_cells_kernel(DevPlan P, AcceptArgs A) {
  const int i = blockIdx.x / A.chunks, chunk = blockIdx.x - i * A.chunks;
  if (i >= P.hdr->batch) return;
  const int a = A.recover_row[i];
  if (a < 0) return;
  const RecRow r = rec_row(P, A, i, a);
  const float inv_den32 = (float)(1.0 / r.den);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kRecThreads / 32;
  const int V = A.vocab;
  const int strips_per_cell = A.cell_elems / 128;
  const int cells_per_chunk = A.chunk_elems / A.cell_elems;
  const int my_cells = (cells_per_chunk - warp + kWarps - 1) / kWarps;     // cells warp, warp + kWarps, ...
  const int my_strips = my_cells * strips_per_cell;
  const bool vz = aligned16(r.z), vq = r.q && aligned16(r.q);
  // first entry this lane reads in the warp's s-th strip, and the cell that strip belongs to
  auto strip_cell = [&](int s) { return chunk * cells_per_chunk + warp + (s / strips_per_cell) * kWarps; };
  auto strip_at = [&](int s) { return strip_cell(s) * A.cell_elems + (s % strips_per_cell) * 128 + lane * 4; };
  double sp = 0.0, sr = 0.0;
  for (int s0 = 0; s0 < my_strips; s0 += 4) {
    float4 x[4], q[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = s0 + u < my_strips ? strip_at(s0 + u) : V;
      x[u] = load4(r.z, v, V, vz, __int_as_float(0x7fc00000));
      q[u] = r.q ? load4(r.q, v, V, vq, 0.f) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int s = s0 + u;
      if (s < my_strips) {
        const int v = strip_at(s);
        // a one-hot draft distribution puts mass 1 on the drafted token
        const float q0 = r.q ? q[u].x : (v == r.onehot ? 1.f : 0.f);
        const float q1 = r.q ? q[u].y : (v + 1 == r.onehot ? 1.f : 0.f);
        const float q2 = r.q ? q[u].z : (v + 2 == r.onehot ? 1.f : 0.f);
        const float q3 = r.q ? q[u].w : (v + 3 == r.onehot ? 1.f : 0.f);
        // Every term carries the transcendental unit's 2^-22 whatever follows, so p = e / den and max(0, p - q) are
        // taken in fp32 and a lane's four entries added there; everything longer is summed in fp64.  (With all of it
        // in fp64 this kernel was bound by fp64 instructions: seven per entry.)
        const float p0 = rec_exp_f32(r, x[u].x) * inv_den32, p1 = rec_exp_f32(r, x[u].y) * inv_den32;
        const float p2 = rec_exp_f32(r, x[u].z) * inv_den32, p3 = rec_exp_f32(r, x[u].w) * inv_den32;
        sp += (double)((p0 + p1) + (p2 + p3));
        sr += (double)((fmaxf(0.f, p0 - q0) + fmaxf(0.f, p1 - q1)) + (fmaxf(0.f, p2 - q2) + fmaxf(0.f, p3 - q3)));
        if ((s + 1) % strips_per_cell == 0) {            // the cell is complete
          const int cell = strip_cell(s);
          sp = warp_sum_f64(sp);
          sr = warp_sum_f64(sr);
          if (lane == 0 && cell < A.cells) {
            double* out = A.rec_cells + ((size_t)i * A.cells + cell) * 2;
            out[0] = sp;
            out[1] = sr;
          }
          sp = 0.0;
          sr = 0.0;
        }
      }
    }
  }
}

// Recovery, step 2: one warp per request walks the cell sums to the cell that holds w * S and scans it.
__global__ void recover_pick_kernel(DevPlan P, AcceptArgs A) {
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= P.hdr->batch) return;
  const int a = A.recover_row[i];
  if (a < 0) return;
  const RecRow r = rec_row(P, A, i, a);
  const double inv_den = 1.0 / r.den;
  const double* cells = A.rec_cells + (size_t)i * A.cells * 2;
  const int ncell = (A.vocab + A.cell_elems - 1) / A.cell_elems;
  const int per = (ncell + 31) / 32;
  const int c0 = min(lane * per, ncell), c1 = min(c0 + per, ncell);   // this lane's run of cells
  double tp = 0.0, tr = 0.0;
  for (int c = c0; c < c1; ++c) {
    tp += cells[2 * c];
    tr += cells[2 * c + 1];
  }
  double ip = tp, ir = tr;                                            // inclusive scans over the lanes
  for (int o = 1; o < 32; o <<= 1) {
    const double up = __shfl_up_sync(0xffffffffu, ip, o), ur = __shfl_up_sync(0xffffffffu, ir, o);
    if (lane >= o) {
      ip += up;
      ir += ur;
    }
  }
  // the residual max(0, p - q), or p itself for a bonus token or when the residual is identically zero
  const bool residual = !r.bonus && __shfl_sync(0xffffffffu, ir, 31) > 0.0;
  const double tot = residual ? tr : tp, incl = residual ? ir : ip;
  const double S = __shfl_sync(0xffffffffu, incl, 31);
  const float wi = A.rng ? rng_uniform(A.rng, i, 0x80000000u, 0) : A.w[P.req[i].cu_q + a];
  const double target = (double)wi * S;
  const double before = incl - tot;
  const unsigned has = __ballot_sync(0xffffffffu, tot > 0.0);
  const unsigned hit = __ballot_sync(0xffffffffu, tot > 0.0 && target < incl);
  int ans = -1;
  if (has) {
    // first lane whose running total passes the target; if rounding left none, the last lane with mass
    const int owner = hit ? __ffs(hit) - 1 : 31 - __clz(has);
    int cell = -1;
    double run = before;
    if (lane == owner) {
      int last = -1;
      double run_last = before;
      for (int c = c0; c < c1 && cell < 0; ++c) {
        const double sc = cells[2 * c + (residual ? 1 : 0)];
        if (sc > 0.0) {
          last = c;
          run_last = run;
          if (target < run + sc) cell = c;
        }
        if (cell < 0) run += sc;
      }
      if (cell < 0) {
        cell = last;
        run = run_last;
      }
    }
    cell = __shfl_sync(0xffffffffu, cell, owner);
    run = __shfl_sync(0xffffffffu, run, owner);
    const int base = cell * A.cell_elems, end = min(base + A.cell_elems, A.vocab);
    int last_pos = -1;
    for (int v0 = base; v0 < end && ans < 0; v0 += 32) {
      const int v = v0 + lane;
      double p = 0.0, res = 0.0;
      if (v < end) rec_weights(r, v, inv_den, p, res);
      const double wv = residual ? res : p;
      double inc = wv;
      for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned pos = __ballot_sync(0xffffffffu, wv > 0.0);
      const unsigned cross = __ballot_sync(0xffffffffu, wv > 0.0 && run + inc > target);
      if (cross) ans = v0 + __ffs(cross) - 1;
      if (pos) last_pos = v0 + 31 - __clz(pos);
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (ans < 0) ans = last_pos;               // the scan's rounding fell just short of the cell total
  }
  if (lane == 0) A.out_tokens[(size_t)i * (P.max_draft + 1) + a] = max(ans, 0);
}

}  // namespace

cudaError_t launch_accept(const DevPlan& P, const AcceptArgs& A, cudaStream_t s) {
  if (P.batch == 0) return cudaSuccess;
  row_stats_kernel<<<(unsigned)A.chunks * (unsigned)P.total_q, kStatThreads, 0, s>>>(P, A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  decide_kernel<<<(P.batch + 3) / 4, 128, 0, s>>>(P, A);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (A.temperature) {
    recover_cells_kernel<<<(unsigned)A.chunks * (unsigned)P.batch, kRecThreads, 0, s>>>(P, A);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    recover_pick_kernel<<<(P.batch + 3) / 4, 128, 0, s>>>(P, A);
    e = cudaGetLastError();
  }
  return e;
}

cudaError_t launch_recover(const DevPlan& P, const AcceptArgs& A, cudaStream_t s) {
  if (P.batch == 0) return cudaSuccess;
  recover_cells_kernel<<<(unsigned)A.chunks * (unsigned)P.batch, kRecThreads, 0, s>>>(P, A);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  recover_pick_kernel<<<(P.batch + 3) / 4, 128, 0, s>>>(P, A);
  return cudaGetLastError();
}

cudaError_t launch_decide(const DevPlan& P, const AcceptArgs& A, cudaStream_t s) {
  if (P.batch == 0) return cudaSuccess;
  decide_kernel<<<(P.batch + 3) / 4, 128, 0, s>>>(P, A);
  return cudaGetLastError();
}

}  // namespace asv
