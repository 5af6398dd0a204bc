// Sampler of the rollout policy (Eq. 3): temperature, ties-inclusive top-p nucleus, Philox draw,
// inverse CDF in ascending token id -- on quantised integer weights, so the token decision is
// exact integer arithmetic and independent of the order in which threads add things up.
//
//   z_i = logit_i / T (IEEE division);  w_i = floor(exp_nonpos(z_i - max z) * 2^30)
//   total = sum w;  target = (total * floor(top_p*2^24)) >> 24
//   tau  = largest weight value t with S(t) = sum_{w_i >= t} w_i >= target;  mass = S(tau)
//   r = (mass * u24) >> 24;  token = first i (ascending) with w_i >= tau whose running sum > r
//
// tau is found without sorting by a three-level radix select (8 + 11 + 12 bits) over histograms
// of *mass* per bucket.  One CTA of 1024 threads per row; the weights are computed once, parked in
// a scratch row (L2-resident) and re-read by the select and inverse-CDF passes.
#pragma once
#include "kernels.cuh"

namespace rpo {

struct SamplerArgs {
  const float* logits;        // [n_logit_rows, V]
  uint32_t* weights;          // scratch [n_rows, V]: quantised weights of the row being sampled
  const int32_t* logit_row;   // row r reads logits row logit_row[r] (NULL: r)
  int V;
  float temperature;
  uint32_t top_p24;
  int greedy, eos_id;
  uint64_t seed;
  const int64_t* seq_ids;     // sequence number per row
  int row_base;               // first row of this launch (rows beyond the scratch capacity run in chunks)
  int step;                   // draw number (suffix position)
  const int32_t* step_ptr;    // non-NULL (decode): step, out_col and last_step come from this device counter
  int n_steps;                // with step_ptr: the call's number of suffix positions
  int out_stride, out_col;    // outputs land at [r*out_stride + out_col]
  const int32_t* forced;      // NULL or forced tokens, same indexing as outputs
  int32_t* tokens_out;
  float* logprobs_out;        // nullable
  int32_t* done;              // nullable decode state, per row
  int32_t* lens;
  int32_t* cur_tok;
  int32_t* row_t;
  int last_step;              // no forward follows this step
  float* logits_dbg;          // nullable [n_rows*out_stride*V]
};

__device__ __forceinline__ uint64_t mul_shift24(uint64_t a, uint32_t b) {  // (a*b) >> 24, a < 2^64, b <= 2^24
  const uint64_t lo = a * (uint64_t)b, hi = __umul64hi(a, (uint64_t)b);
  return (hi << 40) | (lo >> 24);
}

__device__ __forceinline__ uint64_t warp_incl_scan_u64(uint64_t v, int lane) {
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint64_t n = __shfl_up_sync(0xffffffffu, v, o);
    if (lane >= o) v += n;
  }
  return v;
}

// Block-wide reductions for 1024 threads (32 warps); `sh` holds >= 33 uint64.
__device__ __forceinline__ uint64_t block_sum_u64(uint64_t v, uint64_t* sh) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sh[wid] = v;
  __syncthreads();
  uint64_t t = 0;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += sh[i];
  __syncthreads();
  return t;
}
__device__ __forceinline__ uint64_t block_max_u64(uint64_t v, uint64_t* sh) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { const uint64_t n = __shfl_xor_sync(0xffffffffu, v, o); v = n > v ? n : v; }
  __syncthreads();
  if (lane == 0) sh[wid] = v;
  __syncthreads();
  uint64_t t = 0;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t = sh[i] > t ? sh[i] : t;
  __syncthreads();
  return t;
}

// Shared-memory histograms of *mass* per bucket.  A 64-bit shared atomic is a compare-and-swap
// loop, so masses are kept as 32-bit sums of pieces of the weights (exact for vocabularies < 2^18).
//
// Level 1 sees every element of the row, and on a flat distribution most of them fall into a few
// dozen neighbouring buckets: lanes of a warp would collide on addresses and banks.  Its histogram
// is therefore private per lane, [256 buckets][32 lanes]: word (b, lane) sits in bank `lane`, so
// a warp's atomics never conflict, and each word sums at most V/32 < 2^13 sixteen-bit pieces.
struct LaneHist {                         // 64 KB
  uint32_t lo[256 * 32], hi[256 * 32];
  __device__ __forceinline__ void clear(int tid, int n) {
    for (int i = tid; i < 256 * 32; i += n) { lo[i] = 0; hi[i] = 0; }
  }
  __device__ __forceinline__ void add(int bucket, int lane, uint32_t w) {
    atomicAdd(&lo[bucket * 32 + lane], w & 0xFFFFu);
    atomicAdd(&hi[bucket * 32 + lane], w >> 16);
  }
  __device__ __forceinline__ uint64_t mass(int bucket, int skew) const {   // skewed: no bank conflicts
    uint64_t l = 0, h = 0;
#pragma unroll 8
    for (int i = 0; i < 32; ++i) { const int j = (i + skew) & 31; l += lo[bucket * 32 + j]; h += hi[bucket * 32 + j]; }
    return l + (h << 16);
  }
};
// Levels 2 and 3 see only the elements of one bucket of the level above: plain [NB] histograms of
// three 14-bit pieces.
template <int NB>
struct PieceHist {
  uint32_t p0[NB], p1[NB], p2[NB];
  __device__ __forceinline__ void clear(int tid, int n) {
    for (int i = tid; i < NB; i += n) { p0[i] = 0; p1[i] = 0; p2[i] = 0; }
  }
  __device__ __forceinline__ void add(int bucket, uint32_t w) {
    atomicAdd(&p0[bucket], w & 0x3FFFu);
    atomicAdd(&p1[bucket], (w >> 14) & 0x3FFFu);
    if (w >> 28) atomicAdd(&p2[bucket], w >> 28);
  }
  __device__ __forceinline__ uint64_t mass(int bucket) const {
    return (uint64_t)p0[bucket] + ((uint64_t)p1[bucket] << 14) + ((uint64_t)p2[bucket] << 28);
  }
};

// Bucket holding tau among nb buckets: the highest non-empty bucket b with above + C(b) >= target,
// C(b) = mass of this level's buckets >= b.  Thread t owns the K buckets nb-1-(t*K+i), descending.
// Returns the bucket; *above becomes the mass strictly above it, *at its own mass.
template <int K, typename MassFn>
__device__ __forceinline__ int select_bucket(int nb, MassFn mass, uint64_t target, uint64_t* above, uint64_t* at,
                                             uint64_t* sh, int* sh_bin) {
  const int t = threadIdx.x, lane = t & 31, wid = t >> 5;
  uint64_t m[K], loc = 0;
#pragma unroll
  for (int i = 0; i < K; ++i) {
    const int b = nb - 1 - (t * K + i);
    m[i] = (b >= 0) ? mass(b) : 0;
    loc += m[i];
  }
  const uint64_t incl_w = warp_incl_scan_u64(loc, lane);
  if (t == 0) *sh_bin = -1;
  __syncthreads();
  if (lane == 31) sh[wid] = incl_w;
  __syncthreads();
  uint64_t base = 0;
  for (int i = 0; i < wid; ++i) base += sh[i];
  const uint64_t first = *above + base + incl_w - loc;     // mass above this thread's first bucket
  uint64_t run = first;
#pragma unroll
  for (int i = 0; i < K; ++i) {
    const int b = nb - 1 - (t * K + i);
    if (b >= 0 && m[i] > 0 && run + m[i] >= target) atomicMax(sh_bin, b);
    run += m[i];
  }
  __syncthreads();
  const int sel = *sh_bin;
  __syncthreads();
  run = first;
#pragma unroll
  for (int i = 0; i < K; ++i) {
    if (nb - 1 - (t * K + i) == sel) { sh[40] = run; sh[41] = m[i]; }
    run += m[i];
  }
  __syncthreads();
  *above = sh[40];
  *at = sh[41];
  __syncthreads();
  return sel;
}

// Row-scan helper: calls f(c, v) for every column c of a row of n 32-bit words.  Where the row is
// 16-byte aligned it issues four independent 128-bit loads per thread before using any of them, so
// that one CTA keeps 64 KB in flight (a scan is latency-bound otherwise).  All threads take part.
template <typename V4, typename T, typename F>
__device__ __forceinline__ void scan_row(const T* __restrict__ row, int n, int t0, int stride, F f) {
  if ((((uintptr_t)row) & 15) == 0) {
    const int n4 = n >> 2;
    const V4* r4 = (const V4*)row;
    int i = t0;
    for (; i + 3 * stride < n4; i += 4 * stride) {
      const V4 v0 = r4[i], v1 = r4[i + stride], v2 = r4[i + 2 * stride], v3 = r4[i + 3 * stride];
      f(4 * i, v0.x); f(4 * i + 1, v0.y); f(4 * i + 2, v0.z); f(4 * i + 3, v0.w);
      const int i1 = i + stride, i2 = i + 2 * stride, i3 = i + 3 * stride;
      f(4 * i1, v1.x); f(4 * i1 + 1, v1.y); f(4 * i1 + 2, v1.z); f(4 * i1 + 3, v1.w);
      f(4 * i2, v2.x); f(4 * i2 + 1, v2.y); f(4 * i2 + 2, v2.z); f(4 * i2 + 3, v2.w);
      f(4 * i3, v3.x); f(4 * i3 + 1, v3.y); f(4 * i3 + 2, v3.z); f(4 * i3 + 3, v3.w);
    }
    for (; i < n4; i += stride) {
      const V4 v = r4[i];
      f(4 * i, v.x); f(4 * i + 1, v.y); f(4 * i + 2, v.z); f(4 * i + 3, v.w);
    }
    for (int c = (n4 << 2) + t0; c < n; c += stride) f(c, row[c]);
  } else {
    for (int c = t0; c < n; c += stride) f(c, row[c]);
  }
}

constexpr int SAMPLER_SMEM = 64 * 1024;

__global__ void __launch_bounds__(1024) sampler_kernel(SamplerArgs a) {
  pdl_prologue();
  if (a.step_ptr) { a.step = *a.step_ptr; a.out_col = a.step; a.last_step = (a.step == a.n_steps - 1); }
  extern __shared__ __align__(16) uint8_t sampler_smem[];   // SAMPLER_SMEM bytes: the level histograms, in turn
  LaneHist& h1 = *reinterpret_cast<LaneHist*>(sampler_smem);
  PieceHist<2048>& h2 = *reinterpret_cast<PieceHist<2048>*>(sampler_smem);
  PieceHist<4096>& h3 = *reinterpret_cast<PieceHist<4096>*>(sampler_smem);
  __shared__ uint64_t sh[48];
  __shared__ float fred[32];
  __shared__ int sh_bin;
  __shared__ int sh_tok;
  const int r = blockIdx.x + a.row_base, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int64_t oidx = (int64_t)r * a.out_stride + a.out_col;
  if (a.done && a.done[r]) {
    if (tid == 0) {
      a.tokens_out[oidx] = a.eos_id;
      if (a.logprobs_out) a.logprobs_out[oidx] = 0.f;
      if (a.row_t) a.row_t[r] = -1;
    }
    return;
  }
  const int V = a.V;
  const float* row = a.logits + (int64_t)(a.logit_row ? a.logit_row[r] : r) * V;
  uint32_t* wrow = a.weights + (int64_t)blockIdx.x * V;   // this row's quantised weights (scratch)
  const float T = a.temperature;
  const bool unit_T = (T == 1.0f);                  // x / 1 == x exactly: skip the division
  if (a.logits_dbg)
    for (int c = tid; c < V; c += blockDim.x) a.logits_dbg[oidx * V + c] = row[c];

  // pass 1: arg max (lowest id among maxima) on the raw logits.  A thread meets its columns in
  // ascending order, so a strict comparison keeps its lowest maximal id; threads are then merged
  // on (order-preserving value bits, inverted id).
  float best = -INFINITY; int best_c = 0x7FFFFFFF;
  scan_row<float4>(row, V, tid, blockDim.x, [&](int c, float x) {
    const bool up = (x > best) || (x == best && c < best_c);
    best = up ? x : best; best_c = up ? c : best_c;
  });
  uint64_t key = 0;
  if (best_c != 0x7FFFFFFF) {
    const uint32_t b = __float_as_uint(best + 0.0f);   // -0 -> +0: equal values must compare equal
    const uint32_t ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);
    key = ((uint64_t)ord << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)best_c);
  }
  key = block_max_u64(key, sh);
  const int argmax = (int)(0xFFFFFFFFu - (uint32_t)key);
  const float zmax = unit_T ? row[argmax] : __fdiv_rn(row[argmax], T);

  // pass 2: weights (kept in scratch for the later passes) -> total, float sum of exp (for the
  // log-prob), level-1 mass histogram (digit w >> 23)
  h1.clear(tid, blockDim.x);
  __syncthreads();
  const bool need_nucleus = !a.greedy && !a.forced;
  uint64_t tot = 0;
  float sume = 0.f;
  scan_row<float4>(row, V, tid, blockDim.x, [&](int c, float x) {
    const float e = exp_nonpos(radd(unit_T ? x : __fdiv_rn(x, T), -zmax));
    sume += e;
    if (need_nucleus) {
      const uint32_t w = __float2uint_rz(rmul(e, 1073741824.0f));
      wrow[c] = w;
      tot += w;
      if (w) h1.add(w >> 23, lane, w);
    }
  });
  sume = block_reduce_sum(sume, fred);
  int tok;
  if (a.forced) {
    tok = min(max(a.forced[oidx], 0), V - 1);
  } else if (a.greedy) {
    tok = argmax;
  } else {
    tot = block_sum_u64(tot, sh);                   // (its barriers also publish wrow to the CTA)
    const uint64_t target = mul_shift24(tot, a.top_p24);
    uint64_t above = 0, at = 0;
    const int b1 = select_bucket<1>(256, [&](int b) { return h1.mass(b, tid); }, target, &above, &at, sh, &sh_bin);
    // level 2: digit (w >> 12) & 2047 of the elements in bucket b1
    h2.clear(tid, blockDim.x);
    __syncthreads();
    scan_row<uint4>(wrow, V, tid, blockDim.x, [&](int c, uint32_t w) {
      if (w && (int)(w >> 23) == b1) h2.add((w >> 12) & 2047, w);
    });
    __syncthreads();
    const int b2 = select_bucket<2>(2048, [&](int b) { return h2.mass(b); }, target, &above, &at, sh, &sh_bin);
    // level 3: digit w & 4095
    h3.clear(tid, blockDim.x);
    __syncthreads();
    const uint32_t pre = ((uint32_t)b1 << 11) | (uint32_t)b2;
    scan_row<uint4>(wrow, V, tid, blockDim.x, [&](int c, uint32_t w) {
      if (w && (w >> 12) == pre) h3.add(w & 4095, w);
    });
    __syncthreads();
    const int b3 = select_bucket<4>(4096, [&](int b) { return h3.mass(b); }, target, &above, &at, sh, &sh_bin);
    const uint32_t tau = (pre << 12) | (uint32_t)b3;
    const uint64_t mass = above + at;
    const uint32_t u24 = sampler_u24(a.seed, (uint64_t)a.seq_ids[r], (uint32_t)a.step);
    const uint64_t rdraw = mul_shift24(mass, u24);
    // inverse CDF in ascending id: warp wid owns ids [wid*chunk, (wid+1)*chunk)
    const int chunk = (((V + 31) / 32) + 3) & ~3;
    const int c0 = min(V, wid * chunk), c1 = min(V, c0 + chunk);
    uint64_t wsum = 0;
    scan_row<uint4>(wrow + c0, c1 - c0, lane, 32, [&](int c, uint32_t w) { if (w >= tau) wsum += w; });
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
    if (tid == 0) sh_tok = -1;
    __syncthreads();
    if (lane == 0) sh[wid] = wsum;
    __syncthreads();
    uint64_t base = 0;
    for (int i = 0; i < wid; ++i) base += sh[i];
    if (rdraw >= base && rdraw < base + wsum) {         // exactly one warp
      uint64_t run = base;
      for (int cb = c0; cb < c1; cb += 32) {
        const int c = cb + lane;
        uint64_t w = 0;
        if (c < c1) {
          const uint32_t wi = wrow[c];
          if (wi >= tau) w = wi;
        }
        const uint64_t incl = warp_incl_scan_u64(w, lane);
        const unsigned hit = __ballot_sync(0xffffffffu, run + incl > rdraw);
        if (hit) { if (lane == 0) sh_tok = cb + (__ffs(hit) - 1); break; }
        run += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    __syncthreads();
    tok = sh_tok;
    if (tok < 0) tok = argmax;   // unreachable when mass > 0; keeps the output defined
  }
  if (tid == 0) {
    const float lp = radd(unit_T ? row[tok] : __fdiv_rn(row[tok], T), -zmax) - logf(sume);
    a.tokens_out[oidx] = tok;
    if (a.logprobs_out) a.logprobs_out[oidx] = lp;
    if (a.lens) a.lens[r] = a.step + 1;
    const bool stop = (tok == a.eos_id);
    if (a.done && stop) a.done[r] = 1;
    if (a.cur_tok) a.cur_tok[r] = tok;
    if (a.row_t) a.row_t[r] = (stop || a.last_step) ? -1 : a.step;
  }
}

}  // namespace rpo
