// Sampler of the rollout policy (Eq. 3): temperature, ties-inclusive top-p nucleus, Philox draw,
// inverse CDF in ascending token id -- on quantised integer weights, so the token decision is
// exact integer arithmetic and independent of the order in which threads add things up.
//
//   z_i = logit_i / T (IEEE division);  w_i = floor(exp_nonpos(z_i - max z) * 2^30)
//   total = sum w;  target = (total * floor(top_p*2^24)) >> 24
//   tau  = largest weight value t with S(t) = sum_{w_i >= t} w_i >= target;  mass = S(tau)
//   r = (mass * u24) >> 24;  token = first i (ascending) with w_i >= tau whose running sum > r
//
// tau is found without sorting by a three-level radix select (11 + 10 + 10 bits) over histograms
// of *mass* per bucket.  One CTA of 1024 threads per row.
#pragma once
#include "kernels.cuh"

namespace rpo {

struct SamplerArgs {
  const float* logits;        // [n_logit_rows, V]
  const int32_t* logit_row;   // row r reads logits row logit_row[r] (NULL: r)
  int V;
  float temperature;
  uint32_t top_p24;
  int greedy, eos_id;
  uint64_t seed;
  const int64_t* seq_ids;     // sequence number per row
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

// Bucket holding tau: the highest non-empty bucket b with above + C(b) >= target, C(b) = mass of
// buckets >= b.  hist has 2048 entries; thread t owns buckets 2047-2t and 2046-2t (descending).
// Returns the bucket; *above becomes the mass strictly above it, *at its own mass.
__device__ __forceinline__ int select_bucket(const uint64_t* hist, uint64_t target, uint64_t* above, uint64_t* at,
                                             uint64_t* sh, int* sh_bin) {
  const int t = threadIdx.x, lane = t & 31, wid = t >> 5;
  const int b_hi = 2047 - 2 * t, b_lo = b_hi - 1;
  const uint64_t h_hi = hist[b_hi], h_lo = hist[b_lo];
  const uint64_t incl_w = warp_incl_scan_u64(h_hi + h_lo, lane);
  if (t == 0) *sh_bin = -1;
  __syncthreads();
  if (lane == 31) sh[wid] = incl_w;
  __syncthreads();
  uint64_t base = 0;
  for (int i = 0; i < wid; ++i) base += sh[i];
  const uint64_t excl = *above + base + incl_w - (h_hi + h_lo);   // mass above b_hi (incl. carried-in)
  if (h_hi > 0 && excl + h_hi >= target) atomicMax(sh_bin, b_hi);
  if (h_lo > 0 && excl + h_hi + h_lo >= target) atomicMax(sh_bin, b_lo);
  __syncthreads();
  const int b = *sh_bin;
  __syncthreads();
  if (b == b_hi) { sh[40] = excl; sh[41] = h_hi; }
  if (b == b_lo) { sh[40] = excl + h_hi; sh[41] = h_lo; }
  __syncthreads();
  *above = sh[40];
  *at = sh[41];
  __syncthreads();
  return b;
}

__global__ void __launch_bounds__(1024) sampler_kernel(SamplerArgs a) {
  if (a.step_ptr) { a.step = *a.step_ptr; a.out_col = a.step; a.last_step = (a.step == a.n_steps - 1); }
  __shared__ uint64_t hist[2048];
  __shared__ uint64_t sh[48];
  __shared__ float fred[32];
  __shared__ int sh_bin;
  __shared__ int sh_tok;
  const int r = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
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
  if (a.logits_dbg)
    for (int c = tid; c < V; c += blockDim.x) a.logits_dbg[oidx * V + c] = row[c];

  // pass 1: arg max (lowest id among maxima) on the raw logits
  uint64_t key = 0;
  for (int c = tid; c < V; c += blockDim.x) {
    const uint32_t b = __float_as_uint(row[c]);
    const uint32_t ord = (b & 0x80000000u) ? ~b : (b | 0x80000000u);   // order-preserving map
    const uint64_t k = ((uint64_t)ord << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)c);
    key = k > key ? k : key;
  }
  key = block_max_u64(key, sh);
  const int argmax = (int)(0xFFFFFFFFu - (uint32_t)key);
  const float zmax = __fdiv_rn(row[argmax], a.temperature);

  // pass 2: weights -> total, float sum of exp (for the log-prob), level-1 mass histogram
  for (int i = tid; i < 2048; i += blockDim.x) hist[i] = 0;
  __syncthreads();
  const bool need_nucleus = !a.greedy && !a.forced;
  uint64_t tot = 0;
  float sume = 0.f;
  for (int c = tid; c < V; c += blockDim.x) {
    const float e = exp_nonpos(radd(__fdiv_rn(row[c], a.temperature), -zmax));
    sume += e;
    if (need_nucleus) {
      const uint32_t w = __float2uint_rz(rmul(e, 1073741824.0f));
      tot += w;
      if (w) atomicAdd((unsigned long long*)&hist[w >> 20], (unsigned long long)w);
    }
  }
  sume = block_reduce_sum(sume, fred);
  int tok;
  if (a.forced) {
    tok = min(max(a.forced[oidx], 0), V - 1);
  } else if (a.greedy) {
    tok = argmax;
  } else {
    tot = block_sum_u64(tot, sh);
    const uint64_t target = mul_shift24(tot, a.top_p24);
    uint64_t above = 0, at = 0;
    const int b1 = select_bucket(hist, target, &above, &at, sh, &sh_bin);
    // level 2
    for (int i = tid; i < 2048; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    for (int c = tid; c < V; c += blockDim.x) {
      const uint32_t w = sampler_weight(__fdiv_rn(row[c], a.temperature), zmax);
      if (w && (int)(w >> 20) == b1) atomicAdd((unsigned long long*)&hist[(w >> 10) & 1023], (unsigned long long)w);
    }
    __syncthreads();
    const int b2 = select_bucket(hist, target, &above, &at, sh, &sh_bin);
    // level 3
    for (int i = tid; i < 2048; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const uint32_t pre = ((uint32_t)b1 << 10) | (uint32_t)b2;
    for (int c = tid; c < V; c += blockDim.x) {
      const uint32_t w = sampler_weight(__fdiv_rn(row[c], a.temperature), zmax);
      if (w && (w >> 10) == pre) atomicAdd((unsigned long long*)&hist[w & 1023], (unsigned long long)w);
    }
    __syncthreads();
    const int b3 = select_bucket(hist, target, &above, &at, sh, &sh_bin);
    const uint32_t tau = (pre << 10) | (uint32_t)b3;
    const uint64_t mass = above + at;
    const uint32_t u24 = sampler_u24(a.seed, (uint64_t)a.seq_ids[r], (uint32_t)a.step);
    const uint64_t rdraw = mul_shift24(mass, u24);
    // inverse CDF in ascending id: warp wid owns ids [wid*chunk, (wid+1)*chunk)
    const int chunk = (V + 31) / 32;
    const int c0 = wid * chunk, c1 = min(V, c0 + chunk);
    uint64_t wsum = 0;
    for (int c = c0 + lane; c < c1; c += 32) {
      const uint32_t w = sampler_weight(__fdiv_rn(row[c], a.temperature), zmax);
      if (w >= tau) wsum += w;
    }
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
          const uint32_t wi = sampler_weight(__fdiv_rn(row[c], a.temperature), zmax);
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
    const float lp = radd(__fdiv_rn(row[tok], a.temperature), -zmax) - logf(sume);
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
