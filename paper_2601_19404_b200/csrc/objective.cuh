// Forward value of the RPO / GRPO objective for one rollout batch (Section 3.2, Eq. 5-7) with the
// length-aware reward shaping of Section 3.4 (Eq. 11).  One CTA per sampling group, one warp per
// response: group statistics in shared memory, token sums by lanes in a fixed order (reproducible).
#pragma once
#include "kernels.cuh"

namespace rpo {

struct ObjectiveArgs {
  const float* logp_new; const float* logp_old; const float* logp_ref;   // [B, S]; ref may be NULL
  const int32_t* lens; const int32_t* resp_lens;                          // [B]; resp_lens may be NULL (= lens)
  const float* raw_rewards;                                               // [B]
  int G, S;
  float clip_eps, beta, alpha, r_min, r_max;
  int length_shaping;
  float* rewards_out; float* adv_out; float* token_loss_out;              // [B], [B], [B,S] or NULL
  float* group_obj_out;                                                   // [n_groups]
};

constexpr int OBJ_MAX_G = 64;

__global__ void __launch_bounds__(1024) objective_group_kernel(ObjectiveArgs a) {
  pdl_prologue();
  __shared__ float s_R[OBJ_MAX_G], s_A[OBJ_MAX_G], s_seq[OBJ_MAX_G];
  const int g = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, n_warps = blockDim.x >> 5;
  const int b0 = g * a.G;
  // Eq. 11: length-aware rewards (thread i < G), l_ref = mean response length of the group
  if (tid < a.G) {
    float lsum = 0.f;
    for (int i = 0; i < a.G; ++i) lsum += (float)(a.resp_lens ? a.resp_lens[b0 + i] : a.lens[b0 + i]);   // fixed order
    const float l_ref = lsum / (float)a.G;
    const float len = (float)(a.resp_lens ? a.resp_lens[b0 + tid] : a.lens[b0 + tid]);
    float R = a.raw_rewards[b0 + tid];
    if (a.length_shaping) R = fminf(fmaxf(R / (1.0f + expf(-a.alpha * (l_ref - len))), a.r_min), a.r_max);
    s_R[tid] = R;
    a.rewards_out[b0 + tid] = R;
  }
  __syncthreads();
  // Eq. 7: group-relative advantage (population standard deviation; 0 when all rewards are equal)
  if (tid < a.G) {
    float mu = 0.f;
    for (int i = 0; i < a.G; ++i) mu += s_R[i];
    mu /= (float)a.G;
    float var = 0.f;
    for (int i = 0; i < a.G; ++i) var += (s_R[i] - mu) * (s_R[i] - mu);
    const float sd = sqrtf(var / (float)a.G);
    const float A = sd > 0.f ? (s_R[tid] - mu) / sd : 0.f;
    s_A[tid] = A;
    a.adv_out[b0 + tid] = A;
  }
  __syncthreads();
  // Eq. 6 / Eq. 5: clipped token surrogate, minus beta * k3(pi_ref || pi_theta), 1/|o_i| token mean
  for (int i = warp; i < a.G; i += n_warps) {
    const int b = b0 + i, n = a.lens[b];
    const float A = s_A[i];
    float acc = 0.f;
    for (int j0 = 0; j0 < a.S; j0 += 32) {
      const int j = j0 + lane;
      float l = 0.f;
      if (j < n) {
        const int64_t o = (int64_t)b * a.S + j;
        const float ln = a.logp_new[o], r = expf(ln - a.logp_old[o]);
        l = fminf(r * A, fminf(fmaxf(r, 1.0f - a.clip_eps), 1.0f + a.clip_eps) * A);
        if (a.logp_ref && a.beta != 0.f) { const float d = a.logp_ref[o] - ln; l -= a.beta * (expf(d) - d - 1.0f); }
      }
      if (a.token_loss_out && j < a.S) a.token_loss_out[(int64_t)b * a.S + j] = l;
      acc += warp_sum(l);                                   // butterfly: the same order on every run
    }
    if (lane == 0) s_seq[i] = n > 0 ? acc / (float)n : 0.f;
  }
  __syncthreads();
  if (tid == 0) {
    float s = 0.f;
    for (int i = 0; i < a.G; ++i) s += s_seq[i];
    a.group_obj_out[g] = s / (float)a.G;
  }
}

// J = mean over groups, fixed order.
__global__ void objective_reduce_kernel(const float* __restrict__ group_obj, int n_groups, float* __restrict__ out) {
  pdl_prologue();
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    double s = 0.0;
    for (int g = 0; g < n_groups; ++g) s += (double)group_obj[g];
    out[0] = (float)(s / (double)n_groups);
  }
}

}  // namespace rpo
