// Plain CUDA-core GEMM and attention.  They carry the float32 configuration (no tensor-core
// rounding, so tolerances stay tight) and serve as the always-correct alternative of the bf16
// tensor-core kernels in kernel-level tests.
#pragma once
#include "kernels.cuh"

namespace rpo {

enum GemmEpilogue { EPI_STORE_T = 0, EPI_STORE_F32 = 1, EPI_ADD_F32 = 2, EPI_SWIGLU = 3 };

// C[M,N] (+)= A[M,K] * W[N,K]^T.  64x64 tile, 16-deep K slices, 4x4 outputs per thread.
template <typename T, int EPI>
__global__ void __launch_bounds__(256) gemm_ref_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                       void* __restrict__ Cv, int M, int N, int K, int64_t ldc) {
  pdl_prologue();
  __shared__ float sA[16][64 + 4];
  __shared__ float sW[16][64 + 4];
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int i = threadIdx.x; i < 64 * 16; i += 256) {
      const int rr = i / 16, kk = i % 16;
      const int gm = m0 + rr, gn = n0 + rr, gk = k0 + kk;
      sA[kk][rr] = (gm < M && gk < K) ? to_f32(A[(int64_t)gm * K + gk]) : 0.f;
      sW[kk][rr] = (gn < N && gk < K) ? to_f32(W[(int64_t)gn * K + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sA[kk][ty * 4 + i]; b[i] = sW[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      const int64_t o = (int64_t)gm * ldc + gn;
      if (EPI == EPI_STORE_T) ((T*)Cv)[o] = from_f32<T>(acc[i][j]);
      else if (EPI == EPI_STORE_F32) ((float*)Cv)[o] = acc[i][j];
      else ((float*)Cv)[o] += acc[i][j];
    }
  }
}

// Attention of one (row, query head) per warp over [shared segment, all visible] ++ [private
// segment, keys 0..t].  Lanes own head_dim/32 consecutive dimensions; online softmax in float32.
// q is read from the fused qkv buffer (already rotated); output [rows, Hq*dh].
template <typename T, int DH>
__global__ void __launch_bounds__(128) attn_ref_kernel(const T* __restrict__ qkv, T* __restrict__ out,
                                                       const int32_t* __restrict__ row_seq,
                                                       const int32_t* __restrict__ row_t,
                                                       const SeqDesc* __restrict__ seqs,
                                                       const int32_t* __restrict__ block_table, KVPool<T> pool,
                                                       int layer, int rows, int hq, int hkv, float scale,
                                                       int* status) {
  pdl_prologue();
  constexpr int DPL = DH / 32;
  const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (w >= rows * hq) return;
  const int r = w / hq, head = w % hq;
  T* o = out + (int64_t)r * hq * DH + head * DH + lane * DPL;
  const int t = row_t[r];
  if (t < 0) {
#pragma unroll
    for (int i = 0; i < DPL; ++i) o[i] = from_f32<T>(0.f);
    return;
  }
  const SeqDesc sd = seqs[row_seq[r]];
  const int kvh = head / (hq / hkv);
  const T* qp = qkv + (int64_t)r * (hq + 2 * hkv) * DH + head * DH + lane * DPL;
  float q[DPL], acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) { q[i] = to_f32(qp[i]) * scale; acc[i] = 0.f; }
  float m = -INFINITY, l = 0.f;
  const int n_shared = (sd.shared_tbl >= 0) ? sd.shared_len : 0;
  const int n_keys = n_shared + t + 1;
  for (int u = 0; u < n_keys; ++u) {
    int tbl, idx;
    if (u < n_shared) { tbl = sd.shared_tbl; idx = u; } else { tbl = sd.priv_tbl; idx = u - n_shared; }
    const int blk = block_table[tbl + idx / KV_BLOCK];
    if (blk < 0 || blk >= pool.n_blocks) { if (lane == 0) atomicOr(status, STATUS_BAD_BLOCK); continue; }
    const int dim0 = lane * DPL;                  // DPL divides 8: the lane's dims sit inside one chunk
    const T* kp = pool.chunk(layer, 0, kvh, blk, idx % KV_BLOCK, dim0 & ~7) + (dim0 & 7);
    const T* vp = pool.chunk(layer, 1, kvh, blk, idx % KV_BLOCK, dim0 & ~7) + (dim0 & 7);
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < DPL; ++i) s = fmaf(q[i], to_f32(kp[i]), s);
    s = warp_sum(s);
    const float mn = fmaxf(m, s);
    const float corr = __expf(m - mn), p = __expf(s - mn);
    l = l * corr + p;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] = acc[i] * corr + p * to_f32(vp[i]);
    m = mn;
  }
  const float inv = 1.0f / l;
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[i] = from_f32<T>(acc[i] * inv);
}

}  // namespace rpo
