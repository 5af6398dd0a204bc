// Elementwise / row kernels of the rollout path: seeded init, embedding gather, RMSNorm (with the
// split-K reduction and residual add folded in), RoPE + paged K/V write, SwiGLU, row gathers and
// the log-probability row kernel.  T is the storage type (float or bf16); statistics are float32.
#pragma once
#include "common.cuh"

namespace rpo {

// Per-sequence view of the paged KV cache: a shared segment (the group's prefix blocks, fully
// visible) followed by a private segment (causal).  Offsets index the int32 block table.
struct SeqDesc {
  int32_t shared_tbl;  // first block-table entry of the shared segment, -1 if none
  int32_t shared_len;  // tokens in the shared segment
  int32_t priv_tbl;    // first block-table entry of the private segment
  int32_t reserved;
};

// One KV block = 16 tokens of one (layer, K|V, kv head).  For 16-bit storage its head_dim*32 bytes
// are laid out the way the attention kernels want them in shared memory, so that a block is moved
// with ONE contiguous bulk copy and read with conflict-free ldmatrix:
//     [half head h = dim / 64][token 0..15][8 chunks of 16 bytes, chunk c stored at c ^ (token & 7)]
// (for head_dim 64 there is one half).  float32 storage (plain CUDA-core attention only) keeps
// [token][dim].  chunk() returns the address of the 8-element chunk that holds `dim` (dim % 8 == 0).
template <typename T>
struct KVPool {
  T* base;
  int64_t layer_stride, kv_stride, head_stride;  // elements
  int32_t n_blocks, head_dim;
  __device__ __forceinline__ T* block(int layer, int kv, int head, int block) const {
    return base + layer * layer_stride + kv * kv_stride + head * head_stride + (int64_t)block * KV_BLOCK * head_dim;
  }
  __device__ __forceinline__ T* chunk(int layer, int kv, int head, int blk, int token, int dim) const {
    T* b = block(layer, kv, head, blk);
    if (sizeof(T) == 2) {
      const int per_half = head_dim < 64 ? head_dim : 64;
      const int h = dim / per_half, c = (dim % per_half) >> 3;
      return b + h * (KV_BLOCK * per_half) + token * per_half + ((c ^ (token & 7)) << 3);
    }
    return b + token * head_dim + dim;
  }
};

// --------------------------------------------------------------------------------------------
// Seeded N(0, std^2) init.  Thread = one Philox block = 4 consecutive logical elements.
// Logical element e = row*cols + col lands at dst[(row*row_mul + row_add)*cols + col], which
// lets gate/up rows interleave and q/k/v rows stack inside fused matrices.
// --------------------------------------------------------------------------------------------
template <typename T>
__global__ void init_normal_kernel(T* __restrict__ dst, int64_t n_elems, int cols, int row_mul, int row_add,
                                   uint32_t k0, uint32_t k1, uint32_t tensor_id, float stdv) {
  pdl_prologue();
  const int64_t n_blocks = (n_elems + 3) / 4;
  for (int64_t blk = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; blk < n_blocks;
       blk += (int64_t)gridDim.x * blockDim.x) {
    const U4 r = philox4x32_10((uint32_t)blk, (uint32_t)((uint64_t)blk >> 32), tensor_id, 1u, k0, k1);
    float z[4];
    const uint32_t xa[2] = {r.x, r.z}, xb[2] = {r.y, r.w};
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const float u1 = rmul(radd((float)(xa[j] >> 9), 0.5f), 1.1920928955078125e-07f);  // 2^-23
      const float rad = __fsqrt_rn(rmul(-2.0f, ln_unit(u1)));
      float sn, cs;
      sincos_turn24(xb[j] >> 8, &sn, &cs);
      z[2 * j] = rmul(rad, cs);
      z[2 * j + 1] = rmul(rad, sn);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t e = blk * 4 + j;
      if (e < n_elems) {
        const int64_t row = e / cols, col = e % cols;
        dst[(row * row_mul + row_add) * cols + col] = from_f32<T>(rmul(z[j], stdv));
      }
    }
  }
}

template <typename T>
__global__ void fill_kernel(T* dst, int64_t n, float v) {
  pdl_prologue();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = from_f32<T>(v);
}

__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }
// Four consecutive outputs of type T (8 or 16 bytes, aligned) in one store.
template <typename T>
__device__ __forceinline__ void store4(T* dst, float a, float b, float c, float d);
template <>
__device__ __forceinline__ void store4<float>(float* dst, float a, float b, float c, float d) {
  *reinterpret_cast<float4*>(dst) = make_float4(a, b, c, d);
}
template <>
__device__ __forceinline__ void store4<bf16>(bf16* dst, float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  *reinterpret_cast<uint2*>(dst) = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
}

// cos/sin table [max_positions][head_dim/2], angles in float64.
__global__ void rope_table_kernel(float2* __restrict__ tab, int max_pos, int half, double base) {
  pdl_prologue();
  const int64_t n = (int64_t)max_pos * half;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int pos = (int)(i / half), j = (int)(i % half);
    const double theta = pow(base, -2.0 * (double)j / (double)(2 * half));
    double s, c;
    sincos((double)pos * theta, &s, &c);
    tab[i] = make_float2((float)c, (float)s);
  }
}

// x[r,:] = E[tok[r],:]  (float32 residual stream).
// step_ctr (decode only): the first kernel of a decode forward advances the device step counter
// that the sampler at the end of the forward reads, so that every step is the same launch sequence.
// It also resolves, once per pass, what every layer's RoPE / KV-append kernel needs to know about
// the row - absolute position and where its K/V go in the paged pool - so that those kernels read
// one record instead of walking row -> sequence -> block table in every layer.
struct RowMetaArgs {
  const int32_t* row_seq; const int32_t* row_t; const SeqDesc* seqs; const int32_t* block_table;
  int n_blocks, max_pos;
  int4* row_meta;                     // out: (position, block, slot in block, 0); x = -1: inactive row
};
// Sum of v over the block's threads, in a fixed order (same bits on every run); every thread gets it.
__device__ __forceinline__ float block_sum_fixed(float v, float* red) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < (int)(blockDim.x >> 5); ++i) t += red[i];
  return t;
}

// With xg != NULL (the fused-epilogue layer stack, 16-bit models) the kernel also prepares the first
// RMSNorm: xg[r,:] = bf16(x[r,:] * gain) and ssq[r] = sum x[r,:]^2 (one part per row).
template <typename T>
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const T* __restrict__ E, float* __restrict__ x,
                             int rows, int d, int vocab, int* status, int32_t* step_ctr, RowMetaArgs m,
                             const float* __restrict__ gain, bf16* __restrict__ xg, float* __restrict__ ssq) {
  pdl_prologue();
  __shared__ float red[32];
  const int r = blockIdx.x;
  if (step_ctr && r == 0 && threadIdx.x == 0) *step_ctr += 1;
  if (r >= rows) return;
  if (threadIdx.x == 32) {            // a thread of the second warp: the first is about to wait on the token
    int4 out = make_int4(-1, 0, 0, 0);
    const int t = m.row_t[r];
    if (t >= 0) {
      const SeqDesc sd = m.seqs[m.row_seq[r]];
      const int pos = sd.shared_len + t;
      const int blk = (pos < m.max_pos) ? m.block_table[sd.priv_tbl + t / KV_BLOCK] : -1;
      if (blk < 0 || blk >= m.n_blocks) atomicOr(status, STATUS_BAD_BLOCK);
      else out = make_int4(pos, blk, t % KV_BLOCK, 0);
    }
    m.row_meta[r] = out;
  }
  int tok = tokens[r];
  if (tok < 0 || tok >= vocab) {
    if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_TOKEN);
    tok = min(max(tok, 0), vocab - 1);
  }
  const T* src = E + (int64_t)tok * d;
  float* dst = x + (int64_t)r * d;
  if (!xg) {
    for (int i = threadIdx.x; i < d; i += blockDim.x) dst[i] = to_f32(src[i]);
    return;
  }
  float ss = 0.f;
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = to_f32(src[i]);
    dst[i] = v;
    xg[(int64_t)r * d + i] = __float2bfloat16_rn(v * gain[i]);
    ss += v * v;
  }
  ss = block_sum_fixed(ss, red);
  if (threadIdx.x == 0) ssq[r] = ss;
}

// The RMSNorm preparation alone, for residual rows that no GEMM epilogue produced (the rows that go
// into the output head): xg[r,:] = bf16(x[r,:] * gain), ssq[r] = sum x[r,:]^2.
__global__ void norm_prep_kernel(const float* __restrict__ x, const float* __restrict__ gain, bf16* __restrict__ xg,
                                 float* __restrict__ ssq, int rows, int d) {
  pdl_prologue();
  __shared__ float red[32];
  const int r = blockIdx.x;
  if (r >= rows) return;
  float ss = 0.f;
  for (int i = threadIdx.x * 4; i < d; i += blockDim.x * 4) {
    const float4 v = *reinterpret_cast<const float4*>(x + (int64_t)r * d + i);
    const float4 g = *reinterpret_cast<const float4*>(gain + i);
    store4<bf16>(xg + (int64_t)r * d + i, v.x * g.x, v.y * g.y, v.z * g.z, v.w * g.w);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = block_sum_fixed(ss, red);
  if (threadIdx.x == 0) ssq[r] = ss;
}

// dst[idx[r],:] = src[r,:]  (32-bit words; rows whose idx is negative are skipped)
__global__ void scatter_rows_u32_kernel(const uint32_t* __restrict__ src, const int32_t* __restrict__ idx,
                                        uint32_t* __restrict__ dst, int rows, int d) {
  pdl_prologue();
  const int r = blockIdx.x;
  if (r >= rows) return;
  const int s = idx[r];
  if (s < 0) return;
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[(int64_t)s * d + i] = src[(int64_t)r * d + i];
}

// dst[r,:] = src[idx[r],:]  (float32 rows; idx may be NULL = identity)
__global__ void gather_rows_f32_kernel(const float* __restrict__ src, const int32_t* __restrict__ idx,
                                       float* __restrict__ dst, int rows, int d) {
  pdl_prologue();
  const int r = blockIdx.x;
  if (r >= rows) return;
  const int s = idx ? idx[r] : r;
  if (s < 0) {
    for (int i = threadIdx.x; i < d; i += blockDim.x) dst[(int64_t)r * d + i] = 0.f;
    return;
  }
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[(int64_t)r * d + i] = src[(int64_t)s * d + i];
}

// RMSNorm of the float32 residual stream, one CTA per row, 128-bit accesses (d % 4 == 0):
//   x[r,:] += sum_s partial[s][r,:]   (optional split-K partial planes of the previous GEMM, summed
//                                      in plane order; the loads of all planes are independent)
//   h[r,:]  = x[r,:] / sqrt(mean(x^2) + eps) * g
// Dynamic shared memory: d floats (the row, kept between the two passes).
template <typename T>
__global__ void rmsnorm_kernel(float* __restrict__ x, const float* __restrict__ gain, T* __restrict__ h, int rows,
                               int d, float eps, const float* __restrict__ partial, int n_splits,
                               int64_t split_stride) {
  pdl_prologue();
  extern __shared__ __align__(16) float srow[];
  __shared__ float red[32];
  const int r = blockIdx.x;
  if (r >= rows) return;
  const int d4 = d >> 2;
  float4* xr = reinterpret_cast<float4*>(x + (int64_t)r * d);
  float4* s4 = reinterpret_cast<float4*>(srow);
  float ss = 0.f;
  if (d4 <= (int)blockDim.x) {
    // One float4 per thread (decode-sized rows): the row stays in registers, and the gain is
    // requested together with the row and the planes, so the kernel makes one round trip to L2.
    const int i = threadIdx.x;
    const bool on = i < d4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f), g = v;
    if (on) {
      v = xr[i];
      g = reinterpret_cast<const float4*>(gain)[i];
      if (partial) {
        const float4* p4 = reinterpret_cast<const float4*>(partial + (int64_t)r * d) + i;
        const int64_t st4 = split_stride >> 2;
#pragma unroll 4
        for (int s = 0; s < n_splits; ++s) {
          const float4 q = p4[s * st4];
          v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
        }
        xr[i] = v;
      }
      ss = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = (lane_id() < (int)(blockDim.x >> 5)) ? red[lane_id()] : 0.f;
    tot = warp_sum(tot);                       // every warp sums the per-warp parts in the same order
    const float inv = 1.0f / sqrtf(tot / (float)d + eps);
    if (on) store4<T>(h + (int64_t)r * d + 4 * i, v.x * inv * g.x, v.y * inv * g.y, v.z * inv * g.z, v.w * inv * g.w);
    return;
  }
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    float4 v = xr[i];
    if (partial) {
      const float4* p4 = reinterpret_cast<const float4*>(partial + (int64_t)r * d) + i;
      const int64_t st4 = split_stride >> 2;
#pragma unroll 4
      for (int s = 0; s < n_splits; ++s) {
        const float4 q = p4[s * st4];
        v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
      }
      xr[i] = v;
    }
    s4[i] = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x < 32) {
    float v = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.f;
    v = warp_sum(v);
    if (threadIdx.x == 0) red[0] = v;
  }
  __syncthreads();
  const float inv = 1.0f / sqrtf(red[0] / (float)d + eps);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  T* hr = h + (int64_t)r * d;
  for (int i = threadIdx.x; i < d4; i += blockDim.x) {
    const float4 v = s4[i], g = g4[i];
    hr[4 * i] = from_f32<T>(v.x * inv * g.x); hr[4 * i + 1] = from_f32<T>(v.y * inv * g.y);
    hr[4 * i + 2] = from_f32<T>(v.z * inv * g.z); hr[4 * i + 3] = from_f32<T>(v.w * inv * g.w);
  }
}

// RMSNorm for many rows (prefill, log-prob passes): one warp per row, the row held in registers
// (d <= 4096, d % 128 == 0 not required: lanes take float4 number lane, lane + 32, ...), no shared
// memory and no block barrier.  Same arithmetic as rmsnorm_kernel without split-K planes.
template <typename T, int MAXV>
__global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const float* __restrict__ x, const float* __restrict__ gain,
                                                           T* __restrict__ h, int rows, int d, float eps) {
  pdl_prologue();
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= rows) return;
  const int d4 = d >> 2;
  const float4* xr = reinterpret_cast<const float4*>(x + (int64_t)r * d);
  float4 v[MAXV];
  float ss = 0.f;
#pragma unroll
  for (int k = 0; k < MAXV; ++k) {
    const int i = lane + 32 * k;
    if (i < d4) { v[k] = xr[i]; ss += v[k].x * v[k].x + v[k].y * v[k].y + v[k].z * v[k].z + v[k].w * v[k].w; }
  }
  ss = warp_sum(ss);
  const float inv = 1.0f / sqrtf(ss / (float)d + eps);
  const float4* g4 = reinterpret_cast<const float4*>(gain);
  T* hr = h + (int64_t)r * d;
#pragma unroll
  for (int k = 0; k < MAXV; ++k) {
    const int i = lane + 32 * k;
    if (i < d4) {
      const float4 g = g4[i];
      if (sizeof(T) == 2) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[k].x * inv * g.x, v[k].y * inv * g.y);
        __nv_bfloat162 b = __floats2bfloat162_rn(v[k].z * inv * g.z, v[k].w * inv * g.w);
        uint2 o; o.x = *reinterpret_cast<uint32_t*>(&a); o.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(hr + 4 * i) = o;
      } else {
        float4 o = make_float4(v[k].x * inv * g.x, v[k].y * inv * g.y, v[k].z * inv * g.z, v[k].w * inv * g.w);
        *reinterpret_cast<float4*>(hr + 4 * i) = o;
      }
    }
  }
}

// x[i] += sum_s partial[s*stride + i], fixed order (deterministic split-K reduction). n % 4 == 0.
__global__ void reduce_partials_kernel(float* __restrict__ x, const float* __restrict__ partial, int n_splits, int64_t n,
                                       int64_t stride) {
  pdl_prologue();
  for (int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4; i < n; i += (int64_t)gridDim.x * blockDim.x * 4) {
    float4 v = *(const float4*)(x + i);
    for (int s = 0; s < n_splits; ++s) {
      const float4 q = *(const float4*)(partial + s * stride + i);
      v.x += q.x; v.y += q.y; v.z += q.z; v.w += q.w;
    }
    *(float4*)(x + i) = v;
  }
}

// RoPE (rotate-half) on q and k, then K/V written to the row's slot of its private segment.
// qkv row layout: [q heads | k heads | v heads] x head_dim.  A group of dh/16 threads owns one
// (row, head): each thread takes 8 consecutive dimensions of the low half and the 8 dimensions
// they pair with in the high half (128-bit accesses for 16-bit storage).  Grid: ceil(rows * heads *
// dh/16 / blockDim) CTAs.
// With `partial` the projection arrives as n_splits split-K planes [rows, qkv_cols] of float32:
// they are summed in plane order and rounded to the storage type first, exactly what the
// unsplit GEMM epilogue would have stored.
template <typename T>
__global__ void rope_kv_kernel(T* __restrict__ qkv, const int4* __restrict__ row_meta, const float2* __restrict__ rope_tab,
                               KVPool<T> pool, int layer, int rows, int hq, int hkv,
                               const float* __restrict__ partial, int n_splits, int64_t split_stride) {
  pdl_prologue();
  const int dh = pool.head_dim, half = dh / 2, tph = dh / 16, heads = hq + 2 * hkv;
  const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t unit = gid / tph;                       // (row, head)
  if (unit >= (int64_t)rows * heads) return;
  const int r = (int)(unit / heads), head = (int)(unit % heads), i0 = (int)(gid % tph) * 8;
  const int64_t off = (int64_t)r * heads * dh + (int64_t)head * dh;
  T* src = qkv + off;
  // the projection values first: these loads do not depend on the row's metadata, so they are in
  // flight while the (dependent) metadata chain below resolves
  float lo[8], hi[8];
  if (partial) {
#pragma unroll
    for (int j = 0; j < 8; ++j) { lo[j] = 0.f; hi[j] = 0.f; }
#pragma unroll 4
    for (int s = 0; s < n_splits; ++s) {
      const float4* pl = reinterpret_cast<const float4*>(partial + s * split_stride + off + i0);
      const float4* ph = reinterpret_cast<const float4*>(partial + s * split_stride + off + half + i0);
      const float4 a0 = pl[0], a1 = pl[1], b0 = ph[0], b1 = ph[1];
      lo[0] += a0.x; lo[1] += a0.y; lo[2] += a0.z; lo[3] += a0.w; lo[4] += a1.x; lo[5] += a1.y; lo[6] += a1.z; lo[7] += a1.w;
      hi[0] += b0.x; hi[1] += b0.y; hi[2] += b0.z; hi[3] += b0.w; hi[4] += b1.x; hi[5] += b1.y; hi[6] += b1.z; hi[7] += b1.w;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) { lo[j] = to_f32(from_f32<T>(lo[j])); hi[j] = to_f32(from_f32<T>(hi[j])); }
  } else {
    T tl[8], th[8];
    *reinterpret_cast<uint4*>(tl) = *reinterpret_cast<const uint4*>(src + i0);
    if (sizeof(T) == 4) *reinterpret_cast<uint4*>(tl + 4) = *reinterpret_cast<const uint4*>(src + i0 + 4);
    *reinterpret_cast<uint4*>(th) = *reinterpret_cast<const uint4*>(src + half + i0);
    if (sizeof(T) == 4) *reinterpret_cast<uint4*>(th + 4) = *reinterpret_cast<const uint4*>(src + half + i0 + 4);
#pragma unroll
    for (int j = 0; j < 8; ++j) { lo[j] = to_f32(tl[j]); hi[j] = to_f32(th[j]); }
  }
  const int4 meta = row_meta[r];                        // (position, private KV block, slot in block): resolved once per pass
  if (meta.x < 0) return;                               // inactive row (or a bad position / block, flagged when resolved)
  const int pos = meta.x;
  T *dst_lo = src + i0, *dst_hi = src + half + i0;      // q: rotated in place
  if (head >= hq) {
    const int kv = (head - hq) / hkv, kh = (head - hq) % hkv;
    dst_lo = pool.chunk(layer, kv, kh, meta.y, meta.z, i0);
    dst_hi = pool.chunk(layer, kv, kh, meta.y, meta.z, half + i0);
  }
  __align__(16) T ol[8], oh[8];
  if (head < hq + hkv) {                                // q or k: rotate
    const float2* cs = rope_tab + (int64_t)pos * half + i0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const float2 c = cs[j];
      ol[j] = from_f32<T>(lo[j] * c.x - hi[j] * c.y);
      oh[j] = from_f32<T>(hi[j] * c.x + lo[j] * c.y);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) { ol[j] = from_f32<T>(lo[j]); oh[j] = from_f32<T>(hi[j]); }
  }
  *reinterpret_cast<uint4*>(dst_lo) = *reinterpret_cast<const uint4*>(ol);
  if (sizeof(T) == 4) *reinterpret_cast<uint4*>(dst_lo + 4) = *reinterpret_cast<const uint4*>(ol + 4);
  *reinterpret_cast<uint4*>(dst_hi) = *reinterpret_cast<const uint4*>(oh);
  if (sizeof(T) == 4) *reinterpret_cast<uint4*>(dst_hi + 4) = *reinterpret_cast<const uint4*>(oh + 4);
}

// act[r, j] = silu(gu[r, 2j]) * gu[r, 2j+1]   (gate/up interleaved by the fused weight layout)
template <typename T>
__global__ void swiglu_kernel(const T* __restrict__ gu, T* __restrict__ act, int64_t n_out) {
  pdl_prologue();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_out; i += (int64_t)gridDim.x * blockDim.x) {
    const float g = to_f32(gu[2 * i]), u = to_f32(gu[2 * i + 1]);
    act[i] = from_f32<T>(g / (1.0f + __expf(-g)) * u);
  }
}

// Row metadata of a teacher-forced pass: row (s, j), j in [0, S-1), feeds token j of sequence s at
// private index j; it is active when j < len[s]-1.  Also the input token of the row.
__global__ void build_teacher_rows_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ lens,
                                          int seq0, int n_seq, int S, int32_t* __restrict__ row_seq,
                                          int32_t* __restrict__ row_t, int32_t* __restrict__ row_tok) {
  pdl_prologue();
  const int n = n_seq * (S - 1);
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    const int s = i / (S - 1), j = i % (S - 1);
    const int len = lens[seq0 + s];
    row_seq[i] = s;
    row_t[i] = (j < len - 1) ? j : -1;
    row_tok[i] = (j < len - 1) ? tokens[(int64_t)(seq0 + s) * S + j] : 0;
  }
}

// Gather index for the head of a teacher-forced pass over head-rows (s, j), j in [0,S):
// j = 0 reads the group's last-prefix residual (index = -(1 + x_last slot) encoded), j >= 1 reads
// layer-stack row (s, j-1).  Here we simply materialise the head input rows.
__global__ void gather_head_rows_kernel(const float* __restrict__ x, const float* __restrict__ x_last,
                                        const int32_t* __restrict__ seq_slot, int row0, int n_rows, int S, int d,
                                        float* __restrict__ dst) {
  pdl_prologue();
  const int i = blockIdx.x;
  if (i >= n_rows) return;
  const int hr = row0 + i, s = hr / S, j = hr % S;
  const float* src = (j == 0) ? x_last + (int64_t)seq_slot[s] * d : x + ((int64_t)s * (S - 1) + (j - 1)) * d;
  for (int c = threadIdx.x; c < d; c += blockDim.x) dst[(int64_t)i * d + c] = src[c];
}

__device__ __forceinline__ float block_reduce_max(float v, float* red) {
  v = warp_max(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    float w = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : -INFINITY;
    w = warp_max(w);
    if (threadIdx.x == 0) red[0] = w;
  }
  __syncthreads();
  const float out = red[0];
  __syncthreads();
  return out;
}
__device__ __forceinline__ float block_reduce_sum(float v, float* red) {
  v = warp_sum(v);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x < 32) {
    float w = (threadIdx.x < (blockDim.x >> 5)) ? red[threadIdx.x] : 0.f;
    w = warp_sum(w);
    if (threadIdx.x == 0) red[0] = w;
  }
  __syncthreads();
  const float out = red[0];
  __syncthreads();
  return out;
}

// log-prob of the given token per head-row of a teacher-forced pass (full-vocabulary
// normalisation, z = logits * inv_T); rows with j >= len get 0.
__global__ void logprob_rows_kernel(const float* __restrict__ logits, int row0, int n_rows, int V, int S,
                                    const int32_t* __restrict__ tokens, const int32_t* __restrict__ lens, int seq0,
                                    float inv_T, float* __restrict__ out, float* __restrict__ logits_dbg) {
  pdl_prologue();
  __shared__ float red[32];
  const int i = blockIdx.x;
  if (i >= n_rows) return;
  const int hr = row0 + i, s = hr / S, j = hr % S;
  const int64_t o = (int64_t)(seq0 + s) * S + j;
  const float* row = logits + (int64_t)i * V;
  if (logits_dbg)
    for (int c = threadIdx.x; c < V; c += blockDim.x) logits_dbg[o * V + c] = row[c];
  if (j >= lens[seq0 + s]) { if (threadIdx.x == 0) out[o] = 0.f; return; }
  float m = -INFINITY;
  for (int c = threadIdx.x; c < V; c += blockDim.x) m = fmaxf(m, row[c] * inv_T);
  m = block_reduce_max(m, red);
  float sum = 0.f;
  for (int c = threadIdx.x; c < V; c += blockDim.x) sum += __expf(row[c] * inv_T - m);
  sum = block_reduce_sum(sum, red);
  if (threadIdx.x == 0) {
    int tok = tokens[o];
    tok = min(max(tok, 0), V - 1);
    out[o] = (row[tok] * inv_T - m) - logf(sum);
  }
}

// Target token of every head-row of a teacher-forced pass (row i of the launch = head row row0 + i =
// (sequence, suffix position)); -1 beyond the sequence's length.
__global__ void lse_targets_kernel(int row0, int n_rows, int V, int S, const int32_t* __restrict__ tokens,
                                   const int32_t* __restrict__ lens, int seq0, int32_t* __restrict__ target) {
  pdl_prologue();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_rows) return;
  const int hr = row0 + i, s = hr / S, j = hr % S;
  const int64_t o = (int64_t)(seq0 + s) * S + j;
  target[i] = (j < lens[seq0 + s]) ? min(max(tokens[o], 0), V - 1) : -1;
}

// log pi of the target per head-row from the output head's per-unit (max, sum of exponentials) and the
// target's z: log pi = (z_t - M) - log sum_u s_u exp(m_u - M), M = max_u m_u.  A warp per row; rows
// without a target get 0.
__global__ void lse_merge_rows_kernel(const float2* __restrict__ parts, int n_parts, const float* __restrict__ zt,
                                      const int32_t* __restrict__ target, int row0, int n_rows, int S, int seq0,
                                      float* __restrict__ out) {
  pdl_prologue();
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= n_rows) return;
  const int hr = row0 + i, s = hr / S, j = hr % S;
  const int64_t o = (int64_t)(seq0 + s) * S + j;
  if (target[i] < 0) { if (lane == 0) out[o] = 0.f; return; }
  const float2* p = parts + (int64_t)i * n_parts;
  float m = -INFINITY;
  for (int u = lane; u < n_parts; u += 32) m = fmaxf(m, p[u].x);
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, k));
  float sum = 0.f;
  for (int u = lane; u < n_parts; u += 32) { const float2 q = p[u]; sum += q.y * __expf(q.x - m); }
  sum = warp_sum(sum);
  if (lane == 0) out[o] = (zt[i] - m) - logf(sum);
}

}  // namespace rpo
