// Epilogues of the tensor-core GEMMs: what happens to a tile of float32 sums C = A W^T.
//
// Besides plain stores, the layer's elementwise work is done here, so that a decoder layer is five
// kernels (QKV, attention, O projection, gate/up, down) instead of nine:
//
//   * RMSNorm never runs as a kernel of its own.  rmsnorm(x, g) W^T = (1/rms(x)) * ((x * g) W^T): the
//     kernel that produces the residual rows x also emits xg = bf16(x * g) and, per row, partial sums
//     of x^2 (one per column tile, summed in a fixed order by the reader); the GEMM that consumes xg
//     multiplies its output rows by 1/sqrt(mean(x^2) + eps)                     (TC_N* epilogues).
//   * RoPE and the paged K/V append are the epilogue of the QKV projection       (TC_QKV_ROPE).
//   * SwiGLU is the epilogue of the gate/up projection (interleaved columns)     (TC_SWIGLU, TC_NSWIGLU).
//   * the residual add is the epilogue of the O and down projections             (TC_ADD_F32, TC_ADD_NORM).
//
// Split-K.  When a launch splits K, every epilogue warp stores its 32 rows of the float32 partial
// tile to a plane and then counts itself in on an arrival counter; the warp that finds itself last
// (nobody waits) sums the planes in plane order - so the result does not depend on who came last -
// and applies the epilogue (epi_reduce_rows).  It resets the counter for the next launch.
#pragma once
#include "common.cuh"
#include "kernels.cuh"

namespace rpo {

enum TcEpilogue {
  TC_STORE_BF16 = 0, TC_STORE_F32 = 1, TC_ADD_F32 = 2, TC_SWIGLU = 3, TC_PARTIAL = 4,
  TC_NSTORE_F32 = 5,   // rows scaled by 1/rms, float32 store (output head)
  TC_NSWIGLU = 6,      // rows scaled by 1/rms, SwiGLU on interleaved gate/up columns, bf16 store
  TC_QKV_ROPE = 7,     // rows scaled by 1/rms, RoPE on q and k heads, q -> qkv buffer, k / v -> paged pool
  TC_ADD_NORM = 8,     // x += C; xg = bf16(x * gain); partial sums of x^2 per (row, column tile)
  TC_NLSE = 9,         // rows scaled by 1/rms and 1/T; nothing is stored but, per (row, column unit), the running
                       // maximum and the sum of exponentials, and the logit of the row's target token (Eq. 7's
                       // log pi(o_j | ...) without writing the logits out); pair kernel, no split-K
};

__host__ __device__ constexpr bool tc_epi_scaled(int epi) { return epi == TC_NSTORE_F32 || epi == TC_NSWIGLU || epi == TC_QKV_ROPE || epi == TC_NLSE; }
__host__ __device__ constexpr bool tc_epi_fused(int epi) { return epi >= TC_NSTORE_F32; }

struct TcParams {
  void* C;              // output (type by epilogue); TC_QKV_ROPE: the qkv buffer (q heads land in their columns)
  int M, N, K;
  int ldc;              // elements per output row
  int tiles_m, tiles_n, splits, kb_per_split, kb_total;
  int64_t split_stride; // elements between split planes
  int* status;
  // ---- fused epilogues
  float* planes;        // split-K planes [splits][M][N] (float32)
  int* tile_ctr;        // arrival counters, one per (output tile, epilogue warp) unit, zero between launches
  const float* ssq_in;  // TC_N*: [M][ssq_in_parts] partial sums of squares of the rows the A operand was made from
  int ssq_in_parts;
  float inv_norm_dim, eps;   // 1 / (row length of those rows), RMSNorm epsilon
  float* ssq_out;       // TC_ADD_NORM: [M][ssq_out_parts]
  int ssq_out_parts;    //   parts per row = column units of the launch (tiles_n, or 2 tiles_n for pair tiles of 64 rows per CTA)
  bf16* xg_out;         // TC_ADD_NORM: [M][N] = bf16(x * gain)
  const float* gain;    // TC_ADD_NORM: [N]
  const int4* row_meta; // TC_QKV_ROPE: per row (position, KV block, slot, -), x < 0: inactive row
  const float2* rope;   // TC_QKV_ROPE: [positions][head_dim / 2] (cos, sin)
  KVPool<bf16> pool;    // TC_QKV_ROPE
  int layer, hq, hkv, head_dim;
  float2* lse_parts;    // TC_NLSE: [M][lse_stride] (max, sum of exp(z - max)) over the unit's columns, z = logit / T
  int lse_stride;       //   column units per row (as ssq_out_parts)
  float* lse_tgt;       // TC_NLSE: [M] z of the row's target token
  const int32_t* lse_target;   // TC_NLSE: [M] target token id per row, negative = none
  float lse_inv_T;
};

// Epilogue of one 32-column chunk of an accumulator row: r[0..31] are the float32 bit patterns of
// columns col .. col+31 of output row `row`.
// STREAM: the output is far larger than L2 and not read again by this kernel; streaming stores
// keep it from evicting the operand tiles other CTAs are about to fetch.
template <int EPI>
__device__ __forceinline__ void tc_store_chunk(const TcParams& p, const uint32_t* r, int row, int col, int split,
                                               const bool STREAM = false) {
  if (row >= p.M || col >= p.N) return;
  const int ncol = min(32, p.N - col);       // multiple of 8 (N % 8 == 0)
  if (EPI == TC_STORE_BF16) {
    bf16* dst = (bf16*)p.C + (int64_t)row * p.ldc + col;
    for (int j = 0; j < ncol; j += 8) {
      uint4 v;
      __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
      __nv_bfloat162 h1 = __floats2bfloat162_rn(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
      __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(r[j + 4]), __uint_as_float(r[j + 5]));
      __nv_bfloat162 h3 = __floats2bfloat162_rn(__uint_as_float(r[j + 6]), __uint_as_float(r[j + 7]));
      v.x = *(uint32_t*)&h0; v.y = *(uint32_t*)&h1; v.z = *(uint32_t*)&h2; v.w = *(uint32_t*)&h3;
      if (STREAM) __stcs((uint4*)(dst + j), v); else *(uint4*)(dst + j) = v;
    }
  } else if (EPI == TC_SWIGLU) {
    // columns (2j, 2j+1) = (gate_j, up_j)  ->  out[row, col/2 + j]
    bf16* dst = (bf16*)p.C + (int64_t)row * p.ldc + col / 2;
    for (int j = 0; j < ncol; j += 16) {
      uint32_t o[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float g0 = __uint_as_float(r[j + 4 * q]), u0 = __uint_as_float(r[j + 4 * q + 1]);
        const float g1 = __uint_as_float(r[j + 4 * q + 2]), u1 = __uint_as_float(r[j + 4 * q + 3]);
        __nv_bfloat162 h = __floats2bfloat162_rn(g0 / (1.0f + __expf(-g0)) * u0, g1 / (1.0f + __expf(-g1)) * u1);
        o[q] = *(uint32_t*)&h;
      }
      if (STREAM) __stcs((uint4*)(dst + j / 2), make_uint4(o[0], o[1], o[2], o[3]));
      else *(uint4*)(dst + j / 2) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  } else {
    float* dst = (EPI == TC_PARTIAL) ? p.planes + split * p.split_stride + (int64_t)row * p.N + col
                                     : (float*)p.C + (int64_t)row * p.ldc + col;
    for (int j = 0; j < ncol; j += 4) {
      float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                             __uint_as_float(r[j + 3]));
      if (EPI == TC_ADD_F32) {
        const float4 o = *(float4*)(dst + j);
        v.x += o.x; v.y += o.y; v.z += o.z; v.w += o.w;
      }
      if (STREAM) __stcs((float4*)(dst + j), v); else *(float4*)(dst + j) = v;
    }
  }
}

// 1 / rms of the row the A operand's row `row` was made from: the partial sums of squares are added
// in index order by every reader, so all of them get the same bits.
__device__ __forceinline__ float epi_row_scale(const TcParams& p, int row) {
  if (row >= p.M) return 0.f;
  const float* s = p.ssq_in + (int64_t)row * p.ssq_in_parts;
  float t = 0.f;
  for (int i = 0; i < p.ssq_in_parts; ++i) t += s[i];
  return 1.0f / sqrtf(t * p.inv_norm_dim + p.eps);
}

// The same for a whole warp working on one row (split-K reduction): lanes fetch the parts side by side.
__device__ __forceinline__ float epi_row_scale_warp(const TcParams& p, int row, int lane) {
  float t = 0.f;
  if (row < p.M)
    for (int i = lane; i < p.ssq_in_parts; i += 32) t += p.ssq_in[(int64_t)row * p.ssq_in_parts + i];
  t = warp_sum(t);
  return row < p.M ? 1.0f / sqrtf(t * p.inv_norm_dim + p.eps) : 0.f;
}

__device__ __forceinline__ float silu_mul(float g, float u) { return g / (1.0f + __expf(-g)) * u; }

// Where 4 (or 8) consecutive dims [dim, dim + n) of the rotated q / k or of v go.  head = column / head_dim.
__device__ __forceinline__ bf16* epi_qkv_dst(const TcParams& p, int row, int head, int dim, const int4& meta) {
  if (head < p.hq) return (bf16*)p.C + (int64_t)row * p.ldc + head * p.head_dim + dim;
  const int kv = (head - p.hq) / p.hkv, kh = (head - p.hq) % p.hkv;
  return p.pool.chunk(p.layer, kv, kh, meta.y, meta.z, dim & ~7) + (dim & 7);
}

// ---- direct path (no split): thread = row, 32-column chunks out of tensor memory --------------------

// TC_NSTORE_F32 / TC_NSWIGLU on one chunk; `scale` = epi_row_scale of the row.
template <int EPI>
__device__ __forceinline__ void epi_scaled_chunk(const TcParams& p, uint32_t* r, int row, int col, float scale, bool STREAM) {
#pragma unroll
  for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * scale);
  if (EPI == TC_NSTORE_F32) tc_store_chunk<TC_STORE_F32>(p, r, row, col, 0, STREAM);
  else tc_store_chunk<TC_SWIGLU>(p, r, row, col, 0, STREAM);
}

// TC_NLSE on one chunk: z = C * (1/rms) * (1/T); folds the chunk into the row's running (m, s) with
// s = sum exp(z - m), and picks up the target's z when it lies in the chunk.
__device__ __forceinline__ void epi_lse_chunk(const TcParams& p, const uint32_t* r, int col, float scale, int tgt,
                                              float& m, float& s, float& zt) {
  if (col >= p.N) return;
  float z[32];
  float cm = -INFINITY;
#pragma unroll
  for (int j = 0; j < 32; ++j) {
    z[j] = (__uint_as_float(r[j]) * scale) * p.lse_inv_T;
    if (col + j < p.N) cm = fmaxf(cm, z[j]);
  }
  const float mn = fmaxf(m, cm);
  float acc = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (col + j < p.N) acc += __expf(z[j] - mn);
  s = s * __expf(m - mn) + acc;                 // m = -inf at the start: s = 0 * 0
  m = mn;
  if (tgt >= col && tgt < col + 32) {
#pragma unroll
    for (int j = 0; j < 32; ++j)
      if (tgt - col == j) zt = z[j];
  }
}

// TC_QKV_ROPE on the chunk pair (lo, hi): columns col_lo .. +31 and col_lo + head_dim/2 .. +31 of one head.
// Every load is issued before the first store (a store may alias anything as far as the compiler knows,
// and would otherwise put each later load behind a round trip of its own).
__device__ __forceinline__ void epi_rope_pair(const TcParams& p, const uint32_t* lo, const uint32_t* hi, int row, int col_lo,
                                              float scale, const int4& meta) {
  if (row >= p.M || col_lo >= p.N || meta.x < 0) return;
  const int half = p.head_dim >> 1, head = col_lo / p.head_dim, i0 = col_lo % p.head_dim;   // i0 < half
  const bool rotate = head < p.hq + p.hkv;
  float4 cs[16];                                      // (cos, sin) of dims i0 .. i0 + 31, two per float4
  if (rotate) {
    const float4* src = reinterpret_cast<const float4*>(p.rope + (int64_t)meta.x * half + i0);   // i0 % 32 == 0: 16-byte aligned
#pragma unroll
    for (int j = 0; j < 16; ++j) cs[j] = src[j];
  }
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    __align__(16) bf16 ol[8], oh[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float a = __uint_as_float(lo[j + e]) * scale, b = __uint_as_float(hi[j + e]) * scale;
      if (rotate) {
        const float4 c4 = cs[(j + e) >> 1];
        const float cx = (e & 1) ? c4.z : c4.x, cy = (e & 1) ? c4.w : c4.y;
        ol[e] = __float2bfloat16_rn(a * cx - b * cy);
        oh[e] = __float2bfloat16_rn(b * cx + a * cy);
      } else {
        ol[e] = __float2bfloat16_rn(a); oh[e] = __float2bfloat16_rn(b);
      }
    }
    *reinterpret_cast<uint4*>(epi_qkv_dst(p, row, head, i0 + j, meta)) = *reinterpret_cast<const uint4*>(ol);
    *reinterpret_cast<uint4*>(epi_qkv_dst(p, row, head, half + i0 + j, meta)) = *reinterpret_cast<const uint4*>(oh);
  }
}

// TC_ADD_NORM on one chunk: returns the chunk's sum of squares of the updated row.  Loads first, then stores.
__device__ __forceinline__ float epi_add_norm_chunk(const TcParams& p, const uint32_t* r, int row, int col) {
  if (row >= p.M || col >= p.N) return 0.f;
  float* x = (float*)p.C + (int64_t)row * p.ldc + col;
  bf16* xg = p.xg_out + (int64_t)row * p.N + col;
  float4 v[8], g[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const bool on = col + 4 * j < p.N;                // N % 8 == 0
    v[j] = on ? *(const float4*)(x + 4 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
    g[j] = on ? *(const float4*)(p.gain + col + 4 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  float ss = 0.f;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (col + 4 * j >= p.N) break;
    v[j].x += __uint_as_float(r[4 * j]); v[j].y += __uint_as_float(r[4 * j + 1]);
    v[j].z += __uint_as_float(r[4 * j + 2]); v[j].w += __uint_as_float(r[4 * j + 3]);
    *(float4*)(x + 4 * j) = v[j];
    ss += v[j].x * v[j].x + v[j].y * v[j].y + v[j].z * v[j].z + v[j].w * v[j].w;
    store4<bf16>(xg + 4 * j, v[j].x * g[j].x, v[j].y * g[j].y, v[j].z * g[j].z, v[j].w * g[j].w);
  }
  return ss;
}

// ---- split-K: the last warp to arrive at its part of a tile sums the planes and applies the epilogue ----
// The unit of arrival is what ONE epilogue warp stores of a tile: 32 rows x n_cols columns (its tensor-
// memory lane quadrant).  The warp that finds itself last at a unit reduces it alone, so no thread
// ever waits for another one.  A lane owns 4 consecutive columns of a 128-column strip (contiguous
// accesses per row); rows go in batches of RB, PL planes at a time, so that RB x PL plane loads are in
// flight per lane (the reduction is a chain of round trips to L2, not a bandwidth problem).
template <int EPI, int RB, int PL>
__device__ __forceinline__ void epi_reduce_rows_t(const TcParams& p, int row0, int col0, int n_cols, int part_index, int lane) {
  const int64_t st = p.split_stride;
  for (int rb = 0; rb < 32; rb += RB) {
    if (row0 + rb >= p.M) break;
    float scale[RB], ssq[RB];
    int4 meta[RB];
#pragma unroll
    for (int q = 0; q < RB; ++q) {
      const int row = row0 + rb + q;
      ssq[q] = 0.f;
      scale[q] = tc_epi_scaled(EPI) ? epi_row_scale_warp(p, row, lane) : 1.f;
      meta[q] = (EPI == TC_QKV_ROPE && row < p.M) ? p.row_meta[row] : make_int4(-1, 0, 0, 0);
    }
    for (int c0 = 0; c0 < n_cols; c0 += 128) {
      const int col = col0 + c0 + 4 * lane;
      const bool con = (c0 + 4 * lane < n_cols) && col < p.N;
      float4 acc[RB];
      // Everything the epilogue reads is requested together with the planes, before the first store:
      // the residual rows (TC_ADD_*), the gain (TC_ADD_NORM), the rows' (cos, sin) entries (TC_QKV_ROPE).
      float4 xo[RB], cs0[RB], cs1[RB];
      const float4 gn = (EPI == TC_ADD_NORM && con) ? *(const float4*)(p.gain + col) : make_float4(0.f, 0.f, 0.f, 0.f);
      const int r_half = p.head_dim >> 1, r_head = col / max(p.head_dim, 1), r_dim = col % max(p.head_dim, 1);
      const bool r_rot = EPI == TC_QKV_ROPE && con && r_head < p.hq + p.hkv;
#pragma unroll
      for (int q = 0; q < RB; ++q) {
        acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        xo[q] = ((EPI == TC_ADD_NORM || EPI == TC_ADD_F32) && con && row0 + rb + q < p.M)
                    ? *reinterpret_cast<const float4*>((const float*)p.C + (int64_t)(row0 + rb + q) * p.ldc + col)
                    : make_float4(0.f, 0.f, 0.f, 0.f);
        cs0[q] = cs1[q] = make_float4(1.f, 0.f, 1.f, 0.f);
        if (r_rot && meta[q].x >= 0) {
          const float4* src = reinterpret_cast<const float4*>(p.rope + (int64_t)meta[q].x * r_half + (r_dim % r_half));
          cs0[q] = src[0]; cs1[q] = src[1];
        }
      }
      if (con) {
        // PL planes of RB rows are requested together: RB x PL independent 16-byte loads per lane
        const float* src = p.planes + (int64_t)(row0 + rb) * p.N + col;
        for (int s = 0; s < p.splits; s += PL) {
          float4 t[PL][RB];
#pragma unroll
          for (int k = 0; k < PL; ++k) {
#pragma unroll
            for (int q = 0; q < RB; ++q)
              t[k][q] = (s + k < p.splits && row0 + rb + q < p.M)
                            ? __ldcg(reinterpret_cast<const float4*>(src + (int64_t)q * p.N + (int64_t)(s + k) * st))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int k = 0; k < PL; ++k) {            // plane order: the sum does not depend on who arrived last
#pragma unroll
            for (int q = 0; q < RB; ++q) { acc[q].x += t[k][q].x; acc[q].y += t[k][q].y; acc[q].z += t[k][q].z; acc[q].w += t[k][q].w; }
          }
        }
      }
#pragma unroll
      for (int q = 0; q < RB; ++q) {
        const int row = row0 + rb + q;
        const bool on = con && row < p.M;
        float4 v = acc[q];
        if (EPI == TC_NSTORE_F32) {
          if (on) *(float4*)((float*)p.C + (int64_t)row * p.ldc + col) = make_float4(v.x * scale[q], v.y * scale[q], v.z * scale[q], v.w * scale[q]);
        } else if (EPI == TC_NSWIGLU) {
          if (on) {
            __nv_bfloat162 h = __floats2bfloat162_rn(silu_mul(v.x * scale[q], v.y * scale[q]), silu_mul(v.z * scale[q], v.w * scale[q]));
            *(uint32_t*)((bf16*)p.C + (int64_t)row * p.ldc + col / 2) = *(uint32_t*)&h;
          }
        } else if (EPI == TC_QKV_ROPE) {
          // the lane holding the other half of the rotation pair is head_dim/8 lanes away
          const int half = p.head_dim >> 1, hl = p.head_dim >> 3;
          float4 o;
          o.x = __shfl_xor_sync(0xffffffffu, v.x, hl); o.y = __shfl_xor_sync(0xffffffffu, v.y, hl);
          o.z = __shfl_xor_sync(0xffffffffu, v.z, hl); o.w = __shfl_xor_sync(0xffffffffu, v.w, hl);
          if (on && meta[q].x >= 0) {
            const int head = col / p.head_dim, dim = col % p.head_dim;
            const bool low = dim < half;
            float a[4] = {v.x * scale[q], v.y * scale[q], v.z * scale[q], v.w * scale[q]};
            if (head < p.hq + p.hkv) {
              const float b[4] = {o.x * scale[q], o.y * scale[q], o.z * scale[q], o.w * scale[q]};
              const float cx[4] = {cs0[q].x, cs0[q].z, cs1[q].x, cs1[q].z}, cy[4] = {cs0[q].y, cs0[q].w, cs1[q].y, cs1[q].w};
#pragma unroll
              for (int e = 0; e < 4; ++e)
                a[e] = low ? a[e] * cx[e] - b[e] * cy[e] : a[e] * cx[e] + b[e] * cy[e];   // (lo c - hi s) | (hi c + lo s)
            }
            store4<bf16>(epi_qkv_dst(p, row, head, dim, meta[q]), a[0], a[1], a[2], a[3]);
          }
        } else if (EPI == TC_ADD_NORM) {
          if (on) {
            float* x = (float*)p.C + (int64_t)row * p.ldc + col;
            v.x += xo[q].x; v.y += xo[q].y; v.z += xo[q].z; v.w += xo[q].w;
            *(float4*)x = v;
            store4<bf16>(p.xg_out + (int64_t)row * p.N + col, v.x * gn.x, v.y * gn.y, v.z * gn.z, v.w * gn.w);
            ssq[q] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          }
        } else if (EPI == TC_ADD_F32) {
          if (on) {
            float* x = (float*)p.C + (int64_t)row * p.ldc + col;
            *(float4*)x = make_float4(v.x + xo[q].x, v.y + xo[q].y, v.z + xo[q].z, v.w + xo[q].w);
          }
        } else if (EPI == TC_STORE_F32) {
          if (on) *(float4*)((float*)p.C + (int64_t)row * p.ldc + col) = v;
        } else if (EPI == TC_STORE_BF16) {
          if (on) store4<bf16>((bf16*)p.C + (int64_t)row * p.ldc + col, v.x, v.y, v.z, v.w);
        }
      }
    }
    if (EPI == TC_ADD_NORM) {
#pragma unroll
      for (int q = 0; q < RB; ++q) {
        const float t = warp_sum(ssq[q]);
        if (lane == 0 && row0 + rb + q < p.M) p.ssq_out[(int64_t)(row0 + rb + q) * p.ssq_out_parts + part_index] = t;
      }
    }
  }
}

template <int EPI>
__device__ __forceinline__ void epi_reduce_rows(const TcParams& p, int row0, int col0, int n_cols, int part_index, int lane) {
  if (p.splits <= 2) epi_reduce_rows_t<EPI, 8, 2>(p, row0, col0, n_cols, part_index, lane);
  else epi_reduce_rows_t<EPI, 8, 4>(p, row0, col0, n_cols, part_index, lane);
}

// Arrival of one epilogue warp at unit `ctr_index` after it has stored its part of the partial plane.
// True in the warp that arrived last (of p.splits): it may read all planes.
__device__ __forceinline__ bool epi_arrive_last(const TcParams& p, int ctr_index, int lane) {
  __threadfence();                                   // this lane's plane stores are visible device-wide ...
  __syncwarp();                                      // ... for every lane, before the warp is counted in
  int last = 0;
  if (lane == 0) {
    const int old = atomicAdd(p.tile_ctr + ctr_index, 1);
    last = (old == p.splits - 1);
    if (last) p.tile_ctr[ctr_index] = 0;             // every split has arrived: ready for the next launch
  }
  last = __shfl_sync(0xffffffffu, last, 0);
  if (last) __threadfence();                         // order the plane loads after the observed arrivals
  return last != 0;
}

}  // namespace rpo
