// Shared device helpers: storage-type traits, Philox4x32-10, reproducible float32 functions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rpo {

constexpr int KV_BLOCK = 16;          // tokens per KV block
constexpr int STATUS_TIMEOUT = 1;     // device status bits
constexpr int STATUS_BAD_TOKEN = 2;
constexpr int STATUS_BAD_BLOCK = 4;

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(bf16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float x) { return __float2bfloat16_rn(x); }

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization attribute
// may start while its predecessor in the stream is still running; it must not touch global memory
// the predecessor writes (or reads, if this kernel overwrites it) before pdl_wait(), which returns
// once the predecessor grid has completed and its writes are visible.  pdl_launch_dependents()
// lets the successor's CTAs be scheduled early.  Both are no-ops for ordinary launches.
// The kernels read some of what their predecessor wrote with plain stores through bulk / tensor copies
// (the async proxy): the proxy fence after the wait orders those copies behind the predecessor's writes.
__device__ __forceinline__ void pdl_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("fence.proxy.async.global;" ::: "memory");
}
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_prologue() { pdl_launch_dependents(); pdl_wait(); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  counter (c0..c3), key (k0,k1) -> four 32-bit words.
// ---------------------------------------------------------------------------------------------
struct U4 { uint32_t x, y, z, w; };

__host__ __device__ __forceinline__ U4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                                    uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1; c3 = (uint32_t)p0; c0 = n0; c2 = n2;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  return U4{c0, c1, c2, c3};
}

// 24-bit uniform integer of (seed, sequence, step): counter = (step, seq_lo, seq_hi, 0).
__device__ __forceinline__ uint32_t sampler_u24(uint64_t seed, uint64_t seq, uint32_t step) {
  U4 r = philox4x32_10(step, (uint32_t)seq, (uint32_t)(seq >> 32), 0u, (uint32_t)seed, (uint32_t)(seed >> 32));
  return r.x >> 8;
}

// ---------------------------------------------------------------------------------------------
// Reproducible float32 ln / sincos / exp: IEEE add, mul, div, sqrt only, each rounded to nearest,
// never contracted into FMAs (the __f*_rn intrinsics are exempt from contraction).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float rmul(float a, float b) { return __fmul_rn(a, b); }
__device__ __forceinline__ float radd(float a, float b) { return __fadd_rn(a, b); }

// ln(u), u in (0,1], normal.  ln m = 2 atanh((m-1)/(m+1)) with m in (1/sqrt2, sqrt2].
__device__ __forceinline__ float ln_unit(float u) {
  uint32_t bits = __float_as_uint(u);
  int e = (int)(bits >> 23) - 127;
  float m = __uint_as_float((bits & 0x007FFFFFu) | 0x3F800000u);
  if (m > (float)1.41421356237309504880) { m = rmul(m, 0.5f); e += 1; }
  const float f = radd(m, -1.0f);
  const float s = __fdiv_rn(f, radd(2.0f, f));
  const float z = rmul(s, s);
  float t = (float)(1.0 / 11.0);
  t = radd(rmul(t, z), (float)(1.0 / 9.0));
  t = radd(rmul(t, z), (float)(1.0 / 7.0));
  t = radd(rmul(t, z), (float)(1.0 / 5.0));
  t = radd(rmul(t, z), (float)(1.0 / 3.0));
  t = radd(rmul(t, z), 1.0f);
  const float lnm = rmul(rmul(2.0f, s), t);
  return radd(rmul((float)e, (float)0.69314718055994530942), lnm);
}

// (sin, cos) of 2*pi*k24/2^24: exact quadrant from the top two bits, Taylor in [0, pi/2).
__device__ __forceinline__ void sincos_turn24(uint32_t k24, float* sn, float* cs) {
  const int q = (int)(k24 >> 22);
  const float r = (float)(k24 & 0x3FFFFFu);
  const float x = rmul(rmul(r, (float)(1.0 / 4194304.0)), (float)1.57079632679489661923);
  const float x2 = rmul(x, x);
  float ps = (float)(1.0 / 6227020800.0);
  ps = radd(rmul(ps, x2), (float)(-1.0 / 39916800.0));
  ps = radd(rmul(ps, x2), (float)(1.0 / 362880.0));
  ps = radd(rmul(ps, x2), (float)(-1.0 / 5040.0));
  ps = radd(rmul(ps, x2), (float)(1.0 / 120.0));
  ps = radd(rmul(ps, x2), (float)(-1.0 / 6.0));
  ps = radd(rmul(ps, x2), 1.0f);
  const float s = rmul(x, ps);
  float pc = (float)(-1.0 / 87178291200.0);
  pc = radd(rmul(pc, x2), (float)(1.0 / 479001600.0));
  pc = radd(rmul(pc, x2), (float)(-1.0 / 3628800.0));
  pc = radd(rmul(pc, x2), (float)(1.0 / 40320.0));
  pc = radd(rmul(pc, x2), (float)(-1.0 / 720.0));
  pc = radd(rmul(pc, x2), (float)(1.0 / 24.0));
  pc = radd(rmul(pc, x2), -0.5f);
  pc = radd(rmul(pc, x2), 1.0f);
  const float c = pc;
  *sn = (q == 0) ? s : (q == 1) ? c : (q == 2) ? -s : -c;
  *cs = (q == 0) ? c : (q == 1) ? -s : (q == 2) ? -c : s;
}

// exp(x), x <= 0; exactly 0 below -24.
__device__ __forceinline__ float exp_nonpos(float x) {
  if (x < -24.0f) return 0.0f;
  const float n = rintf(rmul(x, (float)1.44269504088896340736));
  float r = radd(x, -rmul(n, __uint_as_float(0x3F317200u)));
  r = radd(r, -rmul(n, (float)(0.69314718055994530942 - 0.693145751953125)));
  float p = (float)(1.0 / 5040.0);
  p = radd(rmul(p, r), (float)(1.0 / 720.0));
  p = radd(rmul(p, r), (float)(1.0 / 120.0));
  p = radd(rmul(p, r), (float)(1.0 / 24.0));
  p = radd(rmul(p, r), (float)(1.0 / 6.0));
  p = radd(rmul(p, r), 0.5f);
  p = radd(rmul(p, r), 1.0f);
  p = radd(rmul(p, r), 1.0f);
  const float scale = __uint_as_float((uint32_t)((int)n + 127) << 23);
  return rmul(p, scale);
}

// Quantised sampler weight: floor(exp(z - zmax) * 2^30).
__device__ __forceinline__ uint32_t sampler_weight(float z, float zmax) {
  const float e = exp_nonpos(radd(z, -zmax));
  return __float2uint_rz(rmul(e, 1073741824.0f));
}

}  // namespace rpo
