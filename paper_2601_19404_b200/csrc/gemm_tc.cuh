// bf16 GEMM on the 5th-generation tensor cores: C[M,N] = A[M,K] * W[N,K]^T, float32 accumulation.
//
//   * operands: TMA (cp.async.bulk.tensor.2d, every CTA fetching its own tiles) into 128-byte-swizzled shared memory,
//     a ring of NS stages of [128 x 64] (A) and [BN x 64] (W) tiles guarded by mbarriers;
//   * math: tcgen05.mma kind::f16 (bf16 x bf16 -> f32), M = 128, N = BN, K = 16 per instruction,
//     issued by one thread; accumulators live in tensor memory, two buffers of BN columns so the
//     epilogue of one tile overlaps the main loop of the next;
//   * epilogue: four warps read their 32-lane quadrant with tcgen05.ld and apply one of
//     {store bf16, store f32, add into the f32 residual stream, SwiGLU on interleaved gate/up
//     columns, store f32 split-K partial};
//   * persistent CTAs walk work items (tile_m, tile_n, k-split); split-K keeps all SMs streaming
//     weights when M is a decode batch.  Partials are reduced in fixed order by the next kernel.
//   * every mbarrier wait is bounded (clock64); on expiry the CTA raises STATUS_TIMEOUT, lets
//     copies in flight land, frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include <map>
#include <tuple>

#include "common.cuh"
#include "context.h"
#include "gemm_epi.cuh"

namespace rpo {

constexpr int TC_BM = 128, TC_BK = 64;
// Limit of every bounded device-side wait, in SM clock cycles (~0.1 s at 2 GHz by default: a thousand
// times the longest legitimate wait of these kernels).  One value per device and library image, shared
// by all contexts on the device; rpo_set_option("wait_limit_cycles") changes it.
constexpr long long TC_TIMEOUT_CYCLES_DEFAULT = 200000000LL;
__device__ long long g_wait_limit_cycles = TC_TIMEOUT_CYCLES_DEFAULT;

namespace tc {

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: false when the time limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64(), limit = g_wait_limit_cycles;
  while (!mbar_try_wait(bar, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) { *abort_flag = 1; return false; }
  }
  return true;
}

// The same for a whole warp that goes on to warp-wide (.sync.aligned) instructions: either every lane
// saw the phase complete, or all of them give up together.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  const bool ok = mbar_wait(bar, parity, abort_flag);
  return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

// Untiled bulk copy global -> shared (both 16-byte aligned, size a multiple of 16), completion on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: rows of 128 bytes, groups of
// 8 rows 1024 bytes apart (SBO), descriptor version 1 (sm_100), layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Registers back into tensor memory: 32 columns of this warp's 32 lanes.
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]),
        "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]),
        "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// 16 columns of this warp's 32 lanes.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// tcgen05.ld without the wait: several loads can be in flight before one tmem_ld_wait().
__device__ __forceinline__ void tmem_ld32_nowait(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

}  // namespace tc

template <int BN>
struct TcCfg {
  static constexpr int A_BYTES = TC_BM * TC_BK * 2;
  static constexpr int B_BYTES = BN * TC_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int NS = (200 * 1024 / STAGE_BYTES) > 8 ? 8 : (200 * 1024 / STAGE_BYTES);
  static constexpr int TMEM_COLS = (2 * BN <= 32) ? 32 : (2 * BN <= 64) ? 64 : (2 * BN <= 128) ? 128 : (2 * BN <= 256) ? 256 : 512;   // power of two
  static constexpr int SMEM_BYTES = NS * STAGE_BYTES + 1024 /*align*/ + 256 /*barriers*/;
};

// 192 threads: warp 0 = TMA producer, warp 1 = MMA issuer (+ TMEM owner), warps 2..5 = epilogue.
template <int BN, int EPI>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, TcParams p) {
  using Cfg = TcCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = (uint64_t*)(smem + Cfg::NS * Cfg::STAGE_BYTES);
  uint64_t* full = bars;
  uint64_t* empty = bars + Cfg::NS;
  uint64_t* acc_full = bars + 2 * Cfg::NS;
  uint64_t* acc_empty = bars + 2 * Cfg::NS + 2;
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * Cfg::NS + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_items = p.tiles_m * p.tiles_n * p.splits;
  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < Cfg::NS; ++i) { tc::mbar_init(&full[i], 1); tc::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)),
                 "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::tmem_fence_before();
  __syncthreads();
  tc::tmem_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      // The weight matrix does not depend on the kernel running before this one: the W tiles of
      // this CTA's first work item go into the (still empty) ring first, then the producer waits
      // for the predecessor and sends the matching A tiles after them.
      int pre = 0;
      if ((int)blockIdx.x < n_items) {
        const int split = blockIdx.x % p.splits, t = blockIdx.x / p.splits;
        const int tn = t % p.tiles_n, tm = t / p.tiles_n;
        const int kb0 = split * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        pre = min(Cfg::NS, kb1 - kb0);
        for (int i = 0; i < pre; ++i) {
          tc::mbar_expect_tx(&full[i], Cfg::STAGE_BYTES);
          tc::tma_load_2d(smem + i * Cfg::STAGE_BYTES + Cfg::A_BYTES, &map_w, (kb0 + i) * TC_BK, tn * BN, &full[i]);
        }
        pdl_wait();
        for (int i = 0; i < pre; ++i)
          tc::tma_load_2d(smem + i * Cfg::STAGE_BYTES, &map_a, (kb0 + i) * TC_BK, tm * TC_BM, &full[i]);
      } else {
        pdl_wait();
      }
      int stage = pre % Cfg::NS; uint32_t phase = (pre == Cfg::NS) ? 1u : 0u;
      bool ok = true;
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        const int split = it % p.splits, t = it / p.splits;
        const int tn = t % p.tiles_n, tm = t / p.tiles_n;
        const int kb0 = split * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        for (int kb = kb0 + (it == (int)blockIdx.x ? pre : 0); kb < kb1; ++kb) {
          if (!tc::mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * Cfg::STAGE_BYTES;
          tc::mbar_expect_tx(&full[stage], Cfg::STAGE_BYTES);
          tc::tma_load_2d(sa, &map_a, kb * TC_BK, tm * TC_BM, &full[stage]);
          tc::tma_load_2d(sa + Cfg::A_BYTES, &map_w, kb * TC_BK, tn * BN, &full[stage]);
          if (++stage == Cfg::NS) { stage = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        const int split = it % p.splits;
        const int kb0 = split * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        if (!tc::mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc::tmem_fence_after();
          const uint32_t sa = tc::smem_u32(smem + stage * Cfg::STAGE_BYTES);
          const uint64_t da = tc::umma_desc_sw128(sa), db = tc::umma_desc_sw128(sa + Cfg::A_BYTES);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)   // +32 bytes per K=16 step inside the 128-byte swizzled row
            tc::umma_bf16(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          tc::umma_commit(&empty[stage]);            // frees the stage once these MMAs have read it
          if (++stage == Cfg::NS) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc::umma_commit(&acc_full[acc]);             // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                       // TMEM lane quadrant this warp may read
    pdl_wait();                                      // the epilogue reads / overwrites what earlier kernels produced
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    const bool split_k = p.splits > 1;
    for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
      const int split = it % p.splits, t = it / p.splits;
      const int tn = t % p.tiles_n, tm = t / p.tiles_n;
      const int row = tm * TC_BM + quad * 32 + lane;
      // what the epilogue needs besides the sums is requested before the wait for the accumulator
      float scale = 1.f;
      int4 meta = make_int4(-1, 0, 0, 0);
      if (tc_epi_scaled(EPI) && !split_k) scale = epi_row_scale(p, row);
      if (EPI == TC_QKV_ROPE && !split_k && row < p.M) meta = p.row_meta[row];
      if (!tc::mbar_wait(&acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc::tmem_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * BN);
      if (split_k) {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          tc_store_chunk<TC_PARTIAL>(p, r, row, tn * BN + c0, split);
        }
      } else if (EPI == TC_QKV_ROPE) {
        const int half = p.head_dim >> 1;
#pragma unroll 1
        for (int h0 = 0; h0 < BN; h0 += p.head_dim) {
#pragma unroll 1
          for (int j = 0; j < half; j += 32) {
            uint32_t lo[32], hi[32];
            tc::tmem_ld32_nowait(t_row + (uint32_t)(h0 + j), lo);
            tc::tmem_ld32_nowait(t_row + (uint32_t)(h0 + j + half), hi);
            tc::tmem_ld_wait();
            epi_rope_pair(p, lo, hi, row, tn * BN + h0 + j, scale, meta);
          }
        }
      } else if (EPI == TC_ADD_NORM) {
        float ss = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          ss += epi_add_norm_chunk(p, r, row, tn * BN + c0);
        }
        if (row < p.M) p.ssq_out[(int64_t)row * p.ssq_out_parts + tn] = ss;
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          if (EPI == TC_NSTORE_F32 || EPI == TC_NSWIGLU) epi_scaled_chunk<EPI>(p, r, row, tn * BN + c0, scale, false);
          else tc_store_chunk<EPI>(p, r, row, tn * BN + c0, split);
        }
      }
      tc::tmem_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&acc_empty[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      // split-K with an epilogue of its own: the last warp to arrive at these 32 rows of the tile reduces them
      if (split_k && EPI != TC_PARTIAL && epi_arrive_last(p, (tm * p.tiles_n + tn) * 4 + quad, lane))
        epi_reduce_rows<EPI>(p, tm * TC_BM + quad * 32, tn * BN, BN, tn, lane);
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc::tmem_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000000);   // let bulk copies in flight land before smem goes away
    __syncthreads();
  }
  if (warp == 1) {
    tc::tmem_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  EncodeTiledFn encode = nullptr;
  std::map<std::tuple<const void*, int, int, int>, CUtensorMap> maps;   // (ptr, rows, cols, box_rows)
  bool attrs_set = false;
};

inline int tc_create(rpo_ctx* c) {
  TcState* s = new TcState();
  c->tc_state = s;
  if (!c->bf16) return RPO_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
  cudaError_t e = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &q);
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    fn = nullptr;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
  }
  if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    fprintf(stderr, "[rpo] cuTensorMapEncodeTiled unavailable (%s, query %d): tensor-core GEMM disabled\n",
            cudaGetErrorName(e), (int)q);
    return RPO_OK;
  }
  s->encode = (EncodeTiledFn)fn;
  return RPO_OK;
}
inline void tc_destroy(rpo_ctx* c) { delete (TcState*)c->tc_state; c->tc_state = nullptr; }

// Row-major bf16 [rows, cols] with a [box_rows x 64] box, 128-byte swizzle, zero fill out of bounds.
inline const CUtensorMap* tc_map(rpo_ctx* c, const void* ptr, int rows, int cols, int box_rows) {
  TcState* s = (TcState*)c->tc_state;
  auto key = std::make_tuple(ptr, rows, cols, box_rows);
  auto it = s->maps.find(key);
  if (it != s->maps.end()) return &it->second;
  CUtensorMap m;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = s->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { fprintf(stderr, "[rpo] cuTensorMapEncodeTiled failed (%d)\n", (int)r); return nullptr; }
  if (s->maps.size() > 4096) s->maps.clear();
  return &(s->maps[key] = m);
}

template <typename T>
inline bool tc_gemm_supported(rpo_ctx* c, int M, int N, int K) { return false; }
template <>
inline bool tc_gemm_supported<bf16>(rpo_ctx* c, int M, int N, int K) {
  TcState* s = (TcState*)c->tc_state;
  return s && s->encode && M >= 1 && (K % TC_BK) == 0 && (N % 16) == 0;
}

// Inputs / outputs of the fused epilogues (gemm_epi.cuh) that the plain GEMM call does not have.
struct TcFuse {
  const float* ssq_in = nullptr; int ssq_in_parts = 0; int norm_dim = 0; float eps = 0.f;       // TC_N*
  float* ssq_out = nullptr; bf16* xg_out = nullptr; const float* gain = nullptr;                 // TC_ADD_NORM
  int ssq_out_parts = 0;                                                                         //   (out) parts per row written (TC_NLSE: units per row)
  float2* lse_parts = nullptr; float* lse_tgt = nullptr; const int32_t* lse_target = nullptr; float lse_inv_T = 1.f;   // TC_NLSE
  const int4* row_meta = nullptr; const float2* rope = nullptr; KVPool<bf16> pool = {}; int layer = 0, hq = 0, hkv = 0, head_dim = 0;   // TC_QKV_ROPE
};

constexpr int TC_CTR_CAPACITY = 1 << 16;     // arrival counters of a split-K launch (ints)

// cudaFuncSetAttribute has to be made once per device, not once per process.
inline bool tc_first_use_on_device(rpo_ctx* c, bool (&done)[64]) {
  const int d = (c->device >= 0 && c->device < 64) ? c->device : 0;
  if (done[d]) return false;
  done[d] = true;
  return true;
}

inline void tc_fill_fuse(rpo_ctx* c, TcParams& p, const TcFuse* f) {
  p.planes = c->ws.partial; p.tile_ctr = c->ws.tile_ctr;
  if (!f) return;
  p.ssq_in = f->ssq_in; p.ssq_in_parts = f->ssq_in_parts; p.inv_norm_dim = f->norm_dim > 0 ? 1.0f / (float)f->norm_dim : 0.f; p.eps = f->eps;
  p.ssq_out = f->ssq_out; p.xg_out = f->xg_out; p.gain = f->gain;
  p.row_meta = f->row_meta; p.rope = f->rope; p.pool = f->pool; p.layer = f->layer; p.hq = f->hq; p.hkv = f->hkv; p.head_dim = f->head_dim;
  p.lse_parts = f->lse_parts; p.lse_tgt = f->lse_tgt; p.lse_target = f->lse_target; p.lse_inv_T = f->lse_inv_T;
}

template <int BN, int EPI>
inline int tc_launch(rpo_ctx* c, const CUtensorMap* ma, const CUtensorMap* mw, const TcParams& p, int grid) {
  using Cfg = TcCfg<BN>;
  static bool attr_done[64] = {};
  if (tc_first_use_on_device(c, attr_done)) {
    if (cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) != cudaSuccess)
      return RPO_ERR_CUDA;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES; cfg.stream = c->stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = c->pdl_now() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, EPI>, *ma, *mw, p) == cudaSuccess ? RPO_OK : RPO_ERR_CUDA;
}

template <int BN>
inline int tc_launch_epi(rpo_ctx* c, int epi, const CUtensorMap* ma, const CUtensorMap* mw, const TcParams& p, int grid) {
  switch (epi) {
    case TC_STORE_BF16: return tc_launch<BN, TC_STORE_BF16>(c, ma, mw, p, grid);
    case TC_STORE_F32: return tc_launch<BN, TC_STORE_F32>(c, ma, mw, p, grid);
    case TC_ADD_F32: return tc_launch<BN, TC_ADD_F32>(c, ma, mw, p, grid);
    case TC_SWIGLU: return tc_launch<BN, TC_SWIGLU>(c, ma, mw, p, grid);
    case TC_NSTORE_F32: return tc_launch<BN, TC_NSTORE_F32>(c, ma, mw, p, grid);
    case TC_NSWIGLU: return tc_launch<BN, TC_NSWIGLU>(c, ma, mw, p, grid);
    case TC_ADD_NORM: return tc_launch<BN, TC_ADD_NORM>(c, ma, mw, p, grid);
    case TC_NLSE: return RPO_ERR_INVALID_ARG;            // pair kernel only
    case TC_QKV_ROPE:
      if constexpr (BN % 64 == 0) return tc_launch<BN, TC_QKV_ROPE>(c, ma, mw, p, grid);
      else return RPO_ERR_INVALID_ARG;
    default: return tc_launch<BN, TC_PARTIAL>(c, ma, mw, p, grid);
  }
}

// Tile width and split-K factor.  Two regimes:
//   * many row tiles (prefill, log-probs): tensor-bound; 256-wide tiles.
//   * few row tiles (decode): the launch streams the weight matrix once from HBM, so every SM must
//     be pulling weights all the time.  If 128-wide tiles alone give about one item per SM, use
//     them unsplit; otherwise (tile_n, k-split) items are sized by a small cost model fitted to
//     measurements: cost of an item ~ k-blocks x (W rows + a share for the A tile re-read from L2)
//     + a pipeline-fill term, cost of the launch = rounds x item cost + a term per split plane
//     (partials written and re-read by whoever reduces them).
// bn_multiple: the epilogue needs whole heads in a tile (RoPE pairs dims half a head apart).
struct TcPlan { int bn, splits, kb_per_split; };

inline TcPlan tc_plan(rpo_ctx* c, int M, int N, int K, int epi, bool allow_split, int bn_multiple = 1) {
  const int sms = c->sm_count, tiles_m = (M + TC_BM - 1) / TC_BM, kb_total = K / TC_BK;
  TcPlan best{256, 1, kb_total};
  const bool self_reduce = tc_epi_fused(epi);           // the kernel's last-arriving warps reduce the planes
  if (c->gemm_bn > 0 && c->gemm_bn < 384 && c->gemm_bn % bn_multiple == 0) {   // test / sweep override
    best.bn = c->gemm_bn;
    best.splits = (allow_split && c->gemm_splits > 0) ? std::min(c->gemm_splits, kb_total) : 1;
  } else if (tiles_m * ((N + 255) / 256) >= sms && tiles_m >= 4) {
    best.bn = 256;
  } else if (tiles_m * ((N + 127) / 128) * 20 >= sms * 17) {
    best.bn = 128;                                       // enough 128-wide tiles for every SM: no split
  } else {
    static const int widths[] = {128, 96, 64, 32};
    double best_cost = 1e30;
    for (int bn : widths) {
      if ((epi == TC_SWIGLU || epi == TC_NSWIGLU) && bn % 32) continue;
      if (bn % bn_multiple) continue;
      const int tiles = tiles_m * ((N + bn - 1) / bn);
      int max_splits = 1;
      if (allow_split && tiles < sms) max_splits = std::max(1, std::min(sms / tiles, kb_total / 2));
      for (int sp = 1; sp <= max_splits; ++sp) {
        const int kbs = (kb_total + sp - 1) / sp;
        const int real = (kb_total + kbs - 1) / kbs;
        if (real > 1 && (size_t)real * M * N > c->ws.partial_elems) continue;
        if (real > 1 && self_reduce && tiles * 4 > TC_CTR_CAPACITY) continue;
        const int rounds = (tiles * real + sms - 1) / sms;
        // planes reduced inside the kernel cost the last-arriving warp a serial pass per pair of planes
        const double plane_cost = self_reduce ? 45.0 * bn / 128.0 * real : 60.0 * real;
        const double cost = (double)rounds * (kbs * (bn + 40.0) + 600.0) + (real > 1 ? plane_cost : 0.0);
        if (cost < best_cost) { best_cost = cost; best.bn = bn; best.splits = real; }
      }
    }
  }
  best.kb_per_split = (kb_total + best.splits - 1) / best.splits;
  best.splits = (kb_total + best.kb_per_split - 1) / best.kb_per_split;
  if (best.splits > 1 && (size_t)best.splits * M * N > c->ws.partial_elems) { best.splits = 1; best.kb_per_split = kb_total; }
  return best;
}

// Plan and launch.  With allow_split the launch may split K.  For the fused epilogues (gemm_epi.cuh)
// the kernel reduces the planes itself and the caller sees a finished result.  For the plain ones it
// writes split-K partial planes [splits][M][N] (float32) to ws.partial instead of applying `epi`;
// `splits_out` then receives the number of planes (> 1) and the caller owns the reduction.
inline int tc_gemm_launch(rpo_ctx* c, const bf16* A, const bf16* W, void* C, int M, int N, int K, int epi, int ldc,
                          bool allow_split, int* splits_out, TcFuse* fuse = nullptr) {
  if (splits_out) *splits_out = 0;
  const int tiles_m = (M + TC_BM - 1) / TC_BM;
  const int kb_total = K / TC_BK;
  const int sms = c->sm_count;
  const int bn_multiple = (epi == TC_QKV_ROPE && fuse) ? fuse->head_dim : 1;
  const TcPlan plan = tc_plan(c, M, N, K, epi, allow_split, bn_multiple);
  const int bn = plan.bn, splits = plan.splits, kb_per_split = plan.kb_per_split;
  const int tiles_n = (N + bn - 1) / bn;
  TcParams p = {};
  p.C = C; p.M = M; p.N = N; p.K = K; p.ldc = ldc;
  p.tiles_m = tiles_m; p.tiles_n = tiles_n; p.splits = splits; p.kb_per_split = kb_per_split; p.kb_total = kb_total;
  p.split_stride = (int64_t)M * N; p.status = c->d_status;
  tc_fill_fuse(c, p, fuse);
  p.ssq_out_parts = tiles_n;
  if (fuse) fuse->ssq_out_parts = tiles_n;
  int use_epi = epi;
  if (splits > 1 && !tc_epi_fused(epi)) { use_epi = TC_PARTIAL; if (splits_out) *splits_out = splits; }
  const CUtensorMap* ma = tc_map(c, A, M, K, TC_BM);
  const CUtensorMap* mw = tc_map(c, W, N, K, bn);
  if (!ma || !mw) return RPO_ERR_CUDA;
  const int grid = std::min(tiles_m * tiles_n * splits, sms);
  switch (bn) {
    case 256: return tc_launch_epi<256>(c, use_epi, ma, mw, p, grid);
    case 128: return tc_launch_epi<128>(c, use_epi, ma, mw, p, grid);
    case 96: return tc_launch_epi<96>(c, use_epi, ma, mw, p, grid);
    case 64: return tc_launch_epi<64>(c, use_epi, ma, mw, p, grid);
    case 32: return tc_launch_epi<32>(c, use_epi, ma, mw, p, grid);
    default: return RPO_ERR_INVALID_ARG;
  }
}

template <typename T>
inline int tc_gemm(rpo_ctx*, const T*, const T*, void*, int, int, int, int) { return RPO_ERR_SHAPE; }

}  // namespace rpo
