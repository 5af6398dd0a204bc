// bf16 GEMM on CTA pairs for passes of more than 128 rows (prefill, token log-probs, decode batches
// above 128 sequences): C[M,N] = A[M,K] * W[N,K]^T.
//
// A 128 x 256 tile per CTA needs 48 KB of operands per 64-wide k-block, and the path from L2 into
// shared memory, not the tensor pipe, then sets the pace.  Here two CTAs of a cluster share one
// 256 x 256 tile: `tcgen05.mma.cta_group::2` (M = 256, N = 256, K = 16) reads rows 128r..128r+127
// of the A tile and rows 128r..128r+127 of the W tile from the shared memory of the CTA of rank r,
// and leaves rows 128r.. of the accumulator in that CTA's tensor memory.  Each CTA therefore loads
// 32 KB per k-block for the same tensor-pipe time: two thirds of the operand traffic per flop.
//
//   * both CTAs run a TMA producer for their own halves (tensor loads qualified `.cta_group::2`,
//     each CTA fetching only what it needs itself), completing on the *leader's* (rank 0) full
//     barrier, which expects the bytes of both;
//   * the leader's MMA thread issues the pair-wide instructions and releases ring stages and
//     accumulators in both CTAs with one `tcgen05.commit` that arrives on both CTAs' barriers;
//   * each CTA drains its own 128 accumulator rows (two buffers of 256 columns = all 512 columns
//     of tensor memory, so the epilogue of one tile overlaps the main loop of the next) and tells
//     the leader when a buffer is free again (remote mbarrier arrive).
//   * persistent: cluster i walks work items i, i + n_clusters, ... (an item is a tile, or a
//     k-split of a tile when a deep, narrow matrix has fewer tiles than the machine has pairs);
//     tiles are ordered in bands of row tiles for L2 locality; every wait is bounded as in
//     gemm_tc.cuh; no CTA leaves before its peer (cluster barrier at the end).
//   * in a decode batch of 256 rows a pair streams every weight tile once for all rows, where
//     single-CTA tiles stream it once per 128-row tile; the W halves of a CTA's first item are
//     requested before the wait on the preceding kernel, as in gemm_tc.cuh.
#pragma once
#include "gemm_tc.cuh"

namespace rpo {

// RM = rows of the A tile per CTA: 128 (256 x 256 tiles) or 64 (128 x 256 tiles, for batches of at
// most 128 rows: the CTA then loads 8 KB of A per 16 KB of W, so more of the bytes it can keep in
// flight are weight bytes).  With 64 rows per CTA the accumulator of a CTA sits in all 128 lanes of
// tensor memory, lanes 0..63 holding columns 0..127 of its rows and lanes 64..127 columns 128..255.
template <int RM>
struct Tc2Cfg {
  static constexpr int A_BYTES = RM * TC_BK * 2;           // 16 KB or 8 KB
  static constexpr int W_BYTES = 128 * TC_BK * 2;          // 16 KB: 128 rows x 64 bf16
  static constexpr int STAGE_BYTES = A_BYTES + W_BYTES;
  static constexpr int NS = 192 * 1024 / STAGE_BYTES;      // 6 or 8
  static constexpr int ACC_COLS = RM == 128 ? 256 : 128;   // tensor-memory columns of one accumulator buffer
  static constexpr int SMEM_BYTES = NS * STAGE_BYTES + 1024 + 256;
};

namespace tc {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_addr), "r"(rank));
  return a;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Pair-wide TMA load into this CTA's shared memory; the bytes complete on `bar_cluster_addr`,
// which may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  const uint32_t z = 0;
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n}"
      ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(z) : "memory");
}
// Arrives (once all MMAs issued so far have completed) on the barrier at this shared-memory
// offset in every CTA of `cta_mask`.
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"(cta_mask) : "memory");
}

}  // namespace tc

// Tile order: bands of TC2_BAND row tiles, walked column by column, so the clusters working at
// the same time share a few A slabs and a few W slabs (both stay hot in L2) instead of one A slab
// and the whole weight matrix.
constexpr int TC2_BAND = 8;
__device__ __forceinline__ void tc2_tile(int it, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int per_band = TC2_BAND * tiles_n;
  const int band = it / per_band, r = it - band * per_band;
  const int h = min(TC2_BAND, tiles_m - band * TC2_BAND);
  tn = r / h;
  tm = band * TC2_BAND + (r - tn * h);
}

// 192 threads per CTA, clusters of two: warp 0 = TMA producer, warp 1 = tensor-memory owner (and,
// in the leader, MMA issuer), warps 2..5 = epilogue.  p.tiles_m / p.tiles_n count 256 x 256 tiles.
template <int EPI, int RM = 128>
__global__ void __launch_bounds__(192, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, TcParams p) {
  using Cfg = Tc2Cfg<RM>;
  constexpr int TC2_NS = Cfg::NS, TC2_STAGE_BYTES = Cfg::STAGE_BYTES, TC2_HALF_BYTES = Cfg::A_BYTES;   // W tile follows the A tile
  constexpr int TM = 2 * RM;                     // rows of a pair tile
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = (uint64_t*)(smem + TC2_NS * TC2_STAGE_BYTES);
  uint64_t* full = bars;                         // used in the leader only
  uint64_t* empty = bars + TC2_NS;
  uint64_t* acc_full = bars + 2 * TC2_NS;
  uint64_t* acc_empty = bars + 2 * TC2_NS + 2;   // used in the leader only
  uint32_t* tmem_slot = (uint32_t*)(bars + 2 * TC2_NS + 4);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = tc::cluster_ctarank();
  const bool leader = (rank == 0);
  const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
  const int n_items = p.tiles_m * p.tiles_n * p.splits;    // work item = (tile, k-split), split fastest
  pdl_launch_dependents();

  if (threadIdx.x == 0) {
    for (int i = 0; i < TC2_NS; ++i) { tc::mbar_init(&full[i], 1); tc::mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { tc::mbar_init(&acc_full[i], 1); tc::mbar_init(&acc_empty[i], 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)),
                 "r"((uint32_t)(2 * Cfg::ACC_COLS)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc::tmem_fence_before();
  __syncthreads();
  tc::cluster_sync_all();                        // the peer's barriers exist before anything arrives on them
  tc::tmem_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_w) : "memory");
      // The weights do not depend on the kernel running before this one: the W halves of the first
      // tile go into the (still empty) ring before the wait for the predecessor, the A halves after.
      int pre = 0;
      if (cluster_id < n_items) {
        int tm, tn;
        tc2_tile(cluster_id / p.splits, p.tiles_m, p.tiles_n, tm, tn);
        const int kb0 = (cluster_id % p.splits) * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        pre = min(TC2_NS, kb1 - kb0);
        for (int i = 0; i < pre; ++i) {
          if (leader) tc::mbar_expect_tx(&full[i], 2 * TC2_STAGE_BYTES);
          tc::tma_load_2d_pair(smem + i * TC2_STAGE_BYTES + TC2_HALF_BYTES, &map_w, (kb0 + i) * TC_BK, tn * 256 + (int)rank * 128,
                               tc::map_to_rank(tc::smem_u32(&full[i]), 0));
        }
        pdl_wait();
        for (int i = 0; i < pre; ++i)
          tc::tma_load_2d_pair(smem + i * TC2_STAGE_BYTES, &map_a, (kb0 + i) * TC_BK, tm * TM + (int)rank * RM,
                               tc::map_to_rank(tc::smem_u32(&full[i]), 0));
      } else {
        pdl_wait();
      }
      int stage = pre % TC2_NS; uint32_t phase = (pre == TC2_NS) ? 1u : 0u;
      bool ok = true;
      for (int it = cluster_id; it < n_items && ok; it += n_clusters) {
        int tm, tn;
        tc2_tile(it / p.splits, p.tiles_m, p.tiles_n, tm, tn);
        const int kb0 = (it % p.splits) * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        const int row_a = tm * TM + (int)rank * RM, row_w = tn * 256 + (int)rank * 128;
        for (int kb = kb0 + (it == cluster_id ? pre : 0); kb < kb1; ++kb) {
          if (!tc::mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * TC2_STAGE_BYTES;
          if (leader) tc::mbar_expect_tx(&full[stage], 2 * TC2_STAGE_BYTES);
          const uint32_t bar = tc::map_to_rank(tc::smem_u32(&full[stage]), 0);
          tc::tma_load_2d_pair(sa, &map_a, kb * TC_BK, row_a, bar);
          tc::tma_load_2d_pair(sa + TC2_HALF_BYTES, &map_w, kb * TC_BK, row_w, bar);
          if (++stage == TC2_NS) { stage = 0; phase ^= 1; }
        }
      }
      // Drain: every stage this CTA filled has been released, i.e. all arrivals aimed at this
      // CTA's barriers have landed before its shared memory goes away.
      for (int i = 0; i < TC2_NS && ok; ++i) {
        if (!tc::mbar_wait(&empty[stage], phase ^ 1, abort_flag)) ok = false;
        if (++stage == TC2_NS) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (leader && lane == 0) {
      constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(TM >> 4) << 24);
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true;
      for (int it = cluster_id; it < n_items && ok; it += n_clusters) {
        if (!tc::mbar_wait(&acc_empty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * Cfg::ACC_COLS);
        const int kb0 = (it % p.splits) * p.kb_per_split, kb1 = min(p.kb_total, kb0 + p.kb_per_split);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!tc::mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc::tmem_fence_after();
          const uint32_t sa = tc::smem_u32(smem + stage * TC2_STAGE_BYTES);
          const uint64_t da = tc::umma_desc_sw128(sa), db = tc::umma_desc_sw128(sa + TC2_HALF_BYTES);
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k)
            tc::umma_bf16_pair(d_tmem, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          tc::umma_commit_pair(&empty[stage], 3);       // frees the stage in both CTAs
          if (++stage == TC2_NS) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        tc::umma_commit_pair(&acc_full[acc], 3);        // accumulator complete, both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5, both CTAs)
    const int quad = warp & 3;
    const bool stream_out = p.M >= 2048;           // output far larger than L2: streaming stores
    const bool split_k = p.splits > 1;
    pdl_wait();
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int it = cluster_id; it < n_items && ok; it += n_clusters) {
      int tm, tn;
      tc2_tile(it / p.splits, p.tiles_m, p.tiles_n, tm, tn);
      // RM = 128: lane = row, 256 columns.  RM = 64: lanes 64.. hold columns 128..255 of rows 0..63.
      const int row0 = tm * TM + (int)rank * RM + (RM == 128 ? quad * 32 : (quad & 1) * 32);
      const int row = row0 + lane;
      const int col_base = tn * 256 + (RM == 128 ? 0 : (quad >> 1) * 128);
      const int part = RM == 128 ? tn : tn * 2 + (quad >> 1);         // column unit of this warp (TC_ADD_NORM statistics)
      float scale = 1.f;
      int4 meta = make_int4(-1, 0, 0, 0);
      if (tc_epi_scaled(EPI) && !split_k) scale = epi_row_scale(p, row);
      if (EPI == TC_QKV_ROPE && !split_k && row < p.M) meta = p.row_meta[row];
      if (!tc::mbar_wait(&acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc::tmem_fence_after();
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * Cfg::ACC_COLS);
      if (split_k) {
#pragma unroll 1
        for (int c0 = 0; c0 < Cfg::ACC_COLS; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          tc_store_chunk<TC_PARTIAL>(p, r, row, col_base + c0, it % p.splits, false);
        }
      } else if (EPI == TC_QKV_ROPE) {
        const int half = p.head_dim >> 1;
#pragma unroll 1
        for (int h0 = 0; h0 < Cfg::ACC_COLS; h0 += p.head_dim) {
#pragma unroll 1
          for (int j = 0; j < half; j += 32) {
            uint32_t lo[32], hi[32];
            tc::tmem_ld32_nowait(t_row + (uint32_t)(h0 + j), lo);
            tc::tmem_ld32_nowait(t_row + (uint32_t)(h0 + j + half), hi);
            tc::tmem_ld_wait();
            epi_rope_pair(p, lo, hi, row, col_base + h0 + j, scale, meta);
          }
        }
      } else if (EPI == TC_ADD_NORM) {
        float ss = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < Cfg::ACC_COLS; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          ss += epi_add_norm_chunk(p, r, row, col_base + c0);
        }
        if (row < p.M) p.ssq_out[(int64_t)row * p.ssq_out_parts + part] = ss;
      } else if (EPI == TC_NLSE) {
        float m = -INFINITY, s = 0.f, zt = 0.f;
        const int tgt = row < p.M ? p.lse_target[row] : -1;
#pragma unroll 1
        for (int c0 = 0; c0 < Cfg::ACC_COLS; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          epi_lse_chunk(p, r, col_base + c0, scale, tgt, m, s, zt);
        }
        if (row < p.M) {
          p.lse_parts[(int64_t)row * p.lse_stride + part] = make_float2(m, s);
          if (tgt >= col_base && tgt < col_base + Cfg::ACC_COLS) p.lse_tgt[row] = zt;
        }
      } else {
#pragma unroll 1
        for (int c0 = 0; c0 < Cfg::ACC_COLS; c0 += 32) {
          uint32_t r[32];
          tc::tmem_ld32(t_row + (uint32_t)c0, r);
          if (EPI == TC_NSTORE_F32 || EPI == TC_NSWIGLU) epi_scaled_chunk<EPI>(p, r, row, col_base + c0, scale, stream_out);
          else tc_store_chunk<EPI>(p, r, row, col_base + c0, it % p.splits, stream_out);
        }
      }
      tc::tmem_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive_cluster(tc::map_to_rank(tc::smem_u32(&acc_empty[acc]), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      // split-K with an epilogue of its own: the last warp to arrive at this 32-row unit reduces it
      if (split_k && EPI != TC_PARTIAL &&
          epi_arrive_last(p, (((tm * p.tiles_n + tn) * 2 + (int)rank) * 4 + quad), lane))
        epi_reduce_rows<EPI>(p, row0, col_base, Cfg::ACC_COLS, part, lane);
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc::tmem_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(p.status, STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000000);   // let copies in flight land before shared memory goes away
    __syncthreads();
  }
  tc::cluster_sync_all();                        // the peer no longer touches this CTA's barriers or tensor memory
  if (warp == 1) {
    tc::tmem_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)(2 * Cfg::ACC_COLS)) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <int EPI, int RM>
inline int tc2_launch(rpo_ctx* c, const CUtensorMap* ma, const CUtensorMap* mw, const TcParams& p) {
  using Cfg = Tc2Cfg<RM>;
  static int max_clusters_dev[64];
  static bool init_done[64] = {};
  const int dev_i = (c->device >= 0 && c->device < 64) ? c->device : 0;
  if (!init_done[dev_i]) { max_clusters_dev[dev_i] = -1; init_done[dev_i] = true; }
  int& max_clusters = max_clusters_dev[dev_i];
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = Cfg::SMEM_BYTES; cfg.stream = c->stream;
  cfg.attrs = attr;
  if (max_clusters < 0) {
    if (cudaFuncSetAttribute(gemm_tc2_kernel<EPI, RM>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM_BYTES) != cudaSuccess)
      return RPO_ERR_CUDA;
    cfg.gridDim = dim3(2 * (c->sm_count / 2)); cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc2_kernel<EPI, RM>, &cfg) != cudaSuccess || n < 1) { cudaGetLastError(); n = c->sm_count / 2; }
    max_clusters = std::min(n, c->sm_count / 2);
  }
  const int clusters = std::min(p.tiles_m * p.tiles_n * p.splits, max_clusters);
  cfg.gridDim = dim3(2 * clusters);
  cfg.numAttrs = c->pdl_now() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI, RM>, *ma, *mw, p) == cudaSuccess ? RPO_OK : RPO_ERR_CUDA;
}

// Rows per CTA of the pair kernel for a pass of M rows: 64 (128-row pair tiles) up to 128 rows,
// else 128 (256-row pair tiles).  gemm_bn = 384 / 512 force the one or the other (tests, sweeps).
inline int tc2_rows(rpo_ctx* c, int M) {
  if (c->gemm_bn == 384) return 64;
  if (c->gemm_bn == 512) return 128;
  return M <= 128 ? 64 : 128;
}

// Split-K factor of the pair kernel for a pass of few tiles: as many k-splits as give every CTA pair
// one work item in a single round, each at least eight k-blocks deep, within the partial workspace.
inline int tc2_splits(rpo_ctx* c, int M, int N, int K, bool allow_split) {
  const int tm = 2 * tc2_rows(c, M);
  const int tiles = ((M + tm - 1) / tm) * ((N + 255) / 256), pairs = c->sm_count / 2, kb_total = K / TC_BK;
  if (c->gemm_bn >= 384 && c->gemm_splits > 0) return allow_split ? std::max(1, std::min(c->gemm_splits, kb_total)) : 1;
  if (!allow_split || tiles >= pairs) return 1;
  int sp = std::max(1, std::min(pairs / tiles, kb_total / 8));
  while (sp > 1 && (size_t)sp * M * N > c->ws.partial_elems) --sp;
  return sp;
}

// True when pair tiles fill the machine.  More than 128 rows (prefill, log-prob passes, decode
// batches above 128 sequences): a pair streams each weight tile once for 256 rows instead of once
// per 128-row tile; deep narrow matrices are split along K to give every pair an item.  Up to 128
// rows: 64 rows per CTA, for matrices wide enough for several rounds of tiles (lm_head) - a
// weight-streaming launch runs as fast as it has weight bytes in flight, and a CTA that loads 8 KB
// of activations per 16 KB of weights keeps a third more of them in flight; launches of a single
// round lose more to the pair's start-up than they gain.
inline bool tc2_wanted(rpo_ctx* c, int M, int N, int K, bool allow_split) {
  if (c->gemm_bn > 0) return c->gemm_bn >= 384;           // test / sweep override: 384 / 512 = pair tiles
  if (!c->use_gemm_pairs) return false;
  const int tm = 2 * tc2_rows(c, M);
  const int tiles = ((M + tm - 1) / tm) * ((N + 255) / 256), sp = tc2_splits(c, M, N, K, allow_split);
  if (M <= 128) return c->use_gemm_pairs_small && M > 64 && tiles >= 3 * (c->sm_count / 2);   // several rounds: measured +6 % on lm_head, -10 % on one-round launches
  if (sp > 1 && K / TC_BK / sp < 32) return false;       // shallow splits: measured no better than single-CTA tiles
  return tiles * sp >= c->sm_count / 2 - 10;
}

// With allow_split the launch may split K: the fused epilogues (gemm_epi.cuh) reduce the planes inside
// the kernel; for the plain ones the planes [splits][M][N] stay in ws.partial instead of applying `epi`
// and *splits_out holds their number (> 1).
inline int tc2_gemm_launch(rpo_ctx* c, const bf16* A, const bf16* W, void* C, int M, int N, int K, int epi, int ldc,
                           bool allow_split, int* splits_out, TcFuse* fuse = nullptr) {
  if (splits_out) *splits_out = 0;
  const int rm = tc2_rows(c, M), tm = 2 * rm;
  TcParams p = {};
  p.C = C; p.M = M; p.N = N; p.K = K; p.ldc = ldc;
  p.tiles_m = (M + tm - 1) / tm; p.tiles_n = (N + 255) / 256; p.kb_total = K / TC_BK;
  int splits = (M <= 128 && c->gemm_bn == 0) ? 1 : tc2_splits(c, M, N, K, allow_split);
  if (tc_epi_fused(epi) && p.tiles_m * p.tiles_n * 8 > TC_CTR_CAPACITY) splits = 1;
  if (epi == TC_NLSE) splits = 1;
  p.kb_per_split = (p.kb_total + splits - 1) / splits;
  splits = (p.kb_total + p.kb_per_split - 1) / p.kb_per_split;
  if (splits > 1 && (size_t)splits * M * N > c->ws.partial_elems) { splits = 1; p.kb_per_split = p.kb_total; }
  p.splits = splits;
  p.split_stride = (int64_t)M * N; p.status = c->d_status;
  tc_fill_fuse(c, p, fuse);
  p.ssq_out_parts = rm == 128 ? p.tiles_n : 2 * p.tiles_n;
  p.lse_stride = p.ssq_out_parts;
  if (fuse) fuse->ssq_out_parts = p.ssq_out_parts;
  if (splits > 1 && !tc_epi_fused(epi)) { epi = TC_PARTIAL; if (splits_out) *splits_out = splits; }
  const CUtensorMap* ma = tc_map(c, A, M, K, rm);
  const CUtensorMap* mw = tc_map(c, W, N, K, 128);
  if (!ma || !mw) return RPO_ERR_CUDA;
  if (rm == 64) {
    switch (epi) {
      case TC_STORE_BF16: return tc2_launch<TC_STORE_BF16, 64>(c, ma, mw, p);
      case TC_STORE_F32: return tc2_launch<TC_STORE_F32, 64>(c, ma, mw, p);
      case TC_ADD_F32: return tc2_launch<TC_ADD_F32, 64>(c, ma, mw, p);
      case TC_SWIGLU: return tc2_launch<TC_SWIGLU, 64>(c, ma, mw, p);
      case TC_NSTORE_F32: return tc2_launch<TC_NSTORE_F32, 64>(c, ma, mw, p);
      case TC_NSWIGLU: return tc2_launch<TC_NSWIGLU, 64>(c, ma, mw, p);
      case TC_QKV_ROPE: return tc2_launch<TC_QKV_ROPE, 64>(c, ma, mw, p);
      case TC_ADD_NORM: return tc2_launch<TC_ADD_NORM, 64>(c, ma, mw, p);
      case TC_NLSE: return tc2_launch<TC_NLSE, 64>(c, ma, mw, p);
      default: return tc2_launch<TC_PARTIAL, 64>(c, ma, mw, p);
    }
  }
  switch (epi) {
    case TC_STORE_BF16: return tc2_launch<TC_STORE_BF16, 128>(c, ma, mw, p);
    case TC_STORE_F32: return tc2_launch<TC_STORE_F32, 128>(c, ma, mw, p);
    case TC_ADD_F32: return tc2_launch<TC_ADD_F32, 128>(c, ma, mw, p);
    case TC_SWIGLU: return tc2_launch<TC_SWIGLU, 128>(c, ma, mw, p);
    case TC_NSTORE_F32: return tc2_launch<TC_NSTORE_F32, 128>(c, ma, mw, p);
    case TC_NSWIGLU: return tc2_launch<TC_NSWIGLU, 128>(c, ma, mw, p);
    case TC_QKV_ROPE: return tc2_launch<TC_QKV_ROPE, 128>(c, ma, mw, p);
    case TC_ADD_NORM: return tc2_launch<TC_ADD_NORM, 128>(c, ma, mw, p);
    case TC_NLSE: return tc2_launch<TC_NLSE, 128>(c, ma, mw, p);
    default: return tc2_launch<TC_PARTIAL, 128>(c, ma, mw, p);
  }
}

}  // namespace rpo
