// Prefill / teacher-forced attention on the 5th-generation tensor cores (head_dim 128).
//
// One CTA = 128 consecutive query rows of one sequence and one query head, walking 128-key tiles of
// [shared prefix segment, all visible] ++ [the sequence's own segment, causal]:
//
//   S = Q K^T      tcgen05.mma, A = Q tile (TMA, 128-byte swizzle, K-major), B = K tile (KV blocks bulk-
//                  copied from the pool, whose block layout IS the 128-byte-swizzled K-major layout),
//                  accumulator in tensor memory, two buffers
//   softmax        eight warps, two threads per query row (= TMEM lane), 64 columns each: tcgen05.ld,
//                  online max / sum in the exp2 domain without any shuffle, P written to shared
//                  memory as bf16 in the swizzled K-major layout
//   O_tile = P V   tcgen05.mma, A = P (shared memory), B = V blocks as stored ([token][dim] rows of
//                  128 bytes = an MN-major operand), one MMA per 16-token block; accumulator in TMEM
//   O += O_tile    the row's running output lives in registers: O = O * 2^(m_old - m_new) + O_tile
//
// Warp roles: 0 = producer (bulk copies K/V, TMA Q), 1 = MMA issuer and TMEM owner, 2..9 = softmax
// (two warps per TMEM lane quadrant, each on half of the columns).
// All mbarrier waits are bounded; on expiry the CTA raises STATUS_TIMEOUT and leaves.
#pragma once
#include "attn_tc.cuh"

namespace rpo {

constexpr int T5_BM = 128, T5_BN = 128, T5_DH = 128;
constexpr int T5_NSK = 2, T5_NSV = 2;
constexpr int T5_TILE = T5_BN * T5_DH * 2;                       // 32 KB: one K or V tile, also Q and P
constexpr int T5_SMEM = (2 + T5_NSK + T5_NSV) * T5_TILE + 1024 + 256 + 3072;   // tiles, alignment, barriers, row-maximum exchange

struct Flash5Args {
  bf16* out; int out_cols;
  const int32_t* row_seq; const int32_t* row_t; const SeqDesc* seqs; const int32_t* block_table;
  KVPool<bf16> pool; int layer, hq, hkv; float scale_log2;
  const int2* tiles;      // (first row, number of rows <= 128)
  int q_col0;             // column of head 0's q inside a qkv row (0)
  int* status;
};

namespace t5 {
// K-major, 128-byte swizzle (same as the GEMM operands).
__device__ __forceinline__ uint64_t desc_k_sw128(uint32_t addr) { return tc::umma_desc_sw128(addr); }
// MN-major, 128-byte swizzle: rows of 128 bytes run along the N (head dim) axis, 8 rows (keys) form
// a 1024-byte swizzle atom; the second half of the head dims sits `mn_stride` bytes further (the
// leading byte offset), groups of 8 keys are `k_stride` bytes apart (the stride byte offset).
__device__ __forceinline__ uint64_t desc_mn_sw128(uint32_t addr, uint32_t mn_stride, uint32_t k_stride) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(mn_stride >> 4) << 16;
  d |= (uint64_t)(k_stride >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
}  // namespace t5

__global__ void __launch_bounds__(320, 1)
flash_attn_tc5_kernel(const __grid_constant__ CUtensorMap q_map, Flash5Args a) {
  pdl_prologue();
  extern __shared__ uint8_t t5_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)t5_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = tc::smem_u32(sm);
  const uint32_t sP = sQ + T5_TILE;
  const uint32_t sK = sP + T5_TILE;
  const uint32_t sV = sK + T5_NSK * T5_TILE;
  uint64_t* bars = (uint64_t*)(sm + (2 + T5_NSK + T5_NSV) * T5_TILE);
  uint64_t *full_k = bars, *empty_k = bars + 2, *full_v = bars + 4, *empty_v = bars + 6;
  uint64_t *s_full = bars + 8, *s_free = bars + 10;            // per S buffer
  uint64_t *p_full = bars + 12, *o_full = bars + 13, *o_free = bars + 14, *q_full = bars + 15;
  uint32_t* tmem_slot = (uint32_t*)(bars + 16);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // grid (heads, tiles): the heads of one row tile run together (the query heads of a KV head
  // share its K/V in L2), and the tile list is ordered heaviest first
  const int2 tile = a.tiles[blockIdx.y];
  const int head = blockIdx.x, kvh = head / (a.hq / a.hkv);
  const int row0 = tile.x, n_rows = tile.y;
  const SeqDesc sd = a.seqs[a.row_seq[row0]];

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(&full_k[i], 1); tc::mbar_init(&empty_k[i], 1);
      tc::mbar_init(&full_v[i], 1); tc::mbar_init(&empty_v[i], 1);
      tc::mbar_init(&s_full[i], 1); tc::mbar_init(&s_free[i], 8);
    }
    tc::mbar_init(p_full, 8); tc::mbar_init(o_full, 1); tc::mbar_init(o_free, 8); tc::mbar_init(q_full, 1);
    for (int i = 0; i < 4; ++i) tc::mbar_init(&bars[17 + i], 2);      // one per lane quadrant: its two softmax warps
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::tmem_fence_before();
  __syncthreads();
  tc::tmem_fence_after();
  const uint32_t tmem = *tmem_slot;

  // ---- key ranges: the causal limit of the tile is its largest private index
  int t_max = -1;
  for (int i = lane; i < n_rows; i += 32) t_max = max(t_max, a.row_t[row0 + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t_max = max(t_max, __shfl_xor_sync(0xffffffffu, t_max, o));
  const int sh_end = (sd.shared_tbl >= 0) ? sd.shared_len : 0;
  const int pr_end = t_max + 1;
  const int n_sh = (sh_end + T5_BN - 1) / T5_BN, n_tiles = n_sh + (pr_end + T5_BN - 1) / T5_BN;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
      tc::mbar_expect_tx(q_full, T5_TILE);
      tc::tma_load_2d((void*)sm, &q_map, a.q_col0 + head * T5_DH, row0, q_full);
      tc::tma_load_2d((void*)(sm + T5_TILE / 2), &q_map, a.q_col0 + head * T5_DH + 64, row0, q_full);
    }
    bool ok = true;
    // lane b < 8: block of keys key0 + 16 b .. of tile `it` (past the end: the last valid one).  The look-up of
    // tile it + 1 is requested before tile it is waited for and sent.
    auto lookup = [&](int it) -> int {
      const bool shared_tile = it < n_sh;
      const int tbl = shared_tile ? sd.shared_tbl : sd.priv_tbl;
      const int key0 = shared_tile ? it * T5_BN : (it - n_sh) * T5_BN, limit = shared_tile ? sh_end : pr_end;
      const int nb = max(1, min(T5_BN / KV_BLOCK, (limit - key0 + KV_BLOCK - 1) / KV_BLOCK));
      return (lane < T5_BN / KV_BLOCK) ? a.block_table[tbl + (key0 + min(lane, nb - 1) * KV_BLOCK) / KV_BLOCK] : 0;
    };
    int blk_next = (n_tiles > 0) ? lookup(0) : 0;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int st = it & 1;
      const uint32_t par = ((it >> 1) & 1) ^ 1;
      int blk = blk_next;
      if (it + 1 < n_tiles) blk_next = lookup(it + 1);
      if (blk < 0 || blk >= a.pool.n_blocks) { atomicOr(a.status, STATUS_BAD_BLOCK); blk = 0; }
      if (lane == 0) { ok = tc::mbar_wait(&empty_k[st], par, abort_flag); if (ok) tc::mbar_expect_tx(&full_k[st], T5_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      {   // K: block b, half h -> plane h, rows 16 b ..: the K-major swizzled tile
        const int b = lane >> 1, h = lane & 1;
        const int kb = __shfl_sync(0xffffffffu, blk, b & 7);
        if (lane < 16)
          tc::bulk_load(sK + st * T5_TILE + h * (T5_TILE / 2) + b * 2048, a.pool.block(a.layer, 0, kvh, kb) + h * 1024, 2048, &full_k[st]);
      }
      if (lane == 0) { ok = tc::mbar_wait(&empty_v[st], par, abort_flag); if (ok) tc::mbar_expect_tx(&full_v[st], T5_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < T5_BN / KV_BLOCK)            // V: block b verbatim
        tc::bulk_load(sV + st * T5_TILE + lane * 4096, a.pool.block(a.layer, 1, kvh, blk), 4096, &full_v[st]);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(T5_BN >> 3) << 17) | ((uint32_t)(T5_BM >> 4) << 24);
      constexpr uint32_t idesc_pv = idesc_qk | (1u << 16);                 // B operand (V) is MN-major
      // operand descriptors built once: inside the loop a descriptor is a base plus a constant number of 16-byte units
      const uint64_t dq = t5::desc_k_sw128(sQ), dk = t5::desc_k_sw128(sK), dp = t5::desc_k_sw128(sP);
      const uint64_t dv = t5::desc_mn_sw128(sV, 2048, 1024);
      bool ok = tc::mbar_wait(q_full, 0, abort_flag);
      auto issue_qk = [&](int it) -> bool {
        const int st = it & 1, sb = it & 1;
        if (!tc::mbar_wait(&full_k[st], (it >> 1) & 1, abort_flag)) return false;
        if (!tc::mbar_wait(&s_free[sb], ((it >> 1) & 1) ^ 1, abort_flag)) return false;
        tc::tmem_fence_after();
        const uint64_t dks = dk + (uint64_t)(st * (T5_TILE >> 4));
#pragma unroll
        for (int k = 0; k < T5_DH / 16; ++k) {                             // dim half plane (k / 4), 32 bytes per 16 dims
          const uint64_t off = (uint64_t)((k >> 2) * (T5_TILE >> 5) + (k & 3) * 2);
          tc::umma_bf16(tmem + sb * T5_BN, dq + off, dks + off, idesc_qk, k > 0);
        }
        tc::umma_commit(&empty_k[st]);
        tc::umma_commit(&s_full[sb]);
        return true;
      };
      if (ok && n_tiles > 0) ok = issue_qk(0);
      for (int it = 0; it < n_tiles && ok; ++it) {
        if (it + 1 < n_tiles) { ok = issue_qk(it + 1); if (!ok) break; }      // S(it+1) overlaps the softmax of tile it
        const int st = it & 1;
        if (!tc::mbar_wait(p_full, it & 1, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(&full_v[st], (it >> 1) & 1, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(o_free, (it & 1) ^ 1, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        const uint64_t dvs = dv + (uint64_t)(st * (T5_TILE >> 4));
#pragma unroll
        for (int b = 0; b < T5_BN / KV_BLOCK; ++b)                           // 16 keys per MMA = one KV block
          tc::umma_bf16(tmem + 2 * T5_BN, dp + (uint64_t)((b >> 2) * (T5_TILE >> 5) + (b & 3) * 2), dvs + (uint64_t)(b * 256), idesc_pv, b > 0);
        tc::umma_commit(&empty_v[st]);
        tc::umma_commit(o_full);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    // Eight warps: warps w and w+4 serve the same TMEM lane quadrant (32 query rows) and split the
    // columns: thread (row r, half hf) owns keys / output dims [64 hf, 64 hf + 64).  The two threads
    // of a row agree on the running maximum through shared memory once per tile.
    const int sw = warp - 2, quad = warp & 3, hf = sw >> 2, r = quad * 32 + lane;
    const bool row_valid = r < n_rows;
    const int t_row = row_valid ? a.row_t[row0 + r] : -1;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16) + hf * 64;
    float* xmax = reinterpret_cast<float*>(bars + 24);                 // [2 slots][2 halves][128 rows], then [2 halves][128] sums
    uint64_t* pair_bar = &bars[17 + quad];                             // bounded rendezvous of the row's two threads
    float o[64];
#pragma unroll
    for (int i = 0; i < 64; ++i) o[i] = 0.f;
    float m = -INFINITY, l = 0.f, corr = 0.f;
    bool ok = true;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int sb = it & 1;
      const bool shared_tile = it < n_sh;
      const int key0 = (shared_tile ? it * T5_BN : (it - n_sh) * T5_BN) + hf * 64;   // first key of my half
      const int lim = shared_tile ? sh_end - 1 : t_row;                       // last visible key of this row in the segment
      if (!tc::mbar_wait_warp(&s_full[sb], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tmem_fence_after();
      // my 64 scores, kept in registers for both passes
      uint32_t v[64];
      tc::tmem_ld32_nowait(t_lane + sb * T5_BN, v);
      tc::tmem_ld32_nowait(t_lane + sb * T5_BN + 32, v + 32);
      tc::tmem_ld_wait();
      const bool whole = key0 + 63 <= lim;
      float mx = -INFINITY;
      if (whole) {
#pragma unroll
        for (int j = 0; j < 64; ++j) mx = fmaxf(mx, __uint_as_float(v[j]));
      } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) if (key0 + j <= lim) mx = fmaxf(mx, __uint_as_float(v[j]));
      }
      mx *= a.scale_log2;
      xmax[(sb * 2 + hf) * 128 + r] = mx;
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(pair_bar);                               // release: my warp's maxima are written
      if (!tc::mbar_wait_warp(pair_bar, it & 1, abort_flag)) { ok = false; break; }
      mx = fmaxf(mx, xmax[(sb * 2 + (hf ^ 1)) * 128 + r]);
      const float m_new = fmaxf(m, mx), mu = (m_new == -INFINITY) ? 0.f : m_new;
      const float c_prev = corr;                                              // factor that goes with O_tile(it-1)
      corr = fa::ex2(m - mu);
      // fold the previous tile's P V into the running output (its MMAs also released the P buffer)
      if (it > 0) {
        if (!tc::mbar_wait_warp(o_full, (it - 1) & 1, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        uint32_t w[64];
        tc::tmem_ld32_nowait(t_lane + 2 * T5_BN, w);
        tc::tmem_ld32_nowait(t_lane + 2 * T5_BN + 32, w + 32);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 64; ++j) o[j] = o[j] * c_prev + __uint_as_float(w[j]);
        tc::tmem_fence_before();
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(o_free);
      }
      // P = 2^(s - m) as bf16 into the swizzled K-major tile (plane hf), row sum of my half
      float ps = 0.f;
      const uint32_t base = sP + hf * (T5_TILE / 2) + r * 128;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
          const int k = 8 * q + j;
          float p0 = fa::ex2(fmaf(__uint_as_float(v[k]), a.scale_log2, -mu));
          float p1 = fa::ex2(fmaf(__uint_as_float(v[k + 1]), a.scale_log2, -mu));
          if (!whole) { p0 = (key0 + k <= lim) ? p0 : 0.f; p1 = (key0 + k + 1 <= lim) ? p1 : 0.f; }
          ps += p0 + p1;
          pk[j >> 1] = fa::pack_bf16(p0, p1);
        }
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(base + ((q ^ (r & 7)) << 4)), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
      }
      l = l * corr + ps;
      m = m_new;
      tc::tmem_fence_before();
      t5::fence_async_smem();
      __syncwarp();
      if (lane == 0) { tc::mbar_arrive(&s_free[sb]); tc::mbar_arrive(p_full); }
    }
    if (ok && n_tiles > 0) {
      if (tc::mbar_wait_warp(o_full, (n_tiles - 1) & 1, abort_flag)) {
        tc::tmem_fence_after();
        uint32_t w[64];
        tc::tmem_ld32_nowait(t_lane + 2 * T5_BN, w);
        tc::tmem_ld32_nowait(t_lane + 2 * T5_BN + 32, w + 32);
        tc::tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 64; ++j) o[j] = o[j] * corr + __uint_as_float(w[j]);
      }
    }
    // the row's sum: both halves used the same sequence of maxima, so the partial sums just add
    xmax[512 + hf * 128 + r] = l;
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(pair_bar);
    if (ok && tc::mbar_wait_warp(pair_bar, n_tiles & 1, abort_flag)) l += xmax[512 + (hf ^ 1) * 128 + r];
    if (row_valid) {
      const float inv = (l > 0.f) ? 1.0f / l : 0.f;
      bf16* dst = a.out + (int64_t)(row0 + r) * a.out_cols + head * T5_DH + hf * 64;
#pragma unroll
      for (int i = 0; i < 64; i += 8) {
        uint4 w4;
        w4.x = fa::pack_bf16(o[i] * inv, o[i + 1] * inv); w4.y = fa::pack_bf16(o[i + 2] * inv, o[i + 3] * inv);
        w4.z = fa::pack_bf16(o[i + 4] * inv, o[i + 5] * inv); w4.w = fa::pack_bf16(o[i + 6] * inv, o[i + 7] * inv);
        *reinterpret_cast<uint4*>(dst + i) = w4;
      }
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();
  tc::tmem_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) atomicOr(a.status, STATUS_TIMEOUT);
    for (int i = 0; i < 64; ++i) __nanosleep(1000000);   // let copies in flight land before the shared memory goes away
    __syncthreads();
  }
  if (warp == 1) {
    tc::tmem_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
  }
}

}  // namespace rpo
