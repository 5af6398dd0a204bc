// Prefill / teacher-forced attention on the 5th-generation tensor cores, pipelined variant (head_dim 128).
//
// Same work item as flash_attn_tc5_kernel (128 consecutive query rows of one sequence and one query head
// against [shared prefix segment, all visible] ++ [the sequence's own segment, causal]) but built so that
// no step of a tile waits for the tile before it:
//
//   * 64-key tiles; S = Q K^T in two tensor-memory buffers, P in two shared-memory buffers, K and V in rings of
//     four tiles each;
//   * O += P V accumulates in tensor memory over all tiles.  P is taken relative to a reference maximum m_ref
//     per row that moves only when the running maximum has grown past it by more than 2^8: then, and only
//     then, the softmax warps wait for the MMAs issued so far and rescale the row's O and its sum.  Otherwise
//     the softmax of a tile waits for nothing but its S and a free P buffer, so the tensor pipe runs
//     Q K^T of tile i + 1 and P V of tile i - 1 while the softmax warps work on tile i;
//   * eight softmax warps, two threads per query row (32 keys and 64 output dims each).
//
// Warp roles: 0 = producer (TMA Q, bulk copies of K/V blocks), 1 = MMA issuer and tensor-memory owner,
// 2..9 = softmax.  All mbarrier waits are bounded; on expiry the CTA raises STATUS_TIMEOUT and leaves.
#pragma once
#include "attn_tc5.cuh"

namespace rpo {

constexpr int P5_BN = 64;                                      // keys per tile
constexpr int P5_NSK = 4, P5_NSV = 4;                          // ring depths
constexpr int P5_KV_TILE = P5_BN * T5_DH * 2;                  // 16 KB: one K or V tile, also one P buffer (128 rows x 64 keys)
constexpr int P5_Q_TILE = T5_BM * T5_DH * 2;                   // 32 KB
constexpr int P5_SMEM = P5_Q_TILE + (2 + P5_NSK + P5_NSV) * P5_KV_TILE + 1024 + 256 + 3072;   // tiles, alignment, barriers, row exchange
constexpr float P5_LAZY = 8.0f;                                // log2 of the largest P entry tolerated before m_ref moves

__global__ void __launch_bounds__(320, 1)
flash_prefill_tc5_kernel(const __grid_constant__ CUtensorMap q_map, Flash5Args a) {
  pdl_prologue();
  extern __shared__ uint8_t p5_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)p5_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = tc::smem_u32(sm);
  const uint32_t sP = sQ + P5_Q_TILE;
  const uint32_t sK = sP + 2 * P5_KV_TILE;
  const uint32_t sV = sK + P5_NSK * P5_KV_TILE;
  uint64_t* bars = (uint64_t*)(sm + P5_Q_TILE + (2 + P5_NSK + P5_NSV) * P5_KV_TILE);
  uint64_t *full_k = bars, *empty_k = bars + 4, *full_v = bars + 8, *empty_v = bars + 12;
  uint64_t *s_full = bars + 16, *s_free = bars + 18;            // per S buffer
  uint64_t *p_full = bars + 20, *p_free = bars + 22;            // per P buffer
  uint64_t *q_full = bars + 24, *pair_bars = bars + 25;         // one rendezvous per lane quadrant
  uint32_t* tmem_slot = (uint32_t*)(bars + 29);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int2 tile = a.tiles[blockIdx.y];
  const int head = blockIdx.x, kvh = head / (a.hq / a.hkv);
  const int row0 = tile.x, n_rows = tile.y;
  const SeqDesc sd = a.seqs[a.row_seq[row0]];

  if (threadIdx.x == 0) {
    for (int i = 0; i < P5_NSK; ++i) { tc::mbar_init(&full_k[i], 1); tc::mbar_init(&empty_k[i], 1); }
    for (int i = 0; i < P5_NSV; ++i) { tc::mbar_init(&full_v[i], 1); tc::mbar_init(&empty_v[i], 1); }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(&s_full[i], 1); tc::mbar_init(&s_free[i], 8);
      tc::mbar_init(&p_full[i], 8); tc::mbar_init(&p_free[i], 1);
    }
    tc::mbar_init(q_full, 1);
    for (int i = 0; i < 4; ++i) tc::mbar_init(&pair_bars[i], 2);      // the two softmax warps of a lane quadrant
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(256u) : "memory");
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
  const int n_sh = (sh_end + P5_BN - 1) / P5_BN, n_tiles = n_sh + (pr_end + P5_BN - 1) / P5_BN;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&q_map) : "memory");
      tc::mbar_expect_tx(q_full, P5_Q_TILE);
      tc::tma_load_2d((void*)sm, &q_map, a.q_col0 + head * T5_DH, row0, q_full);
      tc::tma_load_2d((void*)(sm + P5_Q_TILE / 2), &q_map, a.q_col0 + head * T5_DH + 64, row0, q_full);
    }
    bool ok = true;
    // lane b < 4: block of keys key0 + 16 b .. of tile `it` (past the end of the segment: the last valid one, finite
    // data that the softmax masks).  The look-up of tile it + 1 is requested before tile it is waited for and sent.
    auto lookup = [&](int it) -> int {
      const bool shared_tile = it < n_sh;
      const int tbl = shared_tile ? sd.shared_tbl : sd.priv_tbl;
      const int key0 = shared_tile ? it * P5_BN : (it - n_sh) * P5_BN, limit = shared_tile ? sh_end : pr_end;
      const int nb = max(1, min(P5_BN / KV_BLOCK, (limit - key0 + KV_BLOCK - 1) / KV_BLOCK));
      return (lane < P5_BN / KV_BLOCK) ? a.block_table[tbl + key0 / KV_BLOCK + min(lane, nb - 1)] : 0;
    };
    int blk_next = (n_tiles > 0) ? lookup(0) : 0;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int sk = it % P5_NSK, sv = it % P5_NSV;
      const uint32_t par_k = ((it / P5_NSK) & 1) ^ 1, par_v = ((it / P5_NSV) & 1) ^ 1;
      int blk = blk_next;
      if (it + 1 < n_tiles) blk_next = lookup(it + 1);
      if (blk < 0 || blk >= a.pool.n_blocks) { atomicOr(a.status, STATUS_BAD_BLOCK); blk = 0; }
      if (lane == 0) { ok = tc::mbar_wait(&empty_k[sk], par_k, abort_flag); if (ok) tc::mbar_expect_tx(&full_k[sk], P5_KV_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      {   // K: block b, half h -> plane h, rows 16 b ..: the K-major swizzled tile
        const int b = lane >> 1, h = lane & 1;
        const int kb = __shfl_sync(0xffffffffu, blk, b & 3);
        if (lane < 8)
          tc::bulk_load(sK + sk * P5_KV_TILE + h * (P5_KV_TILE / 2) + b * 2048, a.pool.block(a.layer, 0, kvh, kb) + h * 1024, 2048, &full_k[sk]);
      }
      if (lane == 0) { ok = tc::mbar_wait(&empty_v[sv], par_v, abort_flag); if (ok) tc::mbar_expect_tx(&full_v[sv], P5_KV_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < P5_BN / KV_BLOCK)            // V: block b verbatim
        tc::bulk_load(sV + sv * P5_KV_TILE + lane * 4096, a.pool.block(a.layer, 1, kvh, blk), 4096, &full_v[sv]);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(P5_BN >> 3) << 17) | ((uint32_t)(T5_BM >> 4) << 24);
      constexpr uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(T5_DH >> 3) << 17) | ((uint32_t)(T5_BM >> 4) << 24);   // B operand (V) is MN-major, N = 128 dims
      const uint64_t dq = t5::desc_k_sw128(sQ), dk = t5::desc_k_sw128(sK), dp = t5::desc_k_sw128(sP);
      const uint64_t dv = t5::desc_mn_sw128(sV, 2048, 1024);
      bool ok = tc::mbar_wait(q_full, 0, abort_flag);
      int sk_n = 0, sv_n = 0;                                                // ring stages of the next Q K^T / P V
      uint32_t phk = 0, phv = 0;                                             // and their phases
      auto issue_qk = [&](int it) -> bool {
        const int sb = it & 1;
        if (!tc::mbar_wait(&full_k[sk_n], phk, abort_flag)) return false;
        if (!tc::mbar_wait(&s_free[sb], ((it >> 1) & 1) ^ 1, abort_flag)) return false;
        tc::tmem_fence_after();
        const uint64_t dks = dk + (uint64_t)(sk_n * (P5_KV_TILE >> 4));
#pragma unroll
        for (int k = 0; k < T5_DH / 16; ++k)                                 // dim half plane (k / 4), 32 bytes per 16 dims
          tc::umma_bf16(tmem + sb * P5_BN, dq + (uint64_t)((k >> 2) * (P5_Q_TILE >> 5) + (k & 3) * 2),
                        dks + (uint64_t)((k >> 2) * (P5_KV_TILE >> 5) + (k & 3) * 2), idesc_qk, k > 0);
        tc::umma_commit(&empty_k[sk_n]);
        tc::umma_commit(&s_full[sb]);
        if (++sk_n == P5_NSK) { sk_n = 0; phk ^= 1; }
        return true;
      };
      if (ok && n_tiles > 0) ok = issue_qk(0);
      for (int it = 0; it < n_tiles && ok; ++it) {
        if (it + 1 < n_tiles) { ok = issue_qk(it + 1); if (!ok) break; }      // S(it+1) overlaps the softmax of tile it
        const int pb = it & 1;
        if (!tc::mbar_wait(&p_full[pb], (it >> 1) & 1, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(&full_v[sv_n], phv, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        const uint64_t dps = dp + (uint64_t)(pb * (P5_KV_TILE >> 4)), dvs = dv + (uint64_t)(sv_n * (P5_KV_TILE >> 4));
#pragma unroll
        for (int b = 0; b < P5_BN / KV_BLOCK; ++b)                           // 16 keys per MMA = one KV block: P advances 32 bytes, V 4096
          tc::umma_bf16(tmem + 2 * P5_BN, dps + (uint64_t)(b * 2), dvs + (uint64_t)(b * 256), idesc_pv, (it > 0 || b > 0) ? 1u : 0u);
        tc::umma_commit(&empty_v[sv_n]);
        tc::umma_commit(&p_free[pb]);                                        // every MMA up to P V of tile it is done
        if (++sv_n == P5_NSV) { sv_n = 0; phv ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (2..9)
    // Warps w and w + 4 serve the same tensor-memory lane quadrant (32 query rows): thread (row r, half hf) owns
    // keys [32 hf, 32 hf + 32) of every tile and output dims [64 hf, 64 hf + 64).
    const int quad = warp & 3, hf = (warp - 2) >> 2, r = quad * 32 + lane;
    const bool row_valid = r < n_rows;
    const int t_row = row_valid ? a.row_t[row0 + r] : -1;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    const uint32_t t_o = t_lane + 2 * P5_BN + hf * 64;                 // my 64 output dims of my row
    float* xmax = reinterpret_cast<float*>(bars + 32);                 // [2 S buffers][2 halves][128 rows], then [2][128] sums
    float* xsum = xmax + 2 * 2 * 128;
    uint64_t* pair_bar = &pair_bars[quad];
    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int sb = it & 1, pb = it & 1;
      const bool shared_tile = it < n_sh;
      const int key0 = (shared_tile ? it * P5_BN : (it - n_sh) * P5_BN) + hf * 32;   // first key of my half
      const int lim = shared_tile ? sh_end - 1 : t_row;                       // last visible key of this row in the segment
      if (!tc::mbar_wait_warp(&s_full[sb], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tmem_fence_after();
      uint32_t v[32];
      tc::tmem_ld32(t_lane + sb * P5_BN + hf * 32, v);
      tc::tmem_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&s_free[sb]);                            // S is in registers: the buffer may be refilled
      const bool whole = key0 + 31 <= lim;
      float t4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) t4[j] = -INFINITY;
      if (whole) {
#pragma unroll
        for (int j = 0; j < 32; ++j) t4[j & 3] = fmaxf(t4[j & 3], __uint_as_float(v[j]));
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) if (key0 + j <= lim) t4[j & 3] = fmaxf(t4[j & 3], __uint_as_float(v[j]));
      }
      float mx = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3])) * a.scale_log2;   // scale_log2 > 0
      xmax[(sb * 2 + hf) * 128 + r] = mx;
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(pair_bar);                               // release: my warp's maxima are written
      if (!tc::mbar_wait_warp(pair_bar, it & 1, abort_flag)) { ok = false; break; }
      mx = fmaxf(mx, xmax[(sb * 2 + (hf ^ 1)) * 128 + r]);
      // The tile's P buffer is free once the P V of tile it - 2 has run.
      if (!tc::mbar_wait_warp(&p_free[pb], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
      // Move the row's reference maximum only when this tile's maximum exceeds it by more than 2^P5_LAZY (the two
      // threads of a row see the same numbers and decide alike; so do the two warps of these 32 rows).
      const bool move = mx > m_ref + P5_LAZY || (m_ref == -INFINITY && mx > -INFINITY);
      if (__any_sync(0xffffffffu, move)) {
        const float factor = move ? ((m_ref == -INFINITY) ? 0.f : fa::ex2(m_ref - mx)) : 1.0f;
        if (it > 0) {
          // every P V issued so far has to be in O before the row is rescaled (the P V of this tile waits for our
          // P): the P V of tile it - 1 frees the other P buffer when it is done.  (This warp waited for that
          // buffer's previous phase one tile ago, so the parity cannot be mistaken for an older phase.)
          if (!tc::mbar_wait_warp(&p_free[pb ^ 1], ((it - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
          tc::tmem_fence_after();
#pragma unroll
          for (int c = 0; c < 64; c += 32) {
            uint32_t w[32];
            tc::tmem_ld32(t_o + c, w);
#pragma unroll
            for (int j = 0; j < 32; ++j) w[j] = __float_as_uint(__uint_as_float(w[j]) * factor);
            tc::tmem_st32(t_o + c, w);
          }
          tc::tmem_fence_before();
        }
        if (move) { l *= factor; m_ref = mx; }
      }
      // P = 2^(s - m_ref) as bf16 into the swizzled K-major tile: one 128-byte row of 64 keys per query row; my 32
      // keys are its 16-byte chunks 4 hf .. 4 hf + 3.  (A row that has seen no key yet has m_ref = -inf and only
      // masked keys: the selects below drop whatever the exponential makes of that.)
      float ps = 0.f;
      const uint32_t base = sP + pb * P5_KV_TILE + r * 128;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t pk[4];
#pragma unroll
        for (int j = 0; j < 8; j += 2) {
          const int k = 8 * q + j;
          float p0 = fa::ex2(fmaf(__uint_as_float(v[k]), a.scale_log2, -m_ref));
          float p1 = fa::ex2(fmaf(__uint_as_float(v[k + 1]), a.scale_log2, -m_ref));
          if (!whole) { p0 = (key0 + k <= lim) ? p0 : 0.f; p1 = (key0 + k + 1 <= lim) ? p1 : 0.f; }
          ps += p0 + p1;
          pk[j >> 1] = fa::pack_bf16(p0, p1);
        }
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(base + (((hf * 4 + q) ^ (r & 7)) << 4)), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
      }
      l += ps;
      t5::fence_async_smem();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&p_full[pb]);
    }
    // the row's sum: both halves used the same reference maxima, so the partial sums just add
    xsum[hf * 128 + r] = l;
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(pair_bar);
    if (ok && tc::mbar_wait_warp(pair_bar, n_tiles & 1, abort_flag)) l = xsum[r] + xsum[128 + r];
    else ok = false;
    if (n_tiles == 0 && row_valid) {                                          // a row tile without any key: zeros
      bf16* dst = a.out + (int64_t)(row0 + r) * a.out_cols + head * T5_DH + hf * 64;
#pragma unroll
      for (int i = 0; i < 64; i += 8) *reinterpret_cast<uint4*>(dst + i) = make_uint4(0u, 0u, 0u, 0u);
    }
    if (ok && n_tiles > 0 && tc::mbar_wait_warp(&p_free[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, abort_flag)) {   // the last P V is done
      tc::tmem_fence_after();
      const float inv = (l > 0.f) ? 1.0f / l : 0.f;
      bf16* dst = a.out + (int64_t)(row0 + r) * a.out_cols + head * T5_DH + hf * 64;
#pragma unroll
      for (int c = 0; c < 64; c += 32) {
        uint32_t w[32];
        tc::tmem_ld32(t_o + c, w);                                            // warp-wide: every lane loads, valid rows store
        if (row_valid) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 w4;
            w4.x = fa::pack_bf16(__uint_as_float(w[i]) * inv, __uint_as_float(w[i + 1]) * inv);
            w4.y = fa::pack_bf16(__uint_as_float(w[i + 2]) * inv, __uint_as_float(w[i + 3]) * inv);
            w4.z = fa::pack_bf16(__uint_as_float(w[i + 4]) * inv, __uint_as_float(w[i + 5]) * inv);
            w4.w = fa::pack_bf16(__uint_as_float(w[i + 6]) * inv, __uint_as_float(w[i + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + c + i) = w4;
          }
        }
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
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256u) : "memory");
  }
}

}  // namespace rpo
