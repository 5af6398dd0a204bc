// Decode attention on the 5th-generation tensor cores (head_dim 128).
//
// All G samples of a prompt group continue the same cached prefix (Eq. 3), so their G * (Hq/Hkv) <= 64
// query rows of one KV head form ONE query tile that meets the group's prefix K/V exactly once.  A
// work item = (group, KV head, split) walks 64-key tiles:
//
//   * its split of the group's prefix keys, every key visible to every row, then
//   * its share of the sequences' own suffix tiles (tile j of sequence i belongs to split (i + j) mod
//     n_splits, so a sequence's arithmetic never depends on its siblings): such a tile is visible to
//     the Hq/Hkv rows of its sequence only, causally; the other rows contribute zeros for it,
//
// with, per tile,
//
//   S = Q K^T      tcgen05.mma (M = 128, N = 64 keys), K tile = four KV blocks bulk-copied from the pool,
//                  whose block layout is the swizzled K-major operand; accumulator in tensor memory, two buffers
//   softmax        eight warps, FOUR threads per query row: the tile's 64 rows are stored twice (rows r and
//                  64 + r of Q and of P), so that all four tensor-memory lane quadrants hold every row and a
//                  thread takes 16 of the 64 keys; online max / sum in the exp2 domain, P to shared memory as bf16
//   O += P V       tcgen05.mma accumulating in tensor memory over all tiles, V blocks as stored = MN-major
//                  operand.  P is taken relative to a reference maximum m_ref per row that is only moved when
//                  the running maximum has grown past it by more than 2^8: then, and only then, the softmax
//                  warps wait for the MMAs issued so far, rescale the row's O in tensor memory and its sum, and
//                  go on.  Otherwise the softmax of a tile waits for nothing but its S, so the chain of
//                  warp-to-warp signals of one tile (each a few hundred nanoseconds) overlaps the next tile's.
//
// and leaves (m, l, unnormalised O) of its split in the partial slots that attn_decode_merge_kernel
// combines.  The M = 128 instruction computes every row twice; the tensor pipe is not what bounds
// this kernel (32 KB of K/V per tile against one MMA pair): the duplication buys twice the softmax
// threads.  What bounds it is the K/V stream: a V stage is free again only after its P V has run, so
// the look-ahead is the ring depth.  With 128-key tiles and two stages (all that fits beside Q and P)
// the loads of a tile had one tile's time to arrive; 64-key tiles leave room for four K and five V
// stages (up to 144 KB of K/V in flight) and for two P buffers.
//
// Warp roles: 0 = producer (K/V bulk copies), 1 = MMA issuer and tensor-memory owner, 2..9 = softmax.
// All mbarrier waits are bounded; on expiry the CTA raises STATUS_TIMEOUT and leaves.
#pragma once
#include "attn_tc5.cuh"

namespace rpo {

constexpr int D5_ROWS = 64;                                   // query rows a work item may hold
constexpr int D5_BN = 64;                                     // keys per tile
constexpr int D5_NSK = 4, D5_NSV = 5;                         // ring depths
constexpr int D5_KV_TILE = D5_BN * T5_DH * 2;                 // 16 KB: one K or V tile, also the P tile (128 rows x 64 keys)
constexpr int D5_Q_TILE = 128 * T5_DH * 2;                    // 32 KB
constexpr int D5_SMEM = D5_Q_TILE + (2 + D5_NSK + D5_NSV) * D5_KV_TILE + 1024 + 256 + 3072;   // tiles, alignment, barriers, row exchange
constexpr float D5_LAZY = 8.0f;                               // log2 of the largest P entry tolerated before m_ref moves

struct Decode5Args {
  const bf16* qkv; int qkv_cols;                              // q rows of the decode batch: [seq][head][dim]
  float* part_ml; float* part_o; int n_slots;                 // partial slots per (row, head); split s uses slot s
  const int32_t* pfx_tbl; int pfx_stride;                     // prefix block ids of the call's groups, dense [group][pfx_stride]
  const SeqDesc* seqs;                                        // row i of the pass is sequence i
  const int32_t* row_t;                                       // newest suffix index of each sequence (-1: finished)
  const int32_t* block_table;
  KVPool<bf16> pool; int layer, hq, hkv, G; float scale_log2;
  int n_splits, split_chunk;                                  // keys per prefix split (a multiple of 64)
  int* status;
};

__global__ void __launch_bounds__(320, 1) flash_decode_tc5_kernel(Decode5Args a) {
  pdl_prologue();
  extern __shared__ uint8_t d5_raw[];
  uint8_t* sm = (uint8_t*)(((uintptr_t)d5_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = tc::smem_u32(sm);
  const uint32_t sP = sQ + D5_Q_TILE;
  const uint32_t sK = sP + 2 * D5_KV_TILE;                      // two P buffers
  const uint32_t sV = sK + D5_NSK * D5_KV_TILE;
  uint64_t* bars = (uint64_t*)(sm + D5_Q_TILE + (2 + D5_NSK + D5_NSV) * D5_KV_TILE);
  uint64_t *full_k = bars, *empty_k = bars + 4, *full_v = bars + 8, *empty_v = bars + 13;
  uint64_t *s_full = bars + 18, *s_free = bars + 20;            // per S buffer
  uint64_t *p_full = bars + 22, *p_free = bars + 24;            // per P buffer
  uint64_t *q_full = bars + 27, *row_bars = bars + 28;
  uint32_t* tmem_slot = (uint32_t*)(bars + 30);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  __shared__ int s_sum[D5_ROWS + 1];      // suffix tiles of the group's sequences that fall to this split, prefix-summed
  __shared__ int s_t[D5_ROWS];            // their newest suffix index t (-1: finished)
  __shared__ int s_tbl[D5_ROWS];          // their private block-table offsets

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rep = a.hq / a.hkv;
  const int split = blockIdx.x % a.n_splits, grp = blockIdx.x / a.n_splits, kvh = blockIdx.y;
  const int n_rows = a.G * rep;                                 // <= D5_ROWS (checked by the host)
  const int prefix_len = a.seqs[grp * a.G].shared_len;
  const int sh_begin = min(prefix_len, split * a.split_chunk), sh_end = min(prefix_len, sh_begin + a.split_chunk);
  const int n_pfx = (sh_end - sh_begin + D5_BN - 1) / D5_BN;

  if (threadIdx.x == 0) {
    for (int i = 0; i < D5_NSK; ++i) { tc::mbar_init(&full_k[i], 1); tc::mbar_init(&empty_k[i], 1); }
    for (int i = 0; i < D5_NSV; ++i) { tc::mbar_init(&full_v[i], 1); tc::mbar_init(&empty_v[i], 1); }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(&s_full[i], 1); tc::mbar_init(&s_free[i], 8);
      tc::mbar_init(&p_full[i], 8); tc::mbar_init(&p_free[i], 1);
    }
    tc::mbar_init(q_full, 8);
    for (int i = 0; i < 2; ++i) tc::mbar_init(&row_bars[i], 4);       // one per 32 rows: the four softmax warps that hold them
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < a.G) {
    const int seq = grp * a.G + threadIdx.x;
    const int t = a.row_t[seq];
    s_t[threadIdx.x] = t;
    s_tbl[threadIdx.x] = a.seqs[seq].priv_tbl;
    const int nt = (t >= 0) ? t / D5_BN + 1 : 0;
    const int j0 = ((split - (int)threadIdx.x) % a.n_splits + a.n_splits) % a.n_splits;
    s_sum[threadIdx.x + 1] = (nt > j0) ? (nt - j0 - 1) / a.n_splits + 1 : 0;      // prefix-summed below
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(tmem_slot)), "r"(256u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc::tmem_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    int run = 0;
    s_sum[0] = 0;
    for (int i = 0; i < a.G; ++i) { run += s_sum[i + 1]; s_sum[i + 1] = run; }
  }
  __syncthreads();
  tc::tmem_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_tiles = n_pfx + s_sum[a.G];

  // Tile it: prefix tiles first, then the suffix tiles of sequences 0, 1, .. in order (`cur` is the caller's
  // cursor over the sequences).  seq = -1 for a prefix tile; keys key0 .. key0 + 63 of the segment, of which
  // those below `limit` exist.
  auto tile_info = [&](int it, int& cur, int& seq, int& key0, int& limit) {
    if (it < n_pfx) { seq = -1; key0 = sh_begin + it * D5_BN; limit = sh_end; return; }
    const int q = it - n_pfx;
    while (s_sum[cur + 1] <= q) ++cur;
    const int j0 = ((split - cur) % a.n_splits + a.n_splits) % a.n_splits;
    seq = cur; key0 = (j0 + (q - s_sum[cur]) * a.n_splits) * D5_BN; limit = s_t[cur] + 1;
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    bool ok = true;
    const int32_t* ptbl = a.pfx_tbl + (int64_t)grp * a.pfx_stride;
    int cur = 0;
    // Lane b < 4 looks up the KV block of keys key0 + 16 b .. of tile `it` (past the end of the segment: the last
    // valid block, finite data that the softmax masks).  The look-up of tile it + 1 is requested before tile it is
    // waited for and sent, so the round trip to the table never sits between two tiles.
    auto lookup = [&](int it) -> int {
      int seq, key0, limit;
      tile_info(it, cur, seq, key0, limit);                     // key0 is a multiple of 64: whole KV blocks
      const int nb = max(1, min(D5_BN / KV_BLOCK, (limit - key0 + KV_BLOCK - 1) / KV_BLOCK));
      if (lane >= D5_BN / KV_BLOCK) return 0;
      const int e = key0 / KV_BLOCK + min(lane, nb - 1);
      return (seq < 0) ? ptbl[e] : a.block_table[s_tbl[seq] + e];
    };
    int blk_next = (n_tiles > 0) ? lookup(0) : 0;
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int sk = it % D5_NSK, sv = it % D5_NSV;
      const uint32_t par_k = ((it / D5_NSK) & 1) ^ 1, par_v = ((it / D5_NSV) & 1) ^ 1;
      int blk = blk_next;
      if (it + 1 < n_tiles) blk_next = lookup(it + 1);
      if (blk < 0 || blk >= a.pool.n_blocks) { atomicOr(a.status, STATUS_BAD_BLOCK); blk = 0; }
      if (lane == 0) { ok = tc::mbar_wait(&empty_k[sk], par_k, abort_flag); if (ok) tc::mbar_expect_tx(&full_k[sk], D5_KV_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      {   // K: block b, half h -> plane h, rows 16 b ..: the K-major swizzled tile
        const int b = lane >> 1, h = lane & 1;
        const int kb = __shfl_sync(0xffffffffu, blk, b & 3);
        if (lane < 8)
          tc::bulk_load(sK + sk * D5_KV_TILE + h * (D5_KV_TILE / 2) + b * 2048, a.pool.block(a.layer, 0, kvh, kb) + h * 1024, 2048, &full_k[sk]);
      }
      if (lane == 0) { ok = tc::mbar_wait(&empty_v[sv], par_v, abort_flag); if (ok) tc::mbar_expect_tx(&full_v[sv], D5_KV_TILE); }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      if (lane < D5_BN / KV_BLOCK)            // V: block b verbatim
        tc::bulk_load(sV + sv * D5_KV_TILE + lane * 4096, a.pool.block(a.layer, 1, kvh, blk), 4096, &full_v[sv]);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(D5_BN >> 3) << 17) | ((uint32_t)(T5_BM >> 4) << 24);
      constexpr uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(T5_DH >> 3) << 17) | ((uint32_t)(T5_BM >> 4) << 24);   // B operand (V) is MN-major, N = 128 dims
      // One thread issues every MMA of the CTA, so its instruction stream is on the critical path of every tile:
      // the operand descriptors are built once; inside the loop a descriptor is a base plus a constant (the
      // address field counts 16-byte units and never carries out of its 14 bits within 227 KB of shared memory).
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
        const uint64_t dks = dk + (uint64_t)(sk_n * (D5_KV_TILE >> 4));
#pragma unroll
        for (int k = 0; k < T5_DH / 16; ++k)                                 // dim half plane (k / 4), 32 bytes per 16 dims
          tc::umma_bf16(tmem + sb * D5_BN, dq + (uint64_t)((k >> 2) * (D5_Q_TILE >> 5) + (k & 3) * 2),
                        dks + (uint64_t)((k >> 2) * (D5_KV_TILE >> 5) + (k & 3) * 2), idesc_qk, k > 0);
        tc::umma_commit(&empty_k[sk_n]);
        tc::umma_commit(&s_full[sb]);
        if (++sk_n == D5_NSK) { sk_n = 0; phk ^= 1; }
        return true;
      };
      if (ok && n_tiles > 0) ok = issue_qk(0);
      for (int it = 0; it < n_tiles && ok; ++it) {
        if (it + 1 < n_tiles) { ok = issue_qk(it + 1); if (!ok) break; }      // S(it+1) overlaps the softmax of tile it
        const int pb = it & 1;
        if (!tc::mbar_wait(&p_full[pb], (it >> 1) & 1, abort_flag)) { ok = false; break; }
        if (!tc::mbar_wait(&full_v[sv_n], phv, abort_flag)) { ok = false; break; }
        tc::tmem_fence_after();
        const uint64_t dps = dp + (uint64_t)(pb * (D5_KV_TILE >> 4)), dvs = dv + (uint64_t)(sv_n * (D5_KV_TILE >> 4));
#pragma unroll
        for (int b = 0; b < D5_BN / KV_BLOCK; ++b)                           // 16 keys per MMA = one KV block: P advances 32 bytes, V 4096
          tc::umma_bf16(tmem + 2 * D5_BN, dps + (uint64_t)(b * 2), dvs + (uint64_t)(b * 256), idesc_pv, (it > 0 || b > 0) ? 1u : 0u);
        tc::umma_commit(&empty_v[sv_n]);
        tc::umma_commit(&p_free[pb]);                                        // every MMA up to P V of tile it is done
        if (++sv_n == D5_NSV) { sv_n = 0; phv ^= 1; }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax warps (2..9)
    // Lane quadrants 0, 1 hold rows 0..63, quadrants 2, 3 their copies.  Thread (row r, quarter kq) owns
    // keys [16 kq, 16 kq + 16) of every tile and output dims [32 kq, 32 kq + 32): kq = 2 * copy + hf.
    const int quad = warp & 3, hf = (warp - 2) >> 2, rh = quad & 1, r = rh * 32 + lane, kq = (quad >> 1) * 2 + hf;
    const bool row_valid = r < n_rows;
    const int my_seq = row_valid ? r / rep : -2;
    const uint32_t t_lane = tmem + ((uint32_t)(quad * 32) << 16);
    float* xmax = reinterpret_cast<float*>(bars + 32);                 // [2 S buffers][4 quarters][64 rows], then [4][64] sums
    uint64_t* row_bar = &row_bars[rh];                                 // bounded rendezvous of the four warps holding these rows
    // Q rows into shared memory, each twice (rows i and 64 + i).  Row i = sample i / rep of the group, query head
    // kvh * rep + i % rep; 16-byte chunk c goes to plane c / 8, chunk (c % 8) ^ (i % 8): the swizzled K-major layout.
    for (int e = threadIdx.x - 64; e < n_rows * 16; e += 256) {
      const int i = e >> 4, c = e & 15;
      const bf16* src = a.qkv + (int64_t)(grp * a.G + i / rep) * a.qkv_cols + (kvh * rep + i % rep) * T5_DH + c * 8;
      const uint32_t dst = sQ + (c >> 3) * (D5_Q_TILE / 2) + i * 128 + (((c & 7) ^ (i & 7)) << 4);
      fa::cp_async16(dst, src);
      fa::cp_async16(dst + D5_ROWS * 128, src);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    t5::fence_async_smem();
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(q_full);

    float m_ref = -INFINITY, l = 0.f;
    bool ok = true;
    int cur = 0;
    const uint32_t t_o = t_lane + 2 * D5_BN + kq * 32;                         // my 32 output dims of my row
    for (int it = 0; it < n_tiles && ok; ++it) {
      const int sb = it & 1, pb = it & 1;
      int seq, key0, limit;
      tile_info(it, cur, seq, key0, limit);
      const bool mine = row_valid && (seq < 0 || seq == my_seq);              // does this row see the tile at all
      key0 += kq * 16;                                                        // first key of my quarter
      const int lim = limit - 1;                                              // last visible key (prefix: all; suffix: keys 0..t)
      if (!tc::mbar_wait_warp(&s_full[sb], (it >> 1) & 1, abort_flag)) { ok = false; break; }
      tc::tmem_fence_after();
      uint32_t v[16];
      const bool whole = key0 + 15 <= lim;
      float mx = -INFINITY;
      // tcgen05.ld is a warp-wide instruction: the warp loads if any of its rows sees the tile
      if (__any_sync(0xffffffffu, mine)) tc::tmem_ld16(t_lane + sb * D5_BN + kq * 16, v);
      tc::tmem_fence_before();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&s_free[sb]);                            // S is in registers: the buffer may be refilled
      if (mine) {
        float t4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) t4[j] = -INFINITY;
        if (whole) {
#pragma unroll
          for (int j = 0; j < 16; ++j) t4[j & 3] = fmaxf(t4[j & 3], __uint_as_float(v[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) if (key0 + j <= lim) t4[j & 3] = fmaxf(t4[j & 3], __uint_as_float(v[j]));
        }
        mx = fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3]));
        mx *= a.scale_log2;                                                   // scale_log2 > 0
      }
      xmax[(sb * 4 + kq) * D5_ROWS + r] = mx;
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(row_bar);                                // release: my warp's maxima are written
      if (!tc::mbar_wait_warp(row_bar, it & 1, abort_flag)) { ok = false; break; }
#pragma unroll
      for (int k = 0; k < 4; ++k) mx = fmaxf(mx, xmax[(sb * 4 + k) * D5_ROWS + r]);
      // The tile's P buffer is free once the P V of tile it - 2 has run.
      if (!tc::mbar_wait_warp(&p_free[pb], ((it >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
      // Move the row's reference maximum only when this tile's maximum exceeds it by more than 2^D5_LAZY
      // (the four threads of a row see the same numbers and decide alike; so do the four warps of these 32 rows).
      const bool move = mx > m_ref + D5_LAZY || (m_ref == -INFINITY && mx > -INFINITY);
      if (__any_sync(0xffffffffu, move)) {
        const float factor = move ? ((m_ref == -INFINITY) ? 0.f : fa::ex2(m_ref - mx)) : 1.0f;
        if (it > 0) {
          // every P V issued so far has to be in O before the row is rescaled (P V of this tile waits for our P):
          // P V of tile it - 1 frees the other P buffer when it is done.  (This warp waited for that buffer's
          // previous phase one tile ago, so the parity cannot be mistaken for an older phase.)
          if (!tc::mbar_wait_warp(&p_free[pb ^ 1], ((it - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
          tc::tmem_fence_after();
          uint32_t w[32];
          tc::tmem_ld32(t_o, w);
#pragma unroll
          for (int j = 0; j < 32; ++j) w[j] = __float_as_uint(__uint_as_float(w[j]) * factor);
          tc::tmem_st32(t_o, w);
          tc::tmem_fence_before();
        }
        if (move) { l *= factor; m_ref = mx; }
      }
      // P = 2^(s - m_ref) as bf16 into the swizzled K-major tile (one 128-byte row of 64 keys per query row; my 16
      // keys are 16-byte chunks 2 kq, 2 kq + 1), rows r and 64 + r of the tile's P buffer
      float ps = 0.f;
      const uint32_t base = sP + pb * D5_KV_TILE + r * 128;
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        uint32_t pk[4] = {0u, 0u, 0u, 0u};
        if (mine) {
#pragma unroll
          for (int j = 0; j < 8; j += 2) {
            const int k = 8 * q + j;
            float p0 = fa::ex2(fmaf(__uint_as_float(v[k]), a.scale_log2, -m_ref));
            float p1 = fa::ex2(fmaf(__uint_as_float(v[k + 1]), a.scale_log2, -m_ref));
            if (!whole) { p0 = (key0 + k <= lim) ? p0 : 0.f; p1 = (key0 + k + 1 <= lim) ? p1 : 0.f; }
            ps += p0 + p1;
            pk[j >> 1] = fa::pack_bf16(p0, p1);
          }
        }
        const uint32_t dst = base + (((kq * 2 + q) ^ (r & 7)) << 4);
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(dst + D5_ROWS * 128), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
      }
      l += ps;
      t5::fence_async_smem();
      __syncwarp();
      if (lane == 0) tc::mbar_arrive(&p_full[pb]);
    }
    float o[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) o[i] = 0.f;
    if (ok && n_tiles > 0) {
      if (tc::mbar_wait_warp(&p_free[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, abort_flag)) {   // the last P V is done
        tc::tmem_fence_after();
        uint32_t w[32];
        tc::tmem_ld32(t_o, w);
#pragma unroll
        for (int j = 0; j < 32; ++j) o[j] = __uint_as_float(w[j]);
      } else {
        ok = false;
      }
    }
    // the row's sum: all quarters used the same reference maxima, so the partial sums just add
    xmax[512 + kq * D5_ROWS + r] = l;
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(row_bar);
    if (ok && tc::mbar_wait_warp(row_bar, n_tiles & 1, abort_flag)) {
      l = 0.f;
#pragma unroll
      for (int k = 0; k < 4; ++k) l += xmax[512 + k * D5_ROWS + r];
    } else {
      ok = false;
    }
    if (row_valid) {
      // partial of this split: (m, l) in the exp2 domain and the unnormalised output row (a row that saw no key: l = 0)
      const int qr = grp * a.G + r / rep, head = kvh * rep + r % rep;
      const int64_t slot = ((int64_t)qr * a.hq + head) * a.n_slots + split;
      const bool any_key = ok && l > 0.f;
      if (kq == 0) { a.part_ml[slot * 2] = any_key ? m_ref : -INFINITY; a.part_ml[slot * 2 + 1] = any_key ? l : 0.f; }
      float* dst = a.part_o + slot * T5_DH + kq * 32;
#pragma unroll
      for (int i = 0; i < 32; i += 4)
        *reinterpret_cast<float4*>(dst + i) = any_key ? make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
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
