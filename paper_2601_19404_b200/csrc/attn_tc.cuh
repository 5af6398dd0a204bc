// bf16 attention on tensor cores (mma.sync m16n8k16, float32 softmax and accumulation) over the
// paged KV cache, flash style.  A dedicated producer warp streams 64-key K and V tiles into two
// shared-memory rings with bulk async copies (cp.async.bulk: ONE contiguous copy per 16-token KV
// block, found through the block table; the pool already stores a block in the swizzled layout
// ldmatrix wants, see KVPool), guarded by full/empty mbarriers; the consumer warps never issue a
// global load in the tile loop and do no address arithmetic for K/V.  Keys past
// the end of a segment are masked, not zero-filled: the pool is zeroed at creation, so whatever a
// box brings along is finite.  Every mbarrier wait is bounded (status bit 0 on expiry).
//
// Key space of a query row = [shared segment: the group's prefix blocks, all visible]
//                         ++ [private segment: the sequence's own blocks, keys 0..t visible].
// Three uses:
//   ROWS   (prefill, teacher-forced log-probs): a tile holds 64 consecutive rows of one sequence
//          for one query head; output is the normalised attention, written as bf16.
//   SHARED (decode): a work item holds the G * (Hq/Hkv) query rows of one prompt group that share a
//          KV head and one split of the group's prefix; the prefix K/V of a group is therefore read
//          once per group, not once per sample.  After its prefix tiles the item walks its share
//          of the *suffix* tiles of the group's sequences (dealt round-robin over the splits): a
//          suffix tile belongs to one sequence, only that sequence's rows see its keys (causally),
//          and only the warps holding those rows do the math.  Output: (m, l, unnormalised O)
//          partials per split, merged by attn_decode_merge_kernel.
#pragma once
#include "gemm_tc.cuh"
#include "kernels.cuh"

namespace rpo {

constexpr int FA_BM = 64, FA_BN = 64, FA_THREADS = 128;
enum FlashMode { FA_ROWS = 0, FA_SHARED = 1 };

struct FlashArgs {
  const bf16* qkv; int qkv_cols;
  bf16* out; int out_cols;
  float* part_ml; float* part_o; int n_splits; int split_chunk;   // SHARED: one partial slot per split
  const int32_t* row_seq; const int32_t* row_t; const SeqDesc* seqs; const int32_t* block_table;
  KVPool<bf16> pool; int layer, hq, hkv; float scale_log2;
  const int2* tiles;      // ROWS: (first row, number of rows)
  int G;                  // SHARED: samples per group
  const int32_t* pfx_tbl; int pfx_stride;   // SHARED: prefix block ids of the call's groups, dense [group][pfx_stride]
  int skip_prefix;        // SHARED: the work items carry suffix tiles only (the prefix is another kernel's: attn_dec5.cuh)
  int n_slots, slot_base; // SHARED: partial slots per (row, head); split s writes slot slot_base + s
  int* status;
};

namespace fa {
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void st_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {          // 2^x, one MUFU (ex2.approx: rel. error 2^-22; -inf -> 0)
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t*)&h;
}
// Thread-block cluster: barrier over all threads of all CTAs, and loads from a peer CTA's shared memory.
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void ld_cluster_f32x2(uint32_t addr, float& x, float& y) {
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(x), "=f"(y) : "r"(addr) : "memory");
}
template <int N> __device__ __forceinline__ void ld_cluster_f32(uint32_t addr, float* v);
template <> __device__ __forceinline__ void ld_cluster_f32<4>(uint32_t addr, float* v) {
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]) : "r"(addr) : "memory");
}
template <> __device__ __forceinline__ void ld_cluster_f32<2>(uint32_t addr, float* v) {
  asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(v[0]), "=f"(v[1]) : "r"(addr) : "memory");
}
}  // namespace fa

// Tile shape per mode: 64-key tiles, four consumer warps of 16 query rows each (+ the producer warp),
// Q fragments kept in registers, two CTAs per SM.  Decode (SHARED) looks one K tile further ahead
// than prefill.  KS > 1 (several warp sets sharing the keys of a tile, merged through shared memory
// at the end) is kept as an option; it did not pay at the measured sizes.
template <int MODE> struct FaCfg {
  static constexpr int BN = (MODE == FA_SHARED) ? 64 : 64;     // keys per tile
  static constexpr int NSK = (MODE == FA_SHARED) ? 3 : 2;      // K ring depth: K tiles are fetched NSK-1 tiles ahead,
  static constexpr int NSV = 2;                                //   V tiles (needed half a tile later) NSV-1 ahead
  static constexpr int MIN_CTAS = 2;
  static constexpr int KS = (MODE == FA_SHARED) ? 1 : 1;       // warps sharing the keys of a tile
  static constexpr int THREADS = FA_THREADS * KS;
  static constexpr bool Q_IN_REGS = true;
  template <int DH> static constexpr int smem_bytes() { return (FA_BM + (NSK + NSV) * BN) * DH * 2 + 1024 /*align*/ + 128 /*barriers*/; }
};

// CLM (SHARED only): the CTAs of the splits of one work item form a thread-block cluster
// (cluster rank = split) and merge their partials through distributed shared memory instead of
// global memory and a second kernel; a.n_splits is then the cluster size (1, 2, 4 or 8).
template <int DH, int MODE, bool CLM = false>
__global__ void __launch_bounds__(FaCfg<MODE>::THREADS + 32, FaCfg<MODE>::MIN_CTAS)
flash_attn_kernel(FlashArgs a) {
  pdl_prologue();
  constexpr bool CL = CLM && MODE == FA_SHARED;
  static_assert(!(CLM && FaCfg<MODE>::KS != 1), "the in-cluster merge expects one warp set");
  constexpr int XO_STRIDE = DH + 8;          // floats per row of the partial O kept in shared memory (bank-conflict-free)
  constexpr int NSK = FaCfg<MODE>::NSK, NSV = FaCfg<MODE>::NSV;
  constexpr int BN = FaCfg<MODE>::BN;
  constexpr int KS = FaCfg<MODE>::KS, THREADS = FaCfg<MODE>::THREADS, WBN = BN / KS;   // WBN: keys of a tile per warp
  constexpr bool Q_IN_REGS = FaCfg<MODE>::Q_IN_REGS;
  constexpr int CH = DH / 8;                 // 16-byte chunks per row
  constexpr int ROW_BYTES = DH * 2;
  constexpr int TILE_BYTES = BN * ROW_BYTES;
  constexpr int KSTEPS = DH / 16, ONT = DH / 8;
  constexpr int BLK_BYTES = KV_BLOCK * ROW_BYTES;   // one KV block of K (or V) for one head
  constexpr int PER_HALF = DH < 64 ? DH : 64;       // dims per 128-byte (or shorter) row of the block layout
  constexpr int NW = THREADS / 32;           // consumer warps; warp NW is the producer
  extern __shared__ uint8_t fsm_raw[];
  uint8_t* fsm = (uint8_t*)(((uintptr_t)fsm_raw + 1023) & ~(uintptr_t)1023);
  const uint32_t sK = (uint32_t)__cvta_generic_to_shared(fsm);   // NSK buffers (1024-byte aligned: swizzle atoms)
  const uint32_t sV = sK + NSK * TILE_BYTES;                       // NSV buffers
  const uint32_t sQ = sV + NSV * TILE_BYTES;
  uint64_t* bars = (uint64_t*)(fsm + (NSK + NSV) * TILE_BYTES + FA_BM * ROW_BYTES);
  uint64_t *full_k = bars, *empty_k = bars + NSK, *full_v = bars + 2 * NSK, *empty_v = bars + 2 * NSK + NSV;
  __shared__ int s_abort;
  __shared__ int s_qrow[FA_BM];     // qkv row of each tile row (-1: padding)
  __shared__ int s_head[FA_BM];
  __shared__ int s_t[FA_BM];        // private causal limit (-1: nothing visible / inactive)
  __shared__ int s_pt_sum[FA_BM + 1];   // SHARED: suffix tiles of the tile's sequences that fall to this split, prefix-summed
  __shared__ int s_pt_t[FA_BM];         //         their newest suffix index t (-1: finished)
  __shared__ int s_pt_tbl[FA_BM];       //         their private block-table offsets
  constexpr int BLK_CACHE = (MODE == FA_SHARED) ? 512 : 1;
  __shared__ int s_blk[BLK_CACHE];      //         block ids of this split's prefix keys (one fetch, not one per tile)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
  const int mt = warp & 3, kh = warp >> 2;       // 16-row tile of the warp, its share of each tile's keys
  const int rep = a.hq / a.hkv;
  int kvh, n_rows, split = 0, r0 = 0, sq0 = 0, n_sq = 0;
  int sh_begin = 0, sh_end = 0;
  SeqDesc sd;
  // Q tile: rows of DH*2 bytes, 16-byte chunks XOR-swizzled by the row.  K/V tiles: BN/16 blocks
  // back to back, each in the pool's block layout [half][token][chunk ^ (token & 7)].
  auto sw = [&](int row, int chunk) -> uint32_t { return (uint32_t)(row * ROW_BYTES + ((chunk ^ (row & 7)) << 4)); };
  auto swkv = [&](int row, int chunk) -> uint32_t {
    constexpr int CPH = PER_HALF / 8;          // chunks per half row
    return (uint32_t)((row >> 4) * BLK_BYTES + (chunk / CPH) * (KV_BLOCK * PER_HALF * 2) + (row & 15) * (PER_HALF * 2) +
                      (((chunk % CPH) ^ (row & 7)) << 4));
  };
  if (tid == 0) {
    for (int i = 0; i < NSK; ++i) { tc::mbar_init(&full_k[i], 1); tc::mbar_init(&empty_k[i], NW); }
    for (int i = 0; i < NSV; ++i) { tc::mbar_init(&full_v[i], 1); tc::mbar_init(&empty_v[i], NW); }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  constexpr int QTPR = THREADS / FA_BM;          // threads per Q row
  auto load_q = [&](int qrow, int qpar, int qr, int qhead) {   // qr: qkv row (-1: zero padding)
    const bf16* qp = (qr >= 0) ? a.qkv + (int64_t)qr * a.qkv_cols + qhead * DH : nullptr;
#pragma unroll
    for (int j = 0; j < CH / QTPR; ++j) {
      const int ch = QTPR * j + qpar;
      if (qp) fa::cp_async16(sQ + sw(qrow, ch), qp + ch * 8); else fa::st_zero16(sQ + sw(qrow, ch));
    }
  };
  if (MODE == FA_ROWS) {
    const int2 tile = a.tiles[blockIdx.y];        // grid (heads, tiles), tile list ordered heaviest first
    const int head = blockIdx.x;
    kvh = head / rep; n_rows = tile.y;
    sd = a.seqs[a.row_seq[tile.x]];
    if (tid < FA_BM) {
      const bool v = tid < n_rows;
      s_qrow[tid] = v ? tile.x + tid : -1;
      s_head[tid] = head;
      s_t[tid] = v ? a.row_t[tile.x + tid] : -1;
    }
  } else {
    const int rows_per_group = a.G * rep;
    const int tiles_per_group = (rows_per_group + FA_BM - 1) / FA_BM;
    const int item = blockIdx.x / a.n_splits;
    split = blockIdx.x % a.n_splits;
    const int grp = item / tiles_per_group;
    r0 = (item % tiles_per_group) * FA_BM;
    kvh = blockIdx.y;
    n_rows = min(FA_BM, rows_per_group - r0);
    if (tid < THREADS) {   // the Q rows go first: their addresses need nothing from memory
      const int qrow = tid / QTPR, i = r0 + qrow;
      const bool v = qrow < n_rows;
      load_q(qrow, tid % QTPR, v ? grp * a.G + i / rep : -1, kvh * rep + (v ? i % rep : 0));
    }
    // block ids of this split's prefix keys: one fetch up front instead of one per tile, from the
    // call's dense table, so the request does not wait for the sequence descriptor (entries past a
    // short prefix are padding and never used)
    if (!a.skip_prefix) {
      const int n_cache = min(BLK_CACHE, a.split_chunk / KV_BLOCK);
      const int32_t* src = a.pfx_tbl + (int64_t)grp * a.pfx_stride + split * (a.split_chunk / KV_BLOCK);
      for (int e = tid; e < n_cache; e += THREADS + 32) s_blk[e] = src[e];
    }
    sd = a.seqs[grp * a.G];
    if (tid < FA_BM) {
      const bool v = tid < n_rows;
      const int i = r0 + tid;
      s_qrow[tid] = v ? grp * a.G + i / rep : -1;
      s_head[tid] = kvh * rep + (v ? i % rep : 0);
      s_t[tid] = -1;
    }
    // the sequences that own rows of this tile, their suffix lengths and block tables
    sq0 = r0 / rep;
    n_sq = (r0 + n_rows - 1) / rep - sq0 + 1;              // <= FA_BM
    if (tid < n_sq) {                                      // n_sq <= FA_BM <= THREADS
      const int seq = grp * a.G + sq0 + tid;
      const int t = a.row_t[seq];
      s_pt_t[tid] = t;
      s_pt_tbl[tid] = a.seqs[seq].priv_tbl;               // decode passes: row i is sequence i
      // Suffix tile j of the group's sequence i belongs to split (i + j) % n_splits: a sequence's
      // arithmetic does not depend on how far its siblings have got.  Tiles of this split: j0, j0 + n_splits, ..
      const int nt = (t >= 0) ? t / BN + 1 : 0;
      const int j0 = ((split - (sq0 + tid)) % a.n_splits + a.n_splits) % a.n_splits;
      s_pt_sum[tid + 1] = (nt > j0) ? (nt - j0 - 1) / a.n_splits + 1 : 0;      // prefix-summed below
    }
    sh_begin = min(sd.shared_len, split * a.split_chunk);  // a multiple of 16
    sh_end = min(sd.shared_len, sh_begin + a.split_chunk);
    if (a.skip_prefix) { sh_begin = 0; sh_end = 0; }
  }
  __syncthreads();
  if (MODE == FA_SHARED) {
    if (tid == 0) {
      int run = 0;
      s_pt_sum[0] = 0;
      for (int i = 0; i < n_sq; ++i) { run += s_pt_sum[i + 1]; s_pt_sum[i + 1] = run; }
    }
    __syncthreads();
  }

  // ---- key ranges
  int pr_end = 0, n_pr_tiles;
  if (MODE == FA_ROWS) {
    sh_end = (sd.shared_tbl >= 0) ? sd.shared_len : 0;
    int mt = -1;
    for (int i = 0; i < n_rows; ++i) mt = max(mt, s_t[i]);
    pr_end = mt + 1;
    n_pr_tiles = (pr_end + BN - 1) / BN;
  } else {
    n_pr_tiles = s_pt_sum[n_sq];
  }
  const int n_sh_tiles = (sh_end - sh_begin + BN - 1) / BN;
  const int n_tiles = n_sh_tiles + n_pr_tiles;

  // ---- tile bookkeeping shared by the producer and the consumers: segment, first key, key limit
  auto tile_info = [&](int it, int& cur, int& tbl, int& key0, int& limit) {
    if (it < n_sh_tiles) { tbl = sd.shared_tbl; key0 = sh_begin + it * BN; limit = sh_end; }
    else if (MODE == FA_ROWS) { tbl = sd.priv_tbl; key0 = (it - n_sh_tiles) * BN; limit = pr_end; }
    else {
      const int q = it - n_sh_tiles;                                    // q-th suffix tile of this work item
      while (s_pt_sum[cur + 1] <= q) ++cur;                             // its sequence (tiles are met in order)
      const int j0 = ((split - (sq0 + cur)) % a.n_splits + a.n_splits) % a.n_splits;
      tbl = s_pt_tbl[cur]; key0 = (j0 + (q - s_pt_sum[cur]) * a.n_splits) * BN; limit = s_pt_t[cur] + 1;
    }
  };
  volatile int* abort_flag = &s_abort;
  if (MODE == FA_ROWS && tid < THREADS) load_q(tid / QTPR, tid % QTPR, s_qrow[tid / QTPR], s_head[tid / QTPR]);

  if (warp == NW) {
    // ------------------------------------------------------------------ producer warp
    // Lane b looks up the KV block of the tile's b-th group of 16 keys; lane 0 then sends one box
    // per block and half head.  Groups past the end of the segment re-send the last valid block
    // (finite data, masked by the consumers), so a tile always carries TILE_BYTES.
    int cur = 0;
    auto blocks_of = [&](int it) -> int {       // lane b: block id of keys key0 + 16 b ..
      int tbl, key0, limit;
      tile_info(it, cur, tbl, key0, limit);
      const int nb = max(1, min(BN / KV_BLOCK, (limit - key0 + KV_BLOCK - 1) / KV_BLOCK));
      const int u = key0 + min(lane, nb - 1) * KV_BLOCK;
      int blk = 0;
      if (lane < BN / KV_BLOCK) {
        const int cached = (MODE == FA_SHARED && it < n_sh_tiles) ? (u - sh_begin) / KV_BLOCK : BLK_CACHE;
        blk = (cached < BLK_CACHE) ? s_blk[cached] : a.block_table[tbl + u / KV_BLOCK];
        if (blk < 0 || blk >= a.pool.n_blocks) { atomicOr(a.status, STATUS_BAD_BLOCK); blk = 0; }
      }
      return blk;
    };
    auto send = [&](int blk_lane, int kv, uint32_t dst, uint64_t* bar) {   // lane b copies block b of the tile
      if (lane < BN / KV_BLOCK)
        tc::bulk_load(dst + lane * BLK_BYTES, a.pool.block(a.layer, kv, kvh, blk_lane), BLK_BYTES, bar);
    };
    // Order K0 | K1 V0 | K2 V1 | ...: a K tile is requested one tile ahead of the matching V tile.
    bool ok = true;
    int blk_next = (n_tiles > 0) ? blocks_of(0) : 0, blk_prev_v = 0;
    for (int it = -1; it < n_tiles && ok; ++it) {
      const int itk = it + 1;
      int blk_k = blk_next;
      if (itk < n_tiles) {
        const int sk = itk % NSK;
        if (lane == 0) {
          ok = tc::mbar_wait(&empty_k[sk], ((itk / NSK) & 1) ^ 1, abort_flag);
          if (ok) tc::mbar_expect_tx(&full_k[sk], TILE_BYTES);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        send(blk_k, 0, sK + sk * TILE_BYTES, &full_k[sk]);
        if (itk + 1 < n_tiles) blk_next = blocks_of(itk + 1);      // look the next tile's blocks up early
      }
      if (it >= 0) {
        // the V tile of `it` uses the same blocks as its K tile: keep them from the previous round
        const int sv = it % NSV;
        if (lane == 0) {
          ok = tc::mbar_wait(&empty_v[sv], ((it / NSV) & 1) ^ 1, abort_flag);
          if (ok) tc::mbar_expect_tx(&full_v[sv], TILE_BYTES);
        }
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) break;
        send(blk_prev_v, 1, sV + sv * TILE_BYTES, &full_v[sv]);
      }
      blk_prev_v = blk_k;
    }
    if (!CL) return;                            // the consumers use named barrier 1 from here on
  }

  if (warp < NW) {
  float o[ONT][4];
#pragma unroll
  for (int i = 0; i < ONT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  uint32_t qf[Q_IN_REGS ? KSTEPS : 1][4];
  const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
  int t_lo = s_t[r_lo], t_hi = s_t[r_hi];

  int mm_cur = 0;                              // SHARED: sequence cursor of the math
  asm volatile("cp.async.wait_all;" ::: "memory");                              // this thread's Q chunks
  asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");                    // all of Q (consumers only)
  bool ok = true;
  for (int it = 0; it < n_tiles && ok; ++it) {
    if (!tc::mbar_wait(&full_k[it % NSK], (it / NSK) & 1, abort_flag)) { ok = false; break; }
    if (Q_IN_REGS && it == 0) {
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk)
        fa::ldsm_x4(sQ + sw(mt * 16 + (lane & 15), kk * 2 + (lane >> 4)), qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
    }
    bool warp_has_work = mt * 16 < n_rows;        // warps whose 16 rows are all padding only help with the loads
    int suffix_key0 = 0;
    if (MODE == FA_SHARED && it >= n_sh_tiles) {
      // suffix tile of one sequence: visible to that sequence's rows only, keys 0..t
      const int q = it - n_sh_tiles;
      while (s_pt_sum[mm_cur + 1] <= q) ++mm_cur;
      const int j0 = ((split - (sq0 + mm_cur)) % a.n_splits + a.n_splits) % a.n_splits;
      const int row_first = (sq0 + mm_cur) * rep - r0, row_last = row_first + rep - 1;   // tile-local, may stick out
      const int t_own = s_pt_t[mm_cur];
      suffix_key0 = (j0 + (q - s_pt_sum[mm_cur]) * a.n_splits) * BN;
      t_lo = (r_lo >= row_first && r_lo <= row_last) ? t_own : -1;
      t_hi = (r_hi >= row_first && r_hi <= row_last) ? t_own : -1;
      warp_has_work = warp_has_work && (mt * 16 <= row_last) && (mt * 16 + 15 >= row_first) &&
                      (suffix_key0 + kh * WBN <= t_own);
    }
    uint32_t pf[WBN / 16][4];                     // P as bf16 A-fragments, handed from the softmax to P V
    if (warp_has_work) {
    // ---- S = Q K^T
    float s[WBN / 8][4];
#pragma unroll
    for (int j = 0; j < WBN / 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
    const uint32_t kb = sK + (it % NSK) * TILE_BYTES;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      const int qi = Q_IN_REGS ? kk : 0;
      if (!Q_IN_REGS)
        fa::ldsm_x4(sQ + sw(mt * 16 + (lane & 15), kk * 2 + (lane >> 4)), qf[0][0], qf[0][1], qf[0][2], qf[0][3]);
#pragma unroll
      for (int jp = 0; jp < WBN / 16; ++jp) {
        uint32_t b0, b1, b2, b3;
        fa::ldsm_x4(kb + swkv(kh * WBN + jp * 16 + (lane & 7) + ((lane >> 4) << 3), kk * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
        fa::mma_bf16(s[2 * jp], qf[qi], b0, b1);
        fa::mma_bf16(s[2 * jp + 1], qf[qi], b2, b3);
      }
    }
    // ---- mask + online softmax (base-2 exponent domain)
    const bool shared_tile = it < n_sh_tiles;
    const int key0 = shared_tile ? sh_begin + it * BN : (MODE == FA_ROWS ? (it - n_sh_tiles) * BN : suffix_key0);
    float mx_lo = -INFINITY, mx_hi = -INFINITY;
    if (shared_tile && key0 + BN <= sh_end) {          // tile fully inside the visible prefix: no masking
#pragma unroll
      for (int j = 0; j < WBN / 8; ++j) {
#pragma unroll
        for (int c = 0; c < 4; ++c) s[j][c] *= a.scale_log2;
        mx_lo = fmaxf(mx_lo, fmaxf(s[j][0], s[j][1])); mx_hi = fmaxf(mx_hi, fmaxf(s[j][2], s[j][3]));
      }
    } else {
#pragma unroll
      for (int j = 0; j < WBN / 8; ++j) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int key = key0 + kh * WBN + j * 8 + tq * 2 + (c & 1);
          const bool vis = shared_tile ? (key < sh_end) : (key <= ((c & 2) ? t_hi : t_lo));
          const float v = vis ? s[j][c] * a.scale_log2 : -INFINITY;
          s[j][c] = v;
          if (c & 2) mx_hi = fmaxf(mx_hi, v); else mx_lo = fmaxf(mx_lo, v);
        }
      }
    }
    mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1)); mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
    mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1)); mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
    const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
    const float mu_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, mu_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
    const float c_lo = fa::ex2(m_lo - mu_lo), c_hi = fa::ex2(m_hi - mu_hi);
    m_lo = mn_lo; m_hi = mn_hi;
    float ps_lo = 0.f, ps_hi = 0.f;
#pragma unroll
    for (int j = 0; j < WBN / 8; ++j) {
      const float p0 = fa::ex2(s[j][0] - mu_lo), p1 = fa::ex2(s[j][1] - mu_lo);
      const float p2 = fa::ex2(s[j][2] - mu_hi), p3 = fa::ex2(s[j][3] - mu_hi);
      ps_lo += p0 + p1; ps_hi += p2 + p3;
      pf[j >> 1][(j & 1) * 2] = fa::pack_bf16(p0, p1);
      pf[j >> 1][(j & 1) * 2 + 1] = fa::pack_bf16(p2, p3);
    }
    l_lo = l_lo * c_lo + ps_lo; l_hi = l_hi * c_hi + ps_hi;
    if (!__all_sync(0xffffffffu, c_lo == 1.0f && c_hi == 1.0f)) {   // running maxima unchanged: nothing to rescale
#pragma unroll
      for (int i = 0; i < ONT; ++i) { o[i][0] *= c_lo; o[i][1] *= c_lo; o[i][2] *= c_hi; o[i][3] *= c_hi; }
    }
    }
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(&empty_k[it % NSK]);        // this warp is done with K(it)
    if (!tc::mbar_wait(&full_v[it % NSV], (it / NSV) & 1, abort_flag)) { ok = false; break; }
    if (warp_has_work) {
    // ---- O += P V
    const uint32_t vb = sV + (it % NSV) * TILE_BYTES;
#pragma unroll
    for (int kk = 0; kk < WBN / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < ONT / 2; ++np) {
        uint32_t b0, b1, b2, b3;
        fa::ldsm_x4_t(vb + swkv(kh * WBN + kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3), np * 2 + (lane >> 4)), b0, b1, b2, b3);
        fa::mma_bf16(o[2 * np], pf[kk], b0, b1);
        fa::mma_bf16(o[2 * np + 1], pf[kk], b2, b3);
      }
    }
    }
    __syncwarp();
    if (lane == 0) tc::mbar_arrive(&empty_v[it % NSV]);        // ... and with V(it)
  }
  if (!ok && lane == 0) atomicOr(a.status, STATUS_TIMEOUT);
  if (KS == 2) {
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");   // every consumer warp is done with the rings
    // The warps of the second key half hand their state to the warp holding the same rows in the
    // first half, thread to thread ([value][thread] layout: no bank conflicts), through the K/V ring
    // (free after the loop's last barrier).  m is uniform over a quad, l is still a per-lane partial.
    float* xch = reinterpret_cast<float*>(fsm);
    const int xt = mt * 32 + lane;
    if (kh == 1) {
#pragma unroll
      for (int i = 0; i < ONT; ++i) {
#pragma unroll
        for (int c = 0; c < 4; ++c) xch[(i * 4 + c) * FA_THREADS + xt] = o[i][c];
      }
      xch[(ONT * 4 + 0) * FA_THREADS + xt] = m_lo; xch[(ONT * 4 + 1) * FA_THREADS + xt] = m_hi;
      xch[(ONT * 4 + 2) * FA_THREADS + xt] = l_lo; xch[(ONT * 4 + 3) * FA_THREADS + xt] = l_hi;
    }
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
    if (kh == 1) return;
    const float mb_lo = xch[(ONT * 4 + 0) * FA_THREADS + xt], mb_hi = xch[(ONT * 4 + 1) * FA_THREADS + xt];
    const float mn_lo = fmaxf(m_lo, mb_lo), mn_hi = fmaxf(m_hi, mb_hi);
    const float mu_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, mu_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
    const float ca_lo = fa::ex2(m_lo - mu_lo), cb_lo = fa::ex2(mb_lo - mu_lo);
    const float ca_hi = fa::ex2(m_hi - mu_hi), cb_hi = fa::ex2(mb_hi - mu_hi);
    l_lo = l_lo * ca_lo + xch[(ONT * 4 + 2) * FA_THREADS + xt] * cb_lo;
    l_hi = l_hi * ca_hi + xch[(ONT * 4 + 3) * FA_THREADS + xt] * cb_hi;
    m_lo = mn_lo; m_hi = mn_hi;
#pragma unroll
    for (int i = 0; i < ONT; ++i) {
      o[i][0] = o[i][0] * ca_lo + xch[(i * 4 + 0) * FA_THREADS + xt] * cb_lo;
      o[i][1] = o[i][1] * ca_lo + xch[(i * 4 + 1) * FA_THREADS + xt] * cb_lo;
      o[i][2] = o[i][2] * ca_hi + xch[(i * 4 + 2) * FA_THREADS + xt] * cb_hi;
      o[i][3] = o[i][3] * ca_hi + xch[(i * 4 + 3) * FA_THREADS + xt] * cb_hi;
    }
  }
  l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1); l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
  l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1); l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);

  // ---- write
  if (CL) {
    // partial (m, l, O) of this split into the K/V ring (every consumer warp is done with it)
    float* xo = reinterpret_cast<float*>(fsm);
    float* xml = xo + FA_BM * XO_STRIDE;
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
    if (ok) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const int r = half ? r_hi : r_lo;
        if (tq == 0) { xml[r * 2] = half ? m_hi : m_lo; xml[r * 2 + 1] = half ? l_hi : l_lo; }
#pragma unroll
        for (int i = 0; i < ONT; ++i)
          *(float2*)(xo + r * XO_STRIDE + i * 8 + tq * 2) = make_float2(o[i][half * 2], o[i][half * 2 + 1]);
      }
    }
  } else {
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int r = half ? r_hi : r_lo;
    const int qr = s_qrow[r];
    if (qr < 0) continue;
    const float l = half ? l_hi : l_lo, m = half ? m_hi : m_lo;
    if (MODE == FA_ROWS) {
      const float inv = (l > 0.f) ? 1.0f / l : 0.f;
      bf16* dst = a.out + (int64_t)qr * a.out_cols + s_head[r] * DH;
#pragma unroll
      for (int i = 0; i < ONT; ++i)
        *(uint32_t*)(dst + i * 8 + tq * 2) = fa::pack_bf16(o[i][half * 2] * inv, o[i][half * 2 + 1] * inv);
    } else {
      const int64_t slot = ((int64_t)qr * a.hq + s_head[r]) * a.n_slots + a.slot_base + split;
      if (tq == 0) { a.part_ml[slot * 2] = m; a.part_ml[slot * 2 + 1] = l; }
      float* dst = a.part_o + slot * DH;
#pragma unroll
      for (int i = 0; i < ONT; ++i) *(float2*)(dst + i * 8 + tq * 2) = make_float2(o[i][half * 2], o[i][half * 2 + 1]);
    }
  }
  }
  }   // consumer warps

  if (CL) {
    // Log-sum-exp merge of the cluster's partials: the CTA of rank k owns rows k, k + n_splits, ..;
    // a warp per row, lane s reads (m, l) of split s, every lane DH/32 output dimensions of each
    // split in fixed order (reproducible).  All threads of all CTAs take part in both barriers.
    constexpr int DPL = DH / 32;
    fa::cluster_sync();
    if (warp < NW) {
      const uint32_t xo_addr = (uint32_t)__cvta_generic_to_shared(fsm), xml_addr = xo_addr + FA_BM * XO_STRIDE * 4;
      for (int r = split + a.n_splits * warp; r < n_rows; r += a.n_splits * NW) {
        float ms = -INFINITY, ls = 0.f;
        if (lane < a.n_splits) fa::ld_cluster_f32x2(fa::map_rank(xml_addr + r * 8, lane), ms, ls);
        if (!(ls > 0.f)) ms = -INFINITY;
        const float m_new = warp_max(ms);
        const float wgt = (ls > 0.f) ? exp2f(ms - m_new) : 0.f;
        const float l_tot = warp_sum(ls * wgt);
        float acc[DPL];
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
        for (int k = 0; k < a.n_splits; ++k) {
          const float c = __shfl_sync(0xffffffffu, wgt, k);
          float v[DPL];
          fa::ld_cluster_f32<DPL>(fa::map_rank(xo_addr + (r * XO_STRIDE + lane * DPL) * 4, k), v);
#pragma unroll
          for (int i = 0; i < DPL; ++i) acc[i] += (c != 0.f) ? c * v[i] : 0.f;
        }
        const float inv = (l_tot > 0.f) ? 1.0f / l_tot : 0.f;
        bf16* dst = a.out + (int64_t)s_qrow[r] * a.out_cols + s_head[r] * DH + lane * DPL;
#pragma unroll
        for (int i = 0; i < DPL; i += 2) *(uint32_t*)(dst + i) = fa::pack_bf16(acc[i] * inv, acc[i + 1] * inv);
      }
    }
    fa::cluster_sync();                       // no CTA leaves while a peer may still read its partial
  }
}

// Decode: log-sum-exp merge of the per-split partials of (sequence, query head), n_slots <= 33, one
// warp each.  Lane s first reads (m, l) of slot s, the warp agrees on the maximum and on each
// slot's weight, then all slots' O rows are accumulated with independent loads in slot order
// (reproducible); lanes own DH/32 dimensions.
template <int DH>
__global__ void __launch_bounds__(128) attn_decode_merge_kernel(bf16* __restrict__ out, const float* __restrict__ part_ml,
                                                                const float* __restrict__ part_o, int n_slots,
                                                                const int32_t* __restrict__ row_t, int rows, int hq) {
  pdl_prologue();
  constexpr int DPL = DH / 32;
  const int w = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (w >= rows * hq) return;
  const int r = w / hq, head = w % hq;
  bf16* o = out + (int64_t)r * hq * DH + head * DH + lane * DPL;
  float acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  float l_tot = 0.f, m_run = -INFINITY;        // warp-uniform
  const int64_t slot0 = ((int64_t)r * hq + head) * n_slots;
  if (n_slots <= 8) {
    // Few splits: the (m, l) pairs and every split's partial output are requested together (one
    // round trip to L2 instead of two); the arithmetic and its order are those of the loop below.
    float ms = -INFINITY, ls = 0.f;
    if (lane < n_slots) { const float2 ml = *reinterpret_cast<const float2*>(part_ml + (slot0 + lane) * 2); ms = ml.x; ls = ml.y; }
    float v[8][DPL];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float* po = part_o + (slot0 + min(k, n_slots - 1)) * DH + lane * DPL;
#pragma unroll
      for (int i = 0; i < DPL; ++i) v[k][i] = po[i];
    }
    if (!(ls > 0.f)) ms = -INFINITY;
    const float m_new = warp_max(ms);
    const float wgt = (ls > 0.f) ? exp2f(ms - m_new) : 0.f;
    l_tot = warp_sum(ls * wgt);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const float c = __shfl_sync(0xffffffffu, wgt, k);
      if (k < n_slots) {
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[i] += (c != 0.f) ? c * v[k][i] : 0.f;
      }
    }
  } else {   // rows of finished sequences are merged like any other: nothing downstream reads them
    for (int s0 = 0; s0 < n_slots; s0 += 32) {         // one pass for n_slots <= 32, a second for the 33rd
      const int s = s0 + lane;
      float ms = -INFINITY, ls = 0.f;
      if (s < n_slots) { const float2 ml = *reinterpret_cast<const float2*>(part_ml + (slot0 + s) * 2); ms = ml.x; ls = ml.y; }
      if (!(ls > 0.f)) ms = -INFINITY;
      // running maximum over passes: rescale what has been accumulated so far
      const float m_new = fmaxf(m_run, warp_max(ms));
      const float rescale = (m_run == -INFINITY) ? 0.f : exp2f(m_run - m_new);
      const float wgt = (ls > 0.f) ? exp2f(ms - m_new) : 0.f;
      l_tot = l_tot * rescale + warp_sum(ls * wgt);
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[i] *= rescale;
      const int n_here = min(32, n_slots - s0);
#pragma unroll 4
      for (int k = 0; k < n_here; ++k) {
        const float c = __shfl_sync(0xffffffffu, wgt, k);
        const float* po = part_o + (slot0 + s0 + k) * DH + lane * DPL;
#pragma unroll
        for (int i = 0; i < DPL; ++i) { const float v = po[i]; acc[i] += (c != 0.f) ? c * v : 0.f; }
      }
      m_run = m_new;
    }
  }
  const float inv = (l_tot > 0.f) ? 1.0f / l_tot : 0.f;
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[i] = __float2bfloat16_rn(acc[i] * inv);
}

}  // namespace rpo
