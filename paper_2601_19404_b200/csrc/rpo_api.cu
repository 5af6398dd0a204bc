// C ABI of the rollout library: context, weights, paged KV bookkeeping and the orchestration of
// prefill (Eq. 3: prefix computed once per group), suffix decode (G samples per group, Algorithm 1
// rollout loop) and teacher-forced token log-probabilities (Eq. 7).
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include <type_traits>
#include <utility>

#include "attn_tc.cuh"
#include "attn_tc5.cuh"
#include "attn_dec5.cuh"
#include "attn_pre5.cuh"
#include "context.h"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "kernels.cuh"
#include "objective.cuh"
#include "ref_kernels.cuh"
#include "sampler.cuh"

using namespace rpo;

#define CUDA_TRY(expr)                                                              \
  do {                                                                              \
    cudaError_t e_ = (expr);                                                        \
    if (e_ != cudaSuccess) {                                                        \
      fprintf(stderr, "[rpo] CUDA error %s at %s:%d: %s\n", cudaGetErrorName(e_), __FILE__, __LINE__, \
              cudaGetErrorString(e_));                                              \
      return RPO_ERR_CUDA;                                                          \
    }                                                                               \
  } while (0)

#define RPO_TRY(expr)            \
  do {                           \
    int r_ = (expr);             \
    if (r_ != RPO_OK) return r_; \
  } while (0)

// Kernel classes for the optional per-kernel timing (rpo_set_option "profile").
enum KClass { KC_OTHER = 0, KC_GEMM = 1, KC_ATTN = 2, KC_SAMPLER = 3, KC_NORM = 4, KC_ROPE = 5, KC_COUNT = 6 };

struct ProfScope {
  rpo_ctx* c; int prev;
  ProfScope(rpo_ctx* c_, int k) : c(c_), prev(c_->prof_class) { c->prof_class = k; }
  ~ProfScope() { c->prof_class = prev; }
};

static void prof_begin(rpo_ctx* c, const char* label = "gemm_tc_kernel") {
  if (!c->profile) return;
  cudaEvent_t a, b;
  cudaEventCreate(&a); cudaEventCreate(&b);
  cudaEventRecord(a, c->stream);
  c->prof_events.push_back({a, b, c->prof_class + 16 * c->prof_phase, label});
}
static void prof_end(rpo_ctx* c) {
  if (!c->profile) return;
  cudaEventRecord(c->prof_events.back().b, c->stream);
}

// Every kernel of the library starts with pdl_prologue() (or places pdl_wait() itself), so it may be
// launched with programmatic stream serialization: its CTAs are scheduled while the previous
// kernel drains, which hides launch latency between the many short kernels of a decode step.
// By default that attribute is set in the many-row passes and while a decode step is being captured into its graph
// (rpo_ctx::pdl_now), not on the eagerly launched kernels of a decode call: there it was associated with rare hangs
// of 512-sequence rollouts.
template <typename... KArgs, typename... Args>
static cudaError_t launch_kernel(rpo_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cudaLaunchAttribute attr[2];
  int n_attr = 0;
  if (c->pdl_now()) {
    attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
    ++n_attr;
  }
  if (c->launch_cluster_x > 1) {                     // thread-block clusters along x, requested for this launch only
    attr[n_attr].id = cudaLaunchAttributeClusterDimension;
    attr[n_attr].val.clusterDim.x = c->launch_cluster_x; attr[n_attr].val.clusterDim.y = 1; attr[n_attr].val.clusterDim.z = 1;
    ++n_attr;
  }
  c->launch_cluster_x = 0;
  cfg.attrs = attr; cfg.numAttrs = n_attr;
  return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}

#define LAUNCH(ctx, kern, grid, block, smem, ...)                                            \
  do {                                                                                       \
    prof_begin(ctx, #kern);                                                                  \
    const cudaError_t le_ = launch_kernel(ctx, kern, dim3(grid), dim3(block), (size_t)(smem), __VA_ARGS__); \
    prof_end(ctx);                                                                           \
    (ctx)->launches++;                                                                       \
    CUDA_TRY(le_);                                                                           \
    CUDA_TRY(cudaGetLastError());                                                            \
  } while (0)

// What embed_kernel needs to resolve the rows' positions and KV slots (see RowMetaArgs).
static RowMetaArgs row_meta_args(rpo_ctx* c) {
  RowMetaArgs m;
  m.row_seq = c->ws.row_seq; m.row_t = c->ws.row_t; m.seqs = (const SeqDesc*)c->ws.seqs; m.block_table = c->d_block_table;
  m.n_blocks = (int)c->lim.kv_pool_blocks; m.max_pos = c->lim.max_positions; m.row_meta = c->ws.row_meta;
  return m;
}

// A context lives on the device that was current at rpo_create: calls made with another device current
// switch to it (and leave it current, like the CUDA runtime's own stream calls would require).
static int enter(rpo_ctx* c) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return RPO_ERR_CUDA; }
  if (dev != c->device && cudaSetDevice(c->device) != cudaSuccess) { cudaGetLastError(); return RPO_ERR_CUDA; }
  return RPO_OK;
}

static inline int ceil_div(int64_t a, int64_t b) { return (int)((a + b - 1) / b); }
static inline int grid_for(int64_t n, int block, int cap = 148 * 16) {
  return (int)std::max<int64_t>(1, std::min<int64_t>((n + block - 1) / block, cap));
}

extern "C" const char* rpo_strerror(int code) {
  switch (code) {
    case RPO_OK: return "ok";
    case RPO_ERR_INVALID_ARG: return "invalid argument";
    case RPO_ERR_SHAPE: return "unsupported decoder shape";
    case RPO_ERR_KV_POOL: return "KV pool, group slots or sequence slots exhausted";
    case RPO_ERR_CUDA: return "CUDA runtime error";
    case RPO_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
    case RPO_ERR_NOT_INITIALISED: return "weights not initialised or group handle not live";
    case RPO_ERR_LIMIT: return "request exceeds a limit fixed at rpo_create";
    default: return "unknown error code";
  }
}

extern "C" int rpo_shape_preset(const char* name, rpo_shape* out) {
  if (!name || !out) return RPO_ERR_INVALID_ARG;
  rpo_shape s;
  memset(&s, 0, sizeof(s));
  s.rms_eps = 1e-6f;
  s.kv_block_tokens = KV_BLOCK;
  if (!strcmp(name, "tiny")) {
    s.n_layers = 2; s.d_model = 256; s.n_q_heads = 4; s.n_kv_heads = 2; s.head_dim = 64; s.d_ffn = 688;
    s.vocab = 1024; s.rope_base = 10000.f; s.dtype = RPO_DTYPE_FP32;
  } else if (!strcmp(name, "qwen1.5b-class")) {
    s.n_layers = 28; s.d_model = 1536; s.n_q_heads = 12; s.n_kv_heads = 2; s.head_dim = 128; s.d_ffn = 8960;
    s.vocab = 151936; s.rope_base = 1e6f; s.dtype = RPO_DTYPE_BF16;
  } else if (!strcmp(name, "qwen7b-class")) {
    s.n_layers = 28; s.d_model = 3584; s.n_q_heads = 28; s.n_kv_heads = 4; s.head_dim = 128; s.d_ffn = 18944;
    s.vocab = 152064; s.rope_base = 1e6f; s.dtype = RPO_DTYPE_BF16;
  } else {
    return RPO_ERR_INVALID_ARG;
  }
  *out = s;
  return RPO_OK;
}

// ---------------------------------------------------------------------------------------------
// creation
// ---------------------------------------------------------------------------------------------
static int dev_alloc(rpo_ctx* c, void** p, size_t bytes) {
  *p = nullptr;
  if (bytes == 0) bytes = 16;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) {
    fprintf(stderr, "[rpo] cudaMalloc(%zu) failed: %s\n", bytes, cudaGetErrorString(e));
    cudaGetLastError();
    return RPO_ERR_CUDA;
  }
  c->allocations.push_back(*p);
  return RPO_OK;
}

static void add_tensor(rpo_ctx* c, const std::string& name, void* ptr, int rows, int cols, int row_mul, int row_add,
                       bool gain, uint32_t id) {
  TensorInfo t;
  t.ptr = ptr; t.rows = rows; t.cols = cols; t.row_mul = row_mul; t.row_add = row_add; t.gain = gain; t.tensor_id = id;
  c->tensors[name] = t;
}

extern "C" int rpo_destroy(rpo_ctx* ctx) {
  if (!ctx) return RPO_ERR_INVALID_ARG;
  cudaStreamSynchronize(ctx->stream);
  for (auto& g : ctx->step_graphs) cudaGraphExecDestroy(g.exec);
  ctx->step_graphs.clear();
  tc_destroy(ctx);
  for (void* p : ctx->allocations) cudaFree(p);
  for (void* p : ctx->host_stage) if (p) cudaFree(p);
  if (ctx->own_stream) cudaStreamDestroy(ctx->stream);
  delete ctx;
  return RPO_OK;
}

extern "C" int rpo_create(rpo_ctx** out, const rpo_shape* shape, const rpo_limits* lim, void* cuda_stream) {
  if (!out || !shape || !lim) return RPO_ERR_INVALID_ARG;
  *out = nullptr;
  const rpo_shape& s = *shape;
  if (s.n_layers < 0 || s.d_model <= 0 || s.n_q_heads <= 0 || s.n_kv_heads <= 0 || s.d_ffn <= 0 || s.vocab <= 0)
    return RPO_ERR_SHAPE;
  if (s.vocab >= (1 << 18)) return RPO_ERR_SHAPE;   // sampler mass histograms: 14-bit pieces summed in 32 bits
  if ((s.head_dim != 64 && s.head_dim != 128) || s.n_q_heads % s.n_kv_heads || s.kv_block_tokens != KV_BLOCK ||
      s.d_model % 8 || s.d_ffn % 8 || (s.dtype != RPO_DTYPE_FP32 && s.dtype != RPO_DTYPE_BF16) || s.rms_eps < 0)
    return RPO_ERR_SHAPE;
  if (lim->kv_pool_blocks <= 0 || lim->max_groups <= 0 || lim->max_seqs <= 0 || lim->max_chunk_tokens <= 0 ||
      lim->max_positions <= 1)
    return RPO_ERR_INVALID_ARG;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) {
    cudaGetLastError();
    fprintf(stderr, "[rpo] no CUDA device: this library has no CPU path\n");
    return RPO_ERR_CUDA;
  }
  rpo_ctx* c = new (std::nothrow) rpo_ctx();
  if (!c) return RPO_ERR_CUDA;
  c->shape = s; c->lim = *lim; c->stream = (cudaStream_t)cuda_stream;
  if (!c->stream) {
    // The legacy default stream cannot be captured into a CUDA graph.  A blocking stream of our own
    // keeps the implicit ordering with the caller's default-stream work and can be captured.
    if (cudaStreamCreateWithFlags(&c->stream, cudaStreamDefault) != cudaSuccess) { cudaGetLastError(); delete c; return RPO_ERR_CUDA; }
    c->own_stream = true;
  }
  c->bf16 = s.dtype == RPO_DTYPE_BF16; c->esz = c->bf16 ? 2 : 4;
  c->qkv_cols = (s.n_q_heads + 2 * s.n_kv_heads) * s.head_dim;
  int dev = 0;
  cudaGetDevice(&dev);
  c->device = dev;
  cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev);
  const size_t e = c->esz;
  const int d = s.d_model, dh = s.head_dim, F = s.d_ffn, V = s.vocab, qo = s.n_q_heads * dh;
  int rc = RPO_OK;
#define ALLOC(ptr, bytes)                                         \
  if (rc == RPO_OK) rc = dev_alloc(c, (void**)&(ptr), (size_t)(bytes));
  // ---- weights
  ALLOC(c->embed, (size_t)V * d * e);
  ALLOC(c->lm_head, (size_t)V * d * e);
  ALLOC(c->gf, (size_t)d * 4);
  c->layers.resize(s.n_layers);
  for (int l = 0; l < s.n_layers && rc == RPO_OK; ++l) {
    LayerWeights& L = c->layers[l];
    ALLOC(L.wqkv, (size_t)c->qkv_cols * d * e);
    ALLOC(L.wo, (size_t)d * qo * e);
    ALLOC(L.wgu, (size_t)2 * F * d * e);
    ALLOC(L.wd, (size_t)d * F * e);
    ALLOC(L.g1, (size_t)d * 4);
    ALLOC(L.g2, (size_t)d * 4);
    if (rc != RPO_OK) break;
    const std::string p = "layers." + std::to_string(l) + ".";
    const uint32_t id = 16 + 8 * l;
    char* qkv = (char*)L.wqkv;
    add_tensor(c, p + "wq", qkv, qo, d, 1, 0, false, id + 0);
    add_tensor(c, p + "wk", qkv + (size_t)qo * d * e, s.n_kv_heads * dh, d, 1, 0, false, id + 1);
    add_tensor(c, p + "wv", qkv + (size_t)(qo + s.n_kv_heads * dh) * d * e, s.n_kv_heads * dh, d, 1, 0, false, id + 2);
    add_tensor(c, p + "wo", L.wo, d, qo, 1, 0, false, id + 3);
    add_tensor(c, p + "wg", L.wgu, F, d, 2, 0, false, id + 4);
    add_tensor(c, p + "wu", L.wgu, F, d, 2, 1, false, id + 5);
    add_tensor(c, p + "wd", L.wd, d, F, 1, 0, false, id + 6);
    add_tensor(c, p + "g1", L.g1, 1, d, 1, 0, true, 0);
    add_tensor(c, p + "g2", L.g2, 1, d, 1, 0, true, 0);
  }
  if (rc == RPO_OK) {
    add_tensor(c, "embed", c->embed, V, d, 1, 0, false, 0);
    add_tensor(c, "lm_head", c->lm_head, V, d, 1, 0, false, 1);
    add_tensor(c, "gf", c->gf, 1, d, 1, 0, true, 0);
  }
  // ---- paged KV pool [layer][K|V][kv head][block][16][dh]
  c->kv_head_stride = (int64_t)lim->kv_pool_blocks * KV_BLOCK * dh;
  c->kv_kv_stride = c->kv_head_stride * s.n_kv_heads;
  c->kv_layer_stride = c->kv_kv_stride * 2;
  ALLOC(c->kv_base, (size_t)std::max(1, s.n_layers) * c->kv_layer_stride * e);
  c->free_blocks.resize(lim->kv_pool_blocks);
  for (int64_t i = 0; i < lim->kv_pool_blocks; ++i) c->free_blocks[i] = (int32_t)(lim->kv_pool_blocks - 1 - i);
  c->tbl_stride = ceil_div(lim->max_positions, KV_BLOCK);
  ALLOC(c->d_block_table, (size_t)(lim->max_groups + lim->max_seqs) * c->tbl_stride * 4);
  c->groups.resize(lim->max_groups);
  for (int i = lim->max_groups - 1; i >= 0; --i) c->free_slots.push_back(i);
  ALLOC(c->d_x_last, (size_t)lim->max_groups * d * 4);
  ALLOC(c->d_seq_done, (size_t)std::max(lim->max_seqs, 1) * 4);
  for (int i = lim->max_seqs - 1; i >= 0; --i) c->free_state_rows.push_back(i);
  ALLOC(c->d_rope, (size_t)lim->max_positions * (dh / 2) * sizeof(float2));
  ALLOC(c->d_status, 16);
  // ---- workspaces
  Workspace& w = c->ws;
  w.R = std::max(lim->max_chunk_tokens, lim->max_seqs);
  w.HR = std::max(std::max(lim->max_seqs, lim->max_groups), std::min(1024, std::max(lim->max_chunk_tokens, 1)));
  ALLOC(w.x, (size_t)w.R * d * 4);
  ALLOC(w.h, (size_t)w.R * d * e);
  ALLOC(w.qkv, (size_t)w.R * c->qkv_cols * e);
  ALLOC(w.attn, (size_t)w.R * qo * e);
  ALLOC(w.gu, (size_t)w.R * 2 * F * e);
  ALLOC(w.act, (size_t)w.R * F * e);
  ALLOC(w.xh, (size_t)w.HR * d * 4);
  ALLOC(w.hh, (size_t)w.HR * d * e);
  ALLOC(w.logits, (size_t)(w.HR + lim->max_seqs) * V * 4);   // HR work rows, then one parked row per state row (decode in waves)
  ALLOC(w.row_seq, (size_t)w.R * 4);
  ALLOC(w.row_meta, (size_t)w.R * sizeof(int4));
  ALLOC(w.pfx_tbl, (size_t)lim->max_groups * (c->tbl_stride + 512 + 8) * 4);
  ALLOC(w.row_t, (size_t)w.R * 4);
  ALLOC(w.row_tok, (size_t)w.R * 4);
  const int nseq = std::max(lim->max_seqs, lim->max_groups);
  ALLOC(w.seqs, (size_t)nseq * sizeof(SeqDesc));
  w.sampler_w_rows = nseq;
  ALLOC(w.sampler_w, (size_t)nseq * V * 4);
  ALLOC(w.done, (size_t)nseq * 4);
  ALLOC(w.lens, (size_t)nseq * 4);
  ALLOC(w.cur_tok, (size_t)nseq * 4);
  ALLOC(w.logit_row, (size_t)nseq * 4);
  ALLOC(w.t_base, (size_t)nseq * 4);
  ALLOC(w.state_idx, (size_t)nseq * 4);
  ALLOC(w.done_idx, (size_t)nseq * 4);
  ALLOC(w.lse_parts, (size_t)w.HR * 2 * ceil_div(V, 256) * sizeof(float2));
  ALLOC(w.lse_tgt, (size_t)w.HR * 4);
  ALLOC(w.lse_target, (size_t)w.HR * 4);
  ALLOC(w.slot_idx, (size_t)nseq * 4);
  ALLOC(w.step_ctr, 16);
  ALLOC(w.seq_ids, (size_t)nseq * 8);
  ALLOC(w.tiles, ((size_t)w.R / FA_BM + nseq + 2) * sizeof(int2));
  w.attn_part_elems = (size_t)lim->max_seqs * s.n_q_heads * 33 * (dh + 2);
  ALLOC(w.attn_part, w.attn_part_elems * 4);
  w.partial_elems = (size_t)c->sm_count * 128 * 256;
  ALLOC(w.partial, w.partial_elems * 4);
  w.ssq_stride = std::max((d + 31) / 32, 2 * ((d + 255) / 256));
  ALLOC(w.ssq, (size_t)w.R * w.ssq_stride * 4);
  ALLOC(w.ssq_h, (size_t)w.HR * 4);
  ALLOC(w.tile_ctr, (size_t)TC_CTR_CAPACITY * 4);
  if (rc == RPO_OK && cudaMemsetAsync(w.tile_ctr, 0, (size_t)TC_CTR_CAPACITY * 4, c->stream) != cudaSuccess) { cudaGetLastError(); rc = RPO_ERR_CUDA; }
  if (rc == RPO_OK) rc = tc_create(c);
  // The attention kernels mask keys beyond a segment's end instead of zero-filling them, so the
  // pool must never hold NaN/Inf bit patterns: start from zeros.
  if (rc == RPO_OK && cudaMemsetAsync(c->kv_base, 0, (size_t)std::max(1, s.n_layers) * c->kv_layer_stride * e, c->stream) != cudaSuccess) {
    cudaGetLastError();
    rc = RPO_ERR_CUDA;
  }
#undef ALLOC
  if (rc != RPO_OK) { rpo_destroy(c); return rc; }
  cudaMemsetAsync(c->d_status, 0, 16, c->stream);
  rope_table_kernel<<<grid_for((int64_t)lim->max_positions * (dh / 2), 256), 256, 0, c->stream>>>(
      (float2*)c->d_rope, lim->max_positions, dh / 2, (double)s.rope_base);
  c->launches++;
  if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(c->stream) != cudaSuccess) {
    rpo_destroy(c);
    return RPO_ERR_CUDA;
  }
  *out = c;
  return RPO_OK;
}

// ---------------------------------------------------------------------------------------------
// weights
// ---------------------------------------------------------------------------------------------
template <typename T>
static int init_weights_t(rpo_ctx* c, uint64_t seed, float stdv) {
  const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
  for (auto& kv : c->tensors) {
    const TensorInfo& t = kv.second;
    const int64_t n = (int64_t)t.rows * t.cols;
    if (t.gain) {
      LAUNCH(c, fill_kernel<float>, grid_for(n, 256), 256, 0, (float*)t.ptr, n, 1.0f);
    } else {
      LAUNCH(c, init_normal_kernel<T>, grid_for((n + 3) / 4, 256, 148 * 32), 256, 0, (T*)t.ptr, n, t.cols, t.row_mul,
             t.row_add, k0, k1, t.tensor_id, stdv);
    }
  }
  return RPO_OK;
}

extern "C" int rpo_init_weights(rpo_ctx* c, uint64_t seed, float stdv) {
  if (!c || !(stdv >= 0.f)) return RPO_ERR_INVALID_ARG;
  RPO_TRY(enter(c));
  RPO_TRY(c->bf16 ? init_weights_t<bf16>(c, seed, stdv) : init_weights_t<float>(c, seed, stdv));
  c->weights_ready = true;
  return RPO_OK;
}

static int tensor_io(rpo_ctx* c, const char* name, void* host, size_t bytes, bool write) {
  if (!c || !name || !host) return RPO_ERR_INVALID_ARG;
  auto it = c->tensors.find(name);
  if (it == c->tensors.end()) return RPO_ERR_INVALID_ARG;
  const TensorInfo& t = it->second;
  const size_t e = t.gain ? 4 : c->esz;
  if (bytes != (size_t)t.rows * t.cols * e) return RPO_ERR_INVALID_ARG;
  const size_t row_bytes = (size_t)t.cols * e;
  char* base = (char*)t.ptr + (size_t)t.row_add * row_bytes;
  const size_t pitch = row_bytes * t.row_mul;
  if (write)
    CUDA_TRY(cudaMemcpy2DAsync(base, pitch, host, row_bytes, row_bytes, t.rows, cudaMemcpyHostToDevice, c->stream));
  else
    CUDA_TRY(cudaMemcpy2DAsync(host, row_bytes, base, pitch, row_bytes, t.rows, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  if (write) c->weights_ready = true;
  return RPO_OK;
}
extern "C" int rpo_read_tensor(rpo_ctx* c, const char* name, void* h_dst, size_t bytes) {
  return tensor_io(c, name, h_dst, bytes, false);
}
extern "C" int rpo_write_tensor(rpo_ctx* c, const char* name, const void* h_src, size_t bytes) {
  return tensor_io(c, name, const_cast<void*>(h_src), bytes, true);
}

// ---------------------------------------------------------------------------------------------
// building blocks
// ---------------------------------------------------------------------------------------------
template <typename T>
static KVPool<T> kv_pool(rpo_ctx* c) {
  KVPool<T> p;
  p.base = (T*)c->kv_base; p.layer_stride = c->kv_layer_stride; p.kv_stride = c->kv_kv_stride;
  p.head_stride = c->kv_head_stride; p.n_blocks = (int32_t)c->lim.kv_pool_blocks; p.head_dim = c->shape.head_dim;
  return p;
}

// Split-K partial sums of the last residual-add GEMM wait in ws.partial until the next RMSNorm
// (which folds the reduction in) or an explicit flush.
static int flush_partials(rpo_ctx* c) {
  if (c->pending_splits == 0) return RPO_OK;
  const int64_t n = (int64_t)c->pending_rows * c->shape.d_model;
  LAUNCH(c, reduce_partials_kernel, grid_for(n / 4, 256), 256, 0, c->ws.x, (const float*)c->ws.partial, c->pending_splits,
         n, n);
  c->pending_splits = 0;
  return RPO_OK;
}

// C = A W^T with the chosen epilogue.  impl: 0 auto, 1 CUDA cores, 2 tcgen05.
// EPI_SWIGLU is only valid on the tensor-core path (callers check tc_gemm_supported first).
// allow_split: the tensor-core kernel may leave split-K partial planes in ws.partial instead of
// applying the epilogue.  For EPI_ADD_F32 on ws.x the next RMSNorm (or flush_partials) folds them
// in; for other epilogues the caller must pass splits_out and reduce the planes itself.
// Fused epilogues (TC_N*, TC_QKV_ROPE, TC_ADD_NORM; 16-bit models on the tensor-core kernels only):
// C = A W^T with the layer's elementwise work done in the epilogue; split-K is reduced inside the kernel.
static int gemm_fused(rpo_ctx* c, const bf16* A, const bf16* W, void* C, int M, int N, int K, int tc_epi, int ldc, TcFuse& fuse) {
  if (M <= 0) return RPO_OK;
  ProfScope ps(c, KC_GEMM);
  static const char* labels[] = {"gemm", "gemm", "gemm", "gemm", "gemm", "gemm (1/rms, float32 store: output head)",
                                 "gemm (1/rms, SwiGLU: gate/up)", "gemm (1/rms, RoPE, KV append: qkv)", "gemm (residual add, next norm: O / down)",
                                 "gemm (1/rms, 1/T, log-sum-exp parts: output head of the log-prob pass)"};
  prof_begin(c, labels[tc_epi]);
  const int rc = (tc_epi == TC_NLSE || tc2_wanted(c, M, N, K, true)) ? tc2_gemm_launch(c, A, W, C, M, N, K, tc_epi, ldc, true, nullptr, &fuse)
                                              : tc_gemm_launch(c, A, W, C, M, N, K, tc_epi, ldc, true, nullptr, &fuse);
  prof_end(c);
  c->launches++;
  return rc;
}

template <typename T>
static int gemm(rpo_ctx* c, const T* A, const T* W, void* C, int M, int N, int K, int epi, int impl = 0,
                bool allow_split = false, int* splits_out = nullptr) {
  if (splits_out) *splits_out = 0;
  if (M <= 0) return RPO_OK;
  ProfScope ps(c, KC_GEMM);
  if (impl != 1 && tc_gemm_supported<T>(c, M, N, K) && (impl == 2 || c->use_tcgen05)) {
    const int tc_epi = epi == EPI_STORE_T ? TC_STORE_BF16 : epi == EPI_STORE_F32 ? TC_STORE_F32
                     : epi == EPI_ADD_F32 ? TC_ADD_F32 : TC_SWIGLU;
    int splits = 0;
    prof_begin(c);
    const int ldc = tc_epi == TC_SWIGLU ? N / 2 : N;
    const bool may_split = allow_split && (epi == EPI_ADD_F32 || splits_out);
    const int rc = tc2_wanted(c, M, N, K, may_split)
                       ? tc2_gemm_launch(c, (const bf16*)A, (const bf16*)W, C, M, N, K, tc_epi, ldc, may_split, &splits)
                       : tc_gemm_launch(c, (const bf16*)A, (const bf16*)W, C, M, N, K, tc_epi, ldc, may_split, &splits);
    prof_end(c);
    c->launches++;
    if (rc == RPO_OK && splits > 1) {
      if (epi == EPI_ADD_F32) { c->pending_splits = splits; c->pending_rows = M; }
      else *splits_out = splits;
    }
    return rc;
  }
  if (impl == 2 || epi == EPI_SWIGLU) return RPO_ERR_SHAPE;
  dim3 grid(ceil_div(N, 64), ceil_div(M, 64));
  if (epi == EPI_STORE_T) LAUNCH(c, (gemm_ref_kernel<T, EPI_STORE_T>), grid, 256, 0, A, W, C, M, N, K, (int64_t)N);
  else if (epi == EPI_STORE_F32) LAUNCH(c, (gemm_ref_kernel<T, EPI_STORE_F32>), grid, 256, 0, A, W, C, M, N, K, (int64_t)N);
  else LAUNCH(c, (gemm_ref_kernel<T, EPI_ADD_F32>), grid, 256, 0, A, W, C, M, N, K, (int64_t)N);
  return RPO_OK;
}

template <typename T>
static int rmsnorm(rpo_ctx* c, float* x, const float* g, T* h, int rows) {
  if (rows <= 0) return RPO_OK;
  ProfScope ps(c, KC_NORM);
  const int d = c->shape.d_model;
  const bool fold = (x == c->ws.x && c->pending_splits > 0 && c->pending_rows == rows);
  if (!fold && x == c->ws.x) RPO_TRY(flush_partials(c));
  if (!fold && rows >= 1024 && d <= 4096) {     // many rows: a warp per row, the row in registers
    if (d <= 2048) LAUNCH(c, (rmsnorm_rows_kernel<T, 16>), ceil_div(rows, 8), 256, 0, (const float*)x, g, h, rows, d, c->shape.rms_eps);
    else LAUNCH(c, (rmsnorm_rows_kernel<T, 32>), ceil_div(rows, 8), 256, 0, (const float*)x, g, h, rows, d, c->shape.rms_eps);
    return RPO_OK;
  }
  const int threads = std::min(1024, ((d / 4 + 31) / 32) * 32);
  LAUNCH(c, rmsnorm_kernel<T>, rows, threads, (size_t)d * 4, x, g, h, rows, d, c->shape.rms_eps,
         fold ? (const float*)c->ws.partial : (const float*)nullptr, fold ? c->pending_splits : 0,
         (int64_t)rows * d);
  if (fold) c->pending_splits = 0;
  return RPO_OK;
}

template <int DH, int MODE, bool CLM = false>
static int launch_flash(rpo_ctx* c, const FlashArgs& a, dim3 grid) {
  constexpr int smem = FaCfg<MODE>::template smem_bytes<DH>();
  static bool attr_done[64] = {};
  if (tc_first_use_on_device(c, attr_done))
    CUDA_TRY(cudaFuncSetAttribute(flash_attn_kernel<DH, MODE, CLM>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  if (CLM) c->launch_cluster_x = a.n_splits;         // the splits of a work item are consecutive along x
  LAUNCH(c, (flash_attn_kernel<DH, MODE, CLM>), grid, FaCfg<MODE>::THREADS + 32, smem, a);
  return RPO_OK;
}

// Split counts whose CTAs can merge inside a cluster (portable cluster sizes).
static bool cluster_mergeable(int n_splits) { return n_splits == 1 || n_splits == 2 || n_splits == 4 || n_splits == 8; }

// The tcgen05 attention serves prefill / teacher-forced passes of bf16 models with head_dim 128.
static bool tc5_attention(rpo_ctx* c) {
  return c->bf16 && c->use_tc_attention && c->use_tc5_attention && c->shape.head_dim == T5_DH;
}

template <typename T>
static int attention(rpo_ctx* c, int layer, int rows) {
  const rpo_shape& s = c->shape;
  Workspace& w = c->ws;
  const float scale = 1.0f / sqrtf((float)s.head_dim);
  ProfScope ps(c, KC_ATTN);
  if constexpr (std::is_same<T, bf16>::value) {
    if (c->use_tc_attention) {
      FlashArgs a;
      memset(&a, 0, sizeof(a));
      a.qkv = (const bf16*)w.qkv; a.qkv_cols = c->qkv_cols; a.out = (bf16*)w.attn; a.out_cols = s.n_q_heads * s.head_dim;
      a.part_ml = w.attn_part; a.part_o = w.attn_part + (size_t)2 * c->lim.max_seqs * s.n_q_heads * 33;
      a.row_seq = w.row_seq; a.row_t = w.row_t; a.seqs = (const SeqDesc*)w.seqs; a.block_table = c->d_block_table;
      a.pool = kv_pool<bf16>(c); a.layer = layer; a.hq = s.n_q_heads; a.hkv = s.n_kv_heads;
      a.scale_log2 = scale * 1.4426950408889634f; a.tiles = (const int2*)w.tiles; a.G = c->attn_G; a.status = c->d_status;
      a.n_splits = c->attn_splits; a.split_chunk = c->attn_split_chunk; a.pfx_tbl = w.pfx_tbl; a.pfx_stride = w.pfx_stride;
      if (c->attn_mode == 0 && tc5_attention(c)) {
        // tcgen05 path: 128-row tiles, Q through a tensor map over the fused qkv buffer
        const CUtensorMap* qm = tc_map(c, w.qkv, w.R, c->qkv_cols, T5_BM);
        if (!qm) return RPO_ERR_CUDA;
        Flash5Args f;
        memset(&f, 0, sizeof(f));
        f.out = (bf16*)w.attn; f.out_cols = s.n_q_heads * s.head_dim; f.row_seq = w.row_seq; f.row_t = w.row_t;
        f.seqs = (const SeqDesc*)w.seqs; f.block_table = c->d_block_table; f.pool = kv_pool<bf16>(c); f.layer = layer;
        f.hq = s.n_q_heads; f.hkv = s.n_kv_heads; f.scale_log2 = scale * 1.4426950408889634f; f.tiles = (const int2*)w.tiles;
        f.q_col0 = 0; f.status = c->d_status;
        if (c->use_tc5_pipelined) {                    // 64-key tiles, O accumulated in tensor memory
          static bool p5_attr[64] = {};
          if (tc_first_use_on_device(c, p5_attr))
            CUDA_TRY(cudaFuncSetAttribute(flash_prefill_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P5_SMEM));
          LAUNCH(c, flash_prefill_tc5_kernel, dim3(s.n_q_heads, c->attn_tiles), 320, P5_SMEM, *qm, f);
          return RPO_OK;
        }
        static bool attr_done[64] = {};
        if (tc_first_use_on_device(c, attr_done))
          CUDA_TRY(cudaFuncSetAttribute(flash_attn_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, T5_SMEM));
        LAUNCH(c, flash_attn_tc5_kernel, dim3(s.n_q_heads, c->attn_tiles), 320, T5_SMEM, *qm, f);
        return RPO_OK;
      }
      if (c->attn_mode == 0) {
        dim3 grid(s.n_q_heads, c->attn_tiles);
        return s.head_dim == 128 ? launch_flash<128, FA_ROWS>(c, a, grid) : launch_flash<64, FA_ROWS>(c, a, grid);
      }
      const int rep = s.n_q_heads / s.n_kv_heads;
      a.n_slots = a.n_splits; a.slot_base = 0; a.skip_prefix = 0;
      if (c->attn_dec5) {
        // one tcgen05 work item per (group, KV head, split): its prefix split, then its share of the suffix tiles
        Decode5Args d5;
        memset(&d5, 0, sizeof(d5));
        d5.qkv = (const bf16*)w.qkv; d5.qkv_cols = c->qkv_cols; d5.part_ml = a.part_ml; d5.part_o = a.part_o; d5.n_slots = c->attn_splits;
        d5.pfx_tbl = w.pfx_tbl; d5.pfx_stride = w.pfx_stride; d5.seqs = (const SeqDesc*)w.seqs; d5.row_t = w.row_t;
        d5.block_table = c->d_block_table; d5.pool = kv_pool<bf16>(c);
        d5.layer = layer; d5.hq = s.n_q_heads; d5.hkv = s.n_kv_heads; d5.G = c->attn_G; d5.scale_log2 = a.scale_log2;
        d5.n_splits = c->attn_splits; d5.split_chunk = c->attn_split_chunk; d5.status = c->d_status;
        static bool d5_attr[64] = {};
        if (tc_first_use_on_device(c, d5_attr))
          CUDA_TRY(cudaFuncSetAttribute(flash_decode_tc5_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, D5_SMEM));
        LAUNCH(c, flash_decode_tc5_kernel, dim3(c->attn_groups * c->attn_splits, s.n_kv_heads), 320, D5_SMEM, d5);
        const int mgrid = ceil_div((int64_t)rows * s.n_q_heads, 4);
        LAUNCH(c, (attn_decode_merge_kernel<128>), mgrid, 128, 0, a.out, a.part_ml, a.part_o, c->attn_splits, w.row_t, rows, a.hq);
        return RPO_OK;
      }
      dim3 grid(c->attn_groups * ceil_div(c->attn_G * rep, FA_BM) * c->attn_splits, s.n_kv_heads);
      if (c->use_cluster_merge && cluster_mergeable(a.n_splits))
        return s.head_dim == 128 ? launch_flash<128, FA_SHARED, true>(c, a, grid) : launch_flash<64, FA_SHARED, true>(c, a, grid);
      RPO_TRY((s.head_dim == 128 ? launch_flash<128, FA_SHARED>(c, a, grid) : launch_flash<64, FA_SHARED>(c, a, grid)));
      const int mgrid = ceil_div((int64_t)rows * s.n_q_heads, 4);
      if (s.head_dim == 128)
        LAUNCH(c, (attn_decode_merge_kernel<128>), mgrid, 128, 0, a.out, a.part_ml, a.part_o, a.n_splits, w.row_t, rows, a.hq);
      else
        LAUNCH(c, (attn_decode_merge_kernel<64>), mgrid, 128, 0, a.out, a.part_ml, a.part_o, a.n_splits, w.row_t, rows, a.hq);
      return RPO_OK;
    }
  }
  const int grid = ceil_div((int64_t)rows * s.n_q_heads, 4);
  if (s.head_dim == 64)
    LAUNCH(c, (attn_ref_kernel<T, 64>), grid, 128, 0, (const T*)w.qkv, (T*)w.attn, w.row_seq, w.row_t,
           (const SeqDesc*)w.seqs, c->d_block_table, kv_pool<T>(c), layer, rows, s.n_q_heads, s.n_kv_heads, scale,
           c->d_status);
  else
    LAUNCH(c, (attn_ref_kernel<T, 128>), grid, 128, 0, (const T*)w.qkv, (T*)w.attn, w.row_seq, w.row_t,
           (const SeqDesc*)w.seqs, c->d_block_table, kv_pool<T>(c), layer, rows, s.n_q_heads, s.n_kv_heads, scale,
           c->d_status);
  return RPO_OK;
}

// Query-row tiles (128 rows for the tcgen05 attention, else 64) of a pass whose sequences own
// consecutive row ranges.
static int upload_row_tiles(rpo_ctx* c, const std::vector<int>& rows_per_seq) {
  // Tiles deeper into a sequence see more keys (causal attention): heaviest first, so the launch
  // does not end on a few long tiles.
  std::vector<std::pair<int, int2>> weighted;
  const int bm = tc5_attention(c) ? T5_BM : FA_BM;
  int r = 0;
  for (int n : rows_per_seq) {
    for (int r0 = 0; r0 < n; r0 += bm) weighted.push_back({r0 + std::min(bm, n - r0), make_int2(r + r0, std::min(bm, n - r0))});
    r += n;
  }
  std::stable_sort(weighted.begin(), weighted.end(), [](const std::pair<int, int2>& a, const std::pair<int, int2>& b) { return a.first > b.first; });
  std::vector<int2> tiles;
  tiles.reserve(weighted.size());
  for (const auto& t : weighted) tiles.push_back(t.second);
  c->attn_mode = 0; c->attn_tiles = (int)tiles.size();
  if (!tiles.empty())
    CUDA_TRY(cudaMemcpyAsync(c->ws.tiles, tiles.data(), tiles.size() * sizeof(int2), cudaMemcpyHostToDevice, c->stream));
  return RPO_OK;
}

// Test tap (rpo_debug_tap): the residual rows of the pass are appended to the caller's buffer.
static int tap_copy(rpo_ctx* c, const void* src, int64_t bytes) {
  const int64_t n = (bytes + 3) / 4;
  if (c->tap_used + n > c->tap_capacity) return RPO_ERR_LIMIT;
  CUDA_TRY(cudaMemcpyAsync(c->tap_buf + c->tap_used, src, (size_t)bytes, cudaMemcpyDeviceToDevice, c->stream));
  c->tap_used += n;
  return RPO_OK;
}
static int tap_rows(rpo_ctx* c, int rows) {            // the residual rows
  if (!c->tap_buf) return RPO_OK;
  RPO_TRY(flush_partials(c));
  return tap_copy(c, c->ws.x, (int64_t)rows * c->shape.d_model * 4);
}
static int tap_attn(rpo_ctx* c, int rows) {            // the attention output rows, in the storage type
  if (!c->tap_buf) return RPO_OK;
  return tap_copy(c, c->ws.attn, (int64_t)rows * c->shape.n_q_heads * c->shape.head_dim * (int64_t)c->esz);
}

static int read_status(rpo_ctx* c, int* word);
static bool fused_layers(rpo_ctx* c, int rows);
static int run_layers_fused(rpo_ctx* c, int rows);

// The layer stack over `rows` rows of ws.x, whose (sequence, private index) metadata sits in
// ws.row_seq / ws.row_t and whose sequence descriptors sit in ws.seqs.
// flush = false leaves the last layer's split-K partials pending for the caller's next RMSNorm on ws.x.
template <typename T>
static int run_layers(rpo_ctx* c, int rows, bool flush = true) {
  if (fused_layers(c, rows)) return run_layers_fused(c, rows);
  const rpo_shape& s = c->shape;
  Workspace& w = c->ws;
  const int d = s.d_model, F = s.d_ffn, qo = s.n_q_heads * s.head_dim;
  RPO_TRY(tap_rows(c, rows));
  for (int l = 0; l < s.n_layers; ++l) {
    const LayerWeights& L = c->layers[l];
    RPO_TRY(rmsnorm<T>(c, w.x, L.g1, (T*)w.h, rows));
    int qkv_splits = 0;
    RPO_TRY(gemm<T>(c, (const T*)w.h, (const T*)L.wqkv, w.qkv, rows, c->qkv_cols, d, EPI_STORE_T, 0, true, &qkv_splits));
    { ProfScope ps(c, KC_ROPE);
    LAUNCH(c, rope_kv_kernel<T>, ceil_div((int64_t)rows * (s.n_q_heads + 2 * s.n_kv_heads) * (s.head_dim / 16), 64), 64, 0, (T*)w.qkv,
           (const int4*)w.row_meta, (const float2*)c->d_rope, kv_pool<T>(c), l, rows, s.n_q_heads, s.n_kv_heads,
           qkv_splits > 1 ? (const float*)w.partial : (const float*)nullptr, qkv_splits, (int64_t)rows * c->qkv_cols); }
    RPO_TRY(attention<T>(c, l, rows));
    RPO_TRY(tap_attn(c, rows));
    RPO_TRY(gemm<T>(c, (const T*)w.attn, (const T*)L.wo, w.x, rows, d, qo, EPI_ADD_F32, 0, true));
    RPO_TRY(rmsnorm<T>(c, w.x, L.g2, (T*)w.h, rows));
    if (c->use_tcgen05 && tc_gemm_supported<T>(c, rows, 2 * F, d) && F % 8 == 0) {
      RPO_TRY(gemm<T>(c, (const T*)w.h, (const T*)L.wgu, w.act, rows, 2 * F, d, EPI_SWIGLU));   // SwiGLU in the epilogue
    } else {
      RPO_TRY(gemm<T>(c, (const T*)w.h, (const T*)L.wgu, w.gu, rows, 2 * F, d, EPI_STORE_T));
      LAUNCH(c, swiglu_kernel<T>, grid_for((int64_t)rows * F, 256), 256, 0, (const T*)w.gu, (T*)w.act, (int64_t)rows * F);
    }
    RPO_TRY(gemm<T>(c, (const T*)w.act, (const T*)L.wd, w.x, rows, d, F, EPI_ADD_F32, 0, true));
    RPO_TRY(tap_rows(c, rows));
  }
  return flush ? flush_partials(c) : RPO_OK;
}

// True when the layer stack runs with the fused GEMM epilogues (gemm_epi.cuh): 16-bit model, tensor-
// core kernels on, every product of the layer in the shape the tensor-core kernel takes.
// Split-K factor the planner would pick for a fused product of `rows` rows.
static int fused_splits(rpo_ctx* c, int rows, int N, int K, int epi, int bn_multiple) {
  if (tc2_wanted(c, rows, N, K, true)) return (rows <= 128 && c->gemm_bn == 0) ? 1 : tc2_splits(c, rows, N, K, true);
  return tc_plan(c, rows, N, K, epi, true, bn_multiple).splits;
}

static bool fused_layers(rpo_ctx* c, int rows) {
  const rpo_shape& s = c->shape;
  if (!c->bf16 || !c->use_tcgen05 || !c->use_fused_layers) return false;
  const int qo = s.n_q_heads * s.head_dim;
  if (!(tc_gemm_supported<bf16>(c, 1, c->qkv_cols, s.d_model) && tc_gemm_supported<bf16>(c, 1, s.d_model, qo) &&
        tc_gemm_supported<bf16>(c, 1, 2 * s.d_ffn, s.d_model) && tc_gemm_supported<bf16>(c, 1, s.d_model, s.d_ffn) &&
        tc_gemm_supported<bf16>(c, 1, s.vocab, s.d_model) && s.d_ffn % 8 == 0))
    return false;
  if (c->use_fused_layers >= 2) return true;           // forced (tests)
  // A split-K launch with a fused epilogue is reduced by the last warp to arrive at each 32-row unit, so
  // a few warps per tile do alone what a reduction kernel spreads over the whole machine: measured 12-17 %
  // slower per decode forward (256 / 512 sequences, 2-5 planes), neutral at 128 sequences.  Passes whose
  // products split K (decode batches) therefore keep the unfused kernels; prefill and teacher-forced
  // passes, which never split, run fused (-3 % / -9 % measured).
  const int lim = c->fused_split_limit;
  return fused_splits(c, rows, c->qkv_cols, s.d_model, TC_QKV_ROPE, s.head_dim) <= lim &&
         fused_splits(c, rows, s.d_model, qo, TC_ADD_NORM, 1) <= lim && fused_splits(c, rows, s.d_model, s.d_ffn, TC_ADD_NORM, 1) <= lim;
}

// What embed_kernel writes besides x when the layers are fused: xg = bf16(x * g1 of layer 0), sum of squares.
static void embed_norm_args(rpo_ctx* c, int rows, const float*& gain, bf16*& xg, float*& ssq) {
  gain = nullptr; xg = nullptr; ssq = nullptr;
  if (!fused_layers(c, rows) || c->shape.n_layers == 0) return;
  gain = c->layers[0].g1; xg = (bf16*)c->ws.h; ssq = c->ws.ssq;
  c->ssq_parts = 1;
}

static TcFuse fuse_norm_in(rpo_ctx* c) {             // the consumer side of a fused RMSNorm
  TcFuse f;
  f.ssq_in = c->ws.ssq; f.ssq_in_parts = c->ssq_parts; f.norm_dim = c->shape.d_model; f.eps = c->shape.rms_eps;
  return f;
}

// The layer stack with five kernels per layer.  On entry ws.x holds the residual rows, ws.h = bf16(x *
// g1 of layer 0) and ws.ssq their sums of squares (c->ssq_parts parts per row).  On return ws.h =
// bf16(x * final_gain) and ws.ssq belong to the rows leaving the last layer (the output head's input).
static int run_layers_fused(rpo_ctx* c, int rows) {
  const rpo_shape& s = c->shape;
  Workspace& w = c->ws;
  const int d = s.d_model, F = s.d_ffn, qo = s.n_q_heads * s.head_dim;
  RPO_TRY(tap_rows(c, rows));
  for (int l = 0; l < s.n_layers; ++l) {
    const LayerWeights& L = c->layers[l];
    {
      TcFuse f = fuse_norm_in(c);
      f.row_meta = (const int4*)w.row_meta; f.rope = (const float2*)c->d_rope; f.pool = kv_pool<bf16>(c); f.layer = l;
      f.hq = s.n_q_heads; f.hkv = s.n_kv_heads; f.head_dim = s.head_dim;
      RPO_TRY(gemm_fused(c, (const bf16*)w.h, (const bf16*)L.wqkv, w.qkv, rows, c->qkv_cols, d, TC_QKV_ROPE, c->qkv_cols, f));
    }
    RPO_TRY(attention<bf16>(c, l, rows));
    RPO_TRY(tap_attn(c, rows));
    {
      TcFuse f;
      f.ssq_out = w.ssq; f.xg_out = (bf16*)w.h; f.gain = L.g2;
      RPO_TRY(gemm_fused(c, (const bf16*)w.attn, (const bf16*)L.wo, w.x, rows, d, qo, TC_ADD_NORM, d, f));
      c->ssq_parts = f.ssq_out_parts;
    }
    {
      TcFuse f = fuse_norm_in(c);
      RPO_TRY(gemm_fused(c, (const bf16*)w.h, (const bf16*)L.wgu, w.act, rows, 2 * F, d, TC_NSWIGLU, F, f));
    }
    {
      TcFuse f;
      f.ssq_out = w.ssq; f.xg_out = (bf16*)w.h; f.gain = (l + 1 < s.n_layers) ? c->layers[l + 1].g1 : c->gf;
      RPO_TRY(gemm_fused(c, (const bf16*)w.act, (const bf16*)L.wd, w.x, rows, d, F, TC_ADD_NORM, d, f));
      c->ssq_parts = f.ssq_out_parts;
    }
    RPO_TRY(tap_rows(c, rows));
  }
  return RPO_OK;
}

// logits[n, V] (float32, ws.logits) from n residual rows in ws.xh.
template <typename T>
static int head(rpo_ctx* c, int n) {
  Workspace& w = c->ws;
  if (fused_layers(c, 1 << 20)) {                      // (many rows: no split question) the output head takes bf16(x * g) rows
    ProfScope ps(c, KC_NORM);
    LAUNCH(c, norm_prep_kernel, n, 128, 0, (const float*)w.xh, (const float*)c->gf, (bf16*)w.hh, w.ssq_h, n, c->shape.d_model);
    TcFuse f;
    f.ssq_in = w.ssq_h; f.ssq_in_parts = 1; f.norm_dim = c->shape.d_model; f.eps = c->shape.rms_eps;
    return gemm_fused(c, (const bf16*)w.hh, (const bf16*)c->lm_head, w.logits, n, c->shape.vocab, c->shape.d_model, TC_NSTORE_F32,
                      c->shape.vocab, f);
  }
  RPO_TRY(rmsnorm<T>(c, w.xh, c->gf, (T*)w.hh, n));
  return gemm<T>(c, (const T*)w.hh, (const T*)c->lm_head, w.logits, n, c->shape.vocab, c->shape.d_model, EPI_STORE_F32);
}

static int take_blocks(rpo_ctx* c, int n, std::vector<int32_t>& out) {
  if ((int64_t)c->free_blocks.size() < n) return RPO_ERR_KV_POOL;
  for (int i = 0; i < n; ++i) { out.push_back(c->free_blocks.back()); c->free_blocks.pop_back(); }
  return RPO_OK;
}
static void give_blocks(rpo_ctx* c, std::vector<int32_t>& b) {
  for (auto it = b.rbegin(); it != b.rend(); ++it) c->free_blocks.push_back(*it);
  b.clear();
}

static int check_groups(rpo_ctx* c, int n_groups, const rpo_group* g) {
  if (n_groups > c->lim.max_groups) return RPO_ERR_LIMIT;      // (a handle given twice would also exceed the per-call tables)
  std::vector<char> seen(c->lim.max_groups, 0);
  for (int i = 0; i < n_groups; ++i) {
    if (g[i].slot >= 0 && g[i].slot < c->lim.max_groups) {
      if (seen[g[i].slot]) return RPO_ERR_INVALID_ARG;
      seen[g[i].slot] = 1;
    }
    if (g[i].slot < 0 || g[i].slot >= c->lim.max_groups) return RPO_ERR_NOT_INITIALISED;
    const GroupState& gs = c->groups[g[i].slot];
    if (!gs.live || gs.group_id != g[i].group_id || gs.prefix_len != g[i].prefix_len) return RPO_ERR_NOT_INITIALISED;
  }
  return RPO_OK;
}

// ---------------------------------------------------------------------------------------------
// prefill
// ---------------------------------------------------------------------------------------------
template <typename T>
static int prefill_chunk(rpo_ctx* c, const int32_t* d_tokens, int tok0, const std::vector<int>& slots,
                         const std::vector<int>& lens) {
  Workspace& w = c->ws;
  const int n = (int)slots.size();
  int rows = 0;
  for (int l : lens) rows += l;
  std::vector<int32_t> row_seq(rows), row_t(rows), last(n);
  std::vector<SeqDesc> sd(n);
  int r = 0;
  for (int i = 0; i < n; ++i) {
    sd[i].shared_tbl = -1; sd[i].shared_len = 0; sd[i].priv_tbl = slots[i] * c->tbl_stride; sd[i].reserved = 0;
    for (int t = 0; t < lens[i]; ++t, ++r) { row_seq[r] = i; row_t[r] = t; }
    last[i] = r - 1;
    const GroupState& gs = c->groups[slots[i]];
    CUDA_TRY(cudaMemcpyAsync(c->d_block_table + (size_t)slots[i] * c->tbl_stride, gs.blocks.data(),
                             gs.blocks.size() * 4, cudaMemcpyHostToDevice, c->stream));
  }
  CUDA_TRY(cudaMemcpyAsync(w.row_seq, row_seq.data(), (size_t)rows * 4, cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(cudaMemcpyAsync(w.row_t, row_t.data(), (size_t)rows * 4, cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(cudaMemcpyAsync(w.seqs, sd.data(), (size_t)n * sizeof(SeqDesc), cudaMemcpyHostToDevice, c->stream));
  RPO_TRY(upload_row_tiles(c, lens));
  const float* e_gain; bf16* e_xg; float* e_ssq;
  embed_norm_args(c, rows, e_gain, e_xg, e_ssq);
  LAUNCH(c, embed_kernel<T>, rows, 128, 0, d_tokens + tok0, (const T*)c->embed, w.x, rows, c->shape.d_model,
         c->shape.vocab, c->d_status, (int32_t*)nullptr, row_meta_args(c), e_gain, e_xg, e_ssq);
  RPO_TRY(run_layers<T>(c, rows));
  // keep the residual stream of every group's last prefix token: step-0 logits come from it
  for (int i = 0; i < n; ++i)
    CUDA_TRY(cudaMemcpyAsync(c->d_x_last + (size_t)slots[i] * c->shape.d_model, w.x + (size_t)last[i] * c->shape.d_model,
                             (size_t)c->shape.d_model * 4, cudaMemcpyDeviceToDevice, c->stream));
  return RPO_OK;
}

extern "C" int rpo_prefill_prefix(rpo_ctx* c, int32_t n_groups, const int32_t* d_tokens, const int32_t* h_offsets,
                                  const int32_t* h_group_ids, rpo_group* h_groups_out) {
  if (!c || n_groups < 0 || (n_groups > 0 && (!d_tokens || !h_offsets || !h_groups_out))) return RPO_ERR_INVALID_ARG;
  if (!c->weights_ready) return RPO_ERR_NOT_INITIALISED;
  RPO_TRY(enter(c));
  c->prof_phase = 0;
  int64_t need_blocks = 0;
  for (int g = 0; g < n_groups; ++g) {
    const int len = h_offsets[g + 1] - h_offsets[g];
    if (len < 1) return RPO_ERR_INVALID_ARG;
    if (len > c->lim.max_chunk_tokens || len >= c->lim.max_positions) return RPO_ERR_LIMIT;
    need_blocks += ceil_div(len, KV_BLOCK);
  }
  if (need_blocks > (int64_t)c->free_blocks.size() || n_groups > (int)c->free_slots.size()) return RPO_ERR_KV_POOL;
  std::vector<int> slots(n_groups), lens(n_groups);
  for (int g = 0; g < n_groups; ++g) {
    const int slot = c->free_slots.back();
    c->free_slots.pop_back();
    GroupState& gs = c->groups[slot];
    gs.live = true; gs.group_id = h_group_ids ? h_group_ids[g] : g; gs.prefix_len = h_offsets[g + 1] - h_offsets[g];
    gs.blocks.clear();
    take_blocks(c, ceil_div(gs.prefix_len, KV_BLOCK), gs.blocks);
    slots[g] = slot; lens[g] = gs.prefix_len;
    h_groups_out[g].group_id = gs.group_id; h_groups_out[g].prefix_len = gs.prefix_len;
    h_groups_out[g].slot = slot; h_groups_out[g].n_blocks = (int32_t)gs.blocks.size();
  }
  int rc = RPO_OK;
  int g0 = 0;
  while (g0 < n_groups && rc == RPO_OK) {
    int g1 = g0, rows = 0;
    while (g1 < n_groups && rows + lens[g1] <= c->lim.max_chunk_tokens) rows += lens[g1++];
    std::vector<int> cs(slots.begin() + g0, slots.begin() + g1), cl(lens.begin() + g0, lens.begin() + g1);
    rc = c->bf16 ? prefill_chunk<bf16>(c, d_tokens, h_offsets[g0], cs, cl)
                 : prefill_chunk<float>(c, d_tokens, h_offsets[g0], cs, cl);
    g0 = g1;
  }
  if (rc != RPO_OK) rpo_release_groups(c, n_groups, h_groups_out);
  return rc;
}

extern "C" int rpo_release_groups(rpo_ctx* c, int32_t n_groups, const rpo_group* g) {
  if (!c || n_groups < 0 || (n_groups > 0 && !g)) return RPO_ERR_INVALID_ARG;
  int rc = RPO_OK;
  for (int i = 0; i < n_groups; ++i) {
    if (g[i].slot < 0 || g[i].slot >= c->lim.max_groups || !c->groups[g[i].slot].live) { rc = RPO_ERR_NOT_INITIALISED; continue; }
    GroupState& gs = c->groups[g[i].slot];
    give_blocks(c, gs.blocks);
    give_blocks(c, gs.wave_blocks);
    for (auto it = gs.wave_rows.rbegin(); it != gs.wave_rows.rend(); ++it) c->free_state_rows.push_back(*it);
    gs.wave_rows.clear();
    gs.wave_G = gs.wave_total = gs.wave_t = 0;
    gs.live = false;
    c->free_slots.push_back(g[i].slot);
  }
  return rc;
}

// ---------------------------------------------------------------------------------------------
// decode
// ---------------------------------------------------------------------------------------------
static int launch_sampler(rpo_ctx* c, int n_rows, const SamplerArgs& a) {
  static bool attr_done[64] = {};
  if (tc_first_use_on_device(c, attr_done))
    CUDA_TRY(cudaFuncSetAttribute(sampler_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SAMPLER_SMEM));
  ProfScope ps(c, KC_SAMPLER);
  LAUNCH(c, sampler_kernel, n_rows, 1024, SAMPLER_SMEM, a);
  return RPO_OK;
}

static SamplerArgs sampler_args(rpo_ctx* c, const rpo_sampler* sp) {
  SamplerArgs a;
  memset(&a, 0, sizeof(a));
  a.V = c->shape.vocab;
  a.temperature = sp->temperature;
  a.top_p24 = (uint32_t)floorf(sp->top_p * 16777216.0f);
  a.greedy = sp->greedy; a.eos_id = sp->eos_id; a.seed = sp->seed;
  a.weights = c->ws.sampler_w;
  return a;
}

static int check_sampler(const rpo_sampler* sp) {
  if (!sp || !(sp->temperature > 0.f) || !(sp->top_p >= 0.f && sp->top_p <= 1.f)) return RPO_ERR_INVALID_ARG;
  return RPO_OK;
}

template <typename T>
static int decode_t(rpo_ctx* c, int n_groups, const rpo_group* groups, int G, int S, const rpo_sampler* sp,
                    const int32_t* d_forced, int32_t* d_tokens_out, int32_t* d_lens_out, float* d_logprobs_out,
                    float* d_logits_dbg, std::vector<int32_t>& priv_blocks, bool wave = false) {
  // wave: the call continues the groups' sequences where their last rpo_decode_wave call stopped; blocks and state
  // rows were reserved by the caller and stay with the groups
  Workspace& w = c->ws;
  const int B = n_groups * G, d = c->shape.d_model;
  const int per_seq = ceil_div(std::max(S - 1, 0), KV_BLOCK);
  if (!wave) RPO_TRY(take_blocks(c, B * per_seq, priv_blocks));
  std::vector<SeqDesc> sd(B);
  std::vector<int32_t> tbl((size_t)B * c->tbl_stride, -1), logit_row(B), slot_idx(n_groups), zero(B, 0), seq_of_row(B);
  std::vector<int32_t> t_base(B, 0), state_idx(B, -1), done_idx(B, -1);
  std::vector<int64_t> seq_ids(B);
  int n_fresh = 0;                                       // wave: groups that start with this call, in call order
  for (int g = 0; g < n_groups; ++g) {
    slot_idx[g] = groups[g].slot;
    const GroupState& gs = c->groups[groups[g].slot];
    if (wave && gs.wave_t == 0) slot_idx[n_fresh] = groups[g].slot;
    for (int i = 0; i < G; ++i) {
      const int b = g * G + i;
      sd[b].shared_tbl = groups[g].slot * c->tbl_stride; sd[b].shared_len = groups[g].prefix_len;
      sd[b].priv_tbl = (c->lim.max_groups + b) * c->tbl_stride; sd[b].reserved = 0;
      if (wave) {
        const int per = ceil_div(gs.wave_total, KV_BLOCK);
        for (int k = 0; k < per; ++k) tbl[(size_t)b * c->tbl_stride + k] = gs.wave_blocks[(size_t)i * per + k];
        t_base[b] = gs.wave_t;
        state_idx[b] = gs.wave_rows[i];                                // where the sequence's state is parked
        done_idx[b] = gs.wave_t > 0 ? gs.wave_rows[i] : -1;            // a fresh sequence starts unfinished
        // the row its first logits of this call come from: the parked row, or the row of its (fresh) group
        logit_row[b] = gs.wave_t > 0 ? w.HR + gs.wave_rows[i] : n_fresh;
      } else {
        for (int k = 0; k < per_seq; ++k) tbl[(size_t)b * c->tbl_stride + k] = priv_blocks[(size_t)b * per_seq + k];
        logit_row[b] = g;
      }
      seq_of_row[b] = b;
      seq_ids[b] = (int64_t)groups[g].group_id * G + i;
    }
    if (wave && gs.wave_t == 0) ++n_fresh;
  }
  cudaStream_t st = c->stream;
  CUDA_TRY(cudaMemcpyAsync(w.seqs, sd.data(), (size_t)B * sizeof(SeqDesc), cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(c->d_block_table + (size_t)c->lim.max_groups * c->tbl_stride, tbl.data(), tbl.size() * 4,
                           cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(w.logit_row, logit_row.data(), (size_t)B * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(w.slot_idx, slot_idx.data(), (size_t)n_groups * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(w.row_seq, seq_of_row.data(), (size_t)B * 4, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemcpyAsync(w.seq_ids, seq_ids.data(), (size_t)B * 8, cudaMemcpyHostToDevice, st));
  CUDA_TRY(cudaMemsetAsync(w.done, 0, (size_t)B * 4, st));
  CUDA_TRY(cudaMemsetAsync(w.lens, 0, (size_t)B * 4, st));
  CUDA_TRY(cudaMemsetAsync(w.row_t, 0xFF, (size_t)B * 4, st));
  if (wave) {
    CUDA_TRY(cudaMemcpyAsync(w.t_base, t_base.data(), (size_t)B * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(w.state_idx, state_idx.data(), (size_t)B * 4, cudaMemcpyHostToDevice, st));
    CUDA_TRY(cudaMemcpyAsync(w.done_idx, done_idx.data(), (size_t)B * 4, cudaMemcpyHostToDevice, st));
    // finished flags of the continuing sequences (a negative index yields 0)
    LAUNCH(c, gather_rows_f32_kernel, B, 32, 0, (const float*)c->d_seq_done, (const int32_t*)w.done_idx, (float*)w.done, B, 1);
  }

  {
    int max_p = 1;
    for (int g = 0; g < n_groups; ++g) max_p = std::max(max_p, groups[g].prefix_len);
    const int rep = c->shape.n_q_heads / c->shape.n_kv_heads;
    const int pairs = n_groups * c->shape.n_kv_heads * ceil_div(G * rep, FA_BM);
    // Prefix split: the chunk (a multiple of the key tile) that minimises rounds x (keys per CTA +
    // a fixed per-CTA cost of ~160 keys' worth of set-up and tail), with two CTAs resident per SM;
    // CTAs whose chunk lies beyond a short prefix carry suffix tiles only and are not counted.
    // The tcgen05 kernel takes over when a group's rows of one KV head fit its 64-row tile: one CTA per
    // SM, 128-key tiles, a fixed cost of about 3 tiles (set-up, the pipeline's fill and drain).
    c->attn_dec5 = c->bf16 && c->use_tc_attention && c->use_tc5_decode && c->shape.head_dim == T5_DH && G * rep <= D5_ROWS;
    const int tile = c->attn_dec5 ? T5_BN : FA_BN;
    const double fixed = c->attn_dec5 ? 384.0 : 160.0;
    const int max_splits = c->attn_dec5 ? 24 : 32;
    c->attn_suf_splits = 1;
    const int slots = (c->attn_dec5 ? 1 : 2) * c->sm_count, per_group = pairs / std::max(n_groups, 1);
    double best_cost = 1e30, best_cl_cost = 1e30;
    int best_chunk = std::max(tile, ceil_div(max_p, tile) * tile), best_cl_chunk = best_chunk;
    for (int want = 1; want <= max_splits; ++want) {
      const int chunk = std::max(tile, ceil_div(ceil_div(max_p, want), tile) * tile);
      int64_t ctas = 0;
      for (int g = 0; g < n_groups; ++g) ctas += (int64_t)per_group * ceil_div(std::max(groups[g].prefix_len, 1), chunk);
      const double cost = (double)ceil_div((int)ctas, slots) * (chunk + fixed);
      if (cost < best_cost - 1e-9) { best_cost = cost; best_chunk = chunk; }
      if (cluster_mergeable(ceil_div(max_p, chunk)) && cost < best_cl_cost - 1e-9) { best_cl_cost = cost; best_cl_chunk = chunk; }
    }
    // split counts that merge inside a cluster save the merge kernel: preferred unless clearly costlier
    if (c->use_cluster_merge && !c->attn_dec5 && best_cl_cost <= 1.1 * best_cost) best_chunk = best_cl_chunk;
    c->attn_split_chunk = best_chunk;
    if (ceil_div(max_p, c->attn_split_chunk) > max_splits) c->attn_split_chunk = std::max(tile, ceil_div(ceil_div(max_p, max_splits), tile) * tile);
    c->attn_splits = ceil_div(max_p, c->attn_split_chunk);
    c->attn_mode = 1; c->attn_G = G; c->attn_groups = n_groups;
    // the groups' prefix block ids, dense and padded to splits x chunk: the attention CTA of
    // (group, split) fetches its ids without knowing the group's descriptor
    w.pfx_stride = c->attn_splits * (c->attn_split_chunk / KV_BLOCK);
    if (w.pfx_stride > c->tbl_stride + 512 + 8) return RPO_ERR_LIMIT;
    std::vector<int32_t> pfx((size_t)n_groups * w.pfx_stride, 0);
    for (int g = 0; g < n_groups; ++g) {
      const std::vector<int32_t>& blocks = c->groups[groups[g].slot].blocks;
      const int nb = std::min((int)blocks.size(), ceil_div(groups[g].prefix_len, KV_BLOCK));
      for (int k = 0; k < nb && k < w.pfx_stride; ++k) pfx[(size_t)g * w.pfx_stride + k] = blocks[k];
    }
    CUDA_TRY(cudaMemcpyAsync(w.pfx_tbl, pfx.data(), pfx.size() * 4, cudaMemcpyHostToDevice, st));
  }
  SamplerArgs a = sampler_args(c, sp);
  a.seq_ids = w.seq_ids; a.out_stride = S; a.forced = d_forced; a.tokens_out = d_tokens_out;
  a.logprobs_out = d_logprobs_out; a.done = w.done; a.lens = w.lens; a.cur_tok = w.cur_tok; a.row_t = w.row_t;
  a.logits_dbg = d_logits_dbg; a.logits = w.logits;

  // step 0: the G samples of a group draw from the logits of the group's last prefix token
  CUDA_TRY(cudaMemsetAsync(w.step_ctr, 0, 4, st));
  a.step_ptr = w.step_ctr; a.n_steps = S;
  if (wave) {
    // a fresh group's sequences draw from the logits of its last prefix token, a continuing sequence from the
    // logits parked by its last call; the call's last token is fed too (below), so no step of it is the last one
    a.t_base = w.t_base; a.n_steps = S + 1;
    if (n_fresh > 0) {
      LAUNCH(c, gather_rows_f32_kernel, n_fresh, 128, 0, (const float*)c->d_x_last, (const int32_t*)w.slot_idx, w.xh, n_fresh, d);
      RPO_TRY(head<T>(c, n_fresh));
    }
    a.logit_row = w.logit_row;
    RPO_TRY(launch_sampler(c, B, a));
    a.logit_row = nullptr;
  } else {
    LAUNCH(c, gather_rows_f32_kernel, n_groups, 128, 0, (const float*)c->d_x_last, (const int32_t*)w.slot_idx, w.xh,
           n_groups, d);
    RPO_TRY(head<T>(c, n_groups));
    a.logit_row = w.logit_row;
    RPO_TRY(launch_sampler(c, B, a));
    a.logit_row = nullptr;
  }
  // steps 1..S-1 are one and the same launch sequence (the step number lives on the device):
  // the first runs eagerly, the others replay a CUDA graph of it.
  const bool fused = fused_layers(c, B);
  auto enqueue_step = [&](bool sample = true) -> int {
    const float* e_gain; bf16* e_xg; float* e_ssq;
    embed_norm_args(c, B, e_gain, e_xg, e_ssq);
    LAUNCH(c, embed_kernel<T>, B, 128, 0, (const int32_t*)w.cur_tok, (const T*)c->embed, w.x, B, d, c->shape.vocab,
           c->d_status, w.step_ctr, row_meta_args(c), e_gain, e_xg, e_ssq);
    if (fused && c->shape.n_layers > 0) {
      // the last layer's down projection left bf16(x * final gain) and the rows' sums of squares: the
      // output head scales its rows by 1/rms in its epilogue
      RPO_TRY(run_layers_fused(c, B));
      TcFuse f = fuse_norm_in(c);
      RPO_TRY(gemm_fused(c, (const bf16*)w.h, (const bf16*)c->lm_head, w.logits, B, c->shape.vocab, d, TC_NSTORE_F32, c->shape.vocab, f));
      if (sample) RPO_TRY(launch_sampler(c, B, a));
      return RPO_OK;
    }
    // every row is a sequence's last row: the final RMSNorm reads ws.x directly and folds the last
    // layer's split-K partials in (no separate reduction, no copy of the residual rows)
    RPO_TRY(run_layers<T>(c, B, false));
    RPO_TRY(rmsnorm<T>(c, w.x, c->gf, (T*)w.hh, B));
    RPO_TRY(gemm<T>(c, (const T*)w.hh, (const T*)c->lm_head, w.logits, B, c->shape.vocab, d, EPI_STORE_F32));
    if (sample) RPO_TRY(launch_sampler(c, B, a));
    return RPO_OK;
  };
  int j = 1;
  if (j < S) { RPO_TRY(enqueue_step()); ++j; }
  if (j < S && c->use_graph && !c->profile && !c->tap_buf && S - j >= 2) {
    uint32_t temp_bits; memcpy(&temp_bits, &a.temperature, 4);
    std::vector<uint64_t> key = {(uint64_t)B, (uint64_t)n_groups, (uint64_t)G, (uint64_t)S, (uint64_t)c->attn_splits,
                                 (uint64_t)c->attn_split_chunk, (uint64_t)(uintptr_t)d_forced, (uint64_t)(uintptr_t)d_tokens_out,
                                 (uint64_t)(uintptr_t)d_logprobs_out, (uint64_t)(uintptr_t)d_logits_dbg,
                                 (uint64_t)a.top_p24, (uint64_t)temp_bits,
                                 (uint64_t)a.greedy, (uint64_t)(uint32_t)a.eos_id, a.seed,
                                 (uint64_t)c->use_tcgen05, (uint64_t)c->use_tc_attention, (uint64_t)c->use_pdl,
                                 (uint64_t)c->gemm_bn, (uint64_t)c->gemm_splits, (uint64_t)c->use_gemm_pairs, (uint64_t)c->use_cluster_merge, (uint64_t)c->use_gemm_pairs_small, (uint64_t)c->use_fused_layers,
                                 (uint64_t)c->attn_dec5, (uint64_t)c->attn_suf_splits, (uint64_t)wave};
    rpo_ctx::StepGraph* sg = nullptr;
    for (auto& g : c->step_graphs) if (g.key == key) sg = &g;
    if (!sg) {
      if (c->step_graphs.size() >= 8) {            // drop the oldest; nothing may still be running from it
        CUDA_TRY(cudaStreamSynchronize(st));
        cudaGraphExecDestroy(c->step_graphs.front().exec);
        c->step_graphs.erase(c->step_graphs.begin());
      }
      const int64_t l0 = c->launches;
      cudaGraph_t graph = nullptr;
      CUDA_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
      c->capturing = true;
      const int rc = enqueue_step();
      c->capturing = false;
      const cudaError_t ce = cudaStreamEndCapture(st, &graph);
      const int64_t per_step = c->launches - l0;
      c->launches = l0;
      if (rc != RPO_OK || ce != cudaSuccess || !graph) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return rc != RPO_OK ? rc : RPO_ERR_CUDA; }
      cudaGraphExec_t exec = nullptr;
      const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
      cudaGraphDestroy(graph);
      if (ie != cudaSuccess) { cudaGetLastError(); return RPO_ERR_CUDA; }
      c->step_graphs.push_back({key, exec, per_step});
      sg = &c->step_graphs.back();
    }
    for (; j < S; ++j) { CUDA_TRY(cudaGraphLaunch(sg->exec, st)); c->launches += sg->launches; }
  }
  for (; j < S; ++j) RPO_TRY(enqueue_step());
  CUDA_TRY(cudaMemcpyAsync(d_lens_out, w.lens, (size_t)B * 4, cudaMemcpyDeviceToDevice, st));
  if (wave) {
    // feed the call's last token: its K/V joins the private blocks, and the logits its successor will be drawn from
    // are parked in the sequence's state row together with the finished flag
    RPO_TRY(enqueue_step(false));
    LAUNCH(c, scatter_rows_u32_kernel, B, 256, 0, (const uint32_t*)w.logits, (const int32_t*)w.state_idx,
           (uint32_t*)(w.logits + (size_t)w.HR * c->shape.vocab), B, c->shape.vocab);
    LAUNCH(c, scatter_rows_u32_kernel, B, 32, 0, (const uint32_t*)w.done, (const int32_t*)w.state_idx, (uint32_t*)c->d_seq_done, B, 1);
  }
  return RPO_OK;
}

extern "C" int rpo_decode_suffix(rpo_ctx* c, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                                 const rpo_sampler* sp, const int32_t* d_forced, int32_t* d_tokens_out,
                                 int32_t* d_lens_out, float* d_logprobs_out, float* d_logits_dbg) {
  if (!c || n_groups <= 0 || !h_groups || G <= 0 || max_new <= 0 || !d_tokens_out || !d_lens_out) return RPO_ERR_INVALID_ARG;
  RPO_TRY(check_sampler(sp));
  if (!c->weights_ready) return RPO_ERR_NOT_INITIALISED;
  RPO_TRY(enter(c));
  RPO_TRY(check_groups(c, n_groups, h_groups));
  if ((int64_t)n_groups * G > c->lim.max_seqs) return RPO_ERR_LIMIT;
  for (int g = 0; g < n_groups; ++g)
    if (h_groups[g].prefix_len + max_new > c->lim.max_positions) return RPO_ERR_LIMIT;
  std::vector<int32_t> priv;
  c->prof_phase = 1;
  int rc = c->bf16 ? decode_t<bf16>(c, n_groups, h_groups, G, max_new, sp, d_forced, d_tokens_out, d_lens_out,
                                    d_logprobs_out, d_logits_dbg, priv)
                   : decode_t<float>(c, n_groups, h_groups, G, max_new, sp, d_forced, d_tokens_out, d_lens_out,
                                     d_logprobs_out, d_logits_dbg, priv);
  give_blocks(c, priv);   // stream order protects the blocks until the enqueued work is done
  return rc;
}

extern "C" int rpo_decode_wave(rpo_ctx* c, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                               int32_t max_total, const rpo_sampler* sp, const int32_t* d_forced, int32_t* d_tokens_out,
                               int32_t* d_lens_out, float* d_logprobs_out) {
  if (!c || n_groups <= 0 || !h_groups || G <= 0 || max_new <= 0 || max_total < max_new || !d_tokens_out || !d_lens_out)
    return RPO_ERR_INVALID_ARG;
  RPO_TRY(check_sampler(sp));
  if (!c->weights_ready) return RPO_ERR_NOT_INITIALISED;
  RPO_TRY(enter(c));
  RPO_TRY(check_groups(c, n_groups, h_groups));
  if ((int64_t)n_groups * G > c->lim.max_seqs) return RPO_ERR_LIMIT;
  // first pass: every group must be able to take the wave; nothing is reserved before all of them have been checked
  int64_t need_blocks = 0, need_rows = 0;
  for (int g = 0; g < n_groups; ++g) {
    const GroupState& gs = c->groups[h_groups[g].slot];
    if (gs.wave_G == 0) {
      if (h_groups[g].prefix_len + max_total > c->lim.max_positions) return RPO_ERR_LIMIT;
      need_blocks += (int64_t)G * ceil_div(max_total, KV_BLOCK);
      need_rows += G;
    } else if (gs.wave_G != G || gs.wave_t + max_new > gs.wave_total) {
      return RPO_ERR_LIMIT;                      // another G than the group began with, or past the reserved positions
    }
  }
  if (need_blocks > (int64_t)c->free_blocks.size() || need_rows > (int64_t)c->free_state_rows.size()) return RPO_ERR_KV_POOL;
  for (int g = 0; g < n_groups; ++g) {
    GroupState& gs = c->groups[h_groups[g].slot];
    if (gs.wave_G != 0) continue;
    RPO_TRY(take_blocks(c, G * ceil_div(max_total, KV_BLOCK), gs.wave_blocks));
    for (int i = 0; i < G; ++i) { gs.wave_rows.push_back(c->free_state_rows.back()); c->free_state_rows.pop_back(); }
    gs.wave_G = G; gs.wave_total = max_total; gs.wave_t = 0;
  }
  std::vector<int32_t> none;
  c->prof_phase = 1;
  const int rc = c->bf16 ? decode_t<bf16>(c, n_groups, h_groups, G, max_new, sp, d_forced, d_tokens_out, d_lens_out,
                                          d_logprobs_out, nullptr, none, true)
                         : decode_t<float>(c, n_groups, h_groups, G, max_new, sp, d_forced, d_tokens_out, d_lens_out,
                                           d_logprobs_out, nullptr, none, true);
  if (rc == RPO_OK)
    for (int g = 0; g < n_groups; ++g) c->groups[h_groups[g].slot].wave_t += max_new;
  return rc;
}

// ---------------------------------------------------------------------------------------------
// teacher-forced token log-probabilities
// ---------------------------------------------------------------------------------------------
template <typename T>
static int logprobs_t(rpo_ctx* c, int n_groups, const rpo_group* groups, int G, int S, const int32_t* d_tokens,
                      const int32_t* d_lens, float inv_T, float* d_out, float* d_logits_dbg) {
  Workspace& w = c->ws;
  const int B = n_groups * G, d = c->shape.d_model, V = c->shape.vocab;
  const int in_rows = std::max(S - 1, 1);                       // layer-stack rows per sequence
  const int seq_per_chunk = std::min(std::min(c->lim.max_chunk_tokens / in_rows, c->lim.max_seqs), B);
  if (seq_per_chunk < 1) return RPO_ERR_LIMIT;
  const int per_seq = ceil_div(std::max(S - 1, 0), KV_BLOCK);
  cudaStream_t st = c->stream;
  for (int s0 = 0; s0 < B; s0 += seq_per_chunk) {
    const int ns = std::min(seq_per_chunk, B - s0);
    std::vector<int32_t> priv;
    RPO_TRY(take_blocks(c, ns * per_seq, priv));
    std::vector<SeqDesc> sd(ns);
    std::vector<int32_t> tbl((size_t)ns * c->tbl_stride, -1), slot_of_seq(ns);
    for (int i = 0; i < ns; ++i) {
      const rpo_group& g = groups[(s0 + i) / G];
      sd[i].shared_tbl = g.slot * c->tbl_stride; sd[i].shared_len = g.prefix_len;
      sd[i].priv_tbl = (c->lim.max_groups + i) * c->tbl_stride; sd[i].reserved = 0;
      for (int k = 0; k < per_seq; ++k) tbl[(size_t)i * c->tbl_stride + k] = priv[(size_t)i * per_seq + k];
      slot_of_seq[i] = g.slot;
    }
    int rc = RPO_OK;
    do {
      if (cudaMemcpyAsync(w.seqs, sd.data(), (size_t)ns * sizeof(SeqDesc), cudaMemcpyHostToDevice, st) != cudaSuccess ||
          cudaMemcpyAsync(c->d_block_table + (size_t)c->lim.max_groups * c->tbl_stride, tbl.data(), tbl.size() * 4,
                          cudaMemcpyHostToDevice, st) != cudaSuccess ||
          cudaMemcpyAsync(w.slot_idx, slot_of_seq.data(), (size_t)ns * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        rc = RPO_ERR_CUDA; break;
      }
      const int rows = ns * (S - 1);
      if (rows > 0) {
        if ((rc = upload_row_tiles(c, std::vector<int>(ns, S - 1))) != RPO_OK) break;
        build_teacher_rows_kernel<<<grid_for(rows, 256), 256, 0, st>>>(d_tokens, d_lens, s0, ns, S, w.row_seq, w.row_t,
                                                                      w.row_tok);
        c->launches++;
        const float* e_gain; bf16* e_xg; float* e_ssq;
        embed_norm_args(c, rows, e_gain, e_xg, e_ssq);
        embed_kernel<T><<<rows, 128, 0, st>>>((const int32_t*)w.row_tok, (const T*)c->embed, w.x, rows, d, V, c->d_status, nullptr,
                                              row_meta_args(c), e_gain, e_xg, e_ssq);
        c->launches++;
        if ((rc = run_layers<T>(c, rows)) != RPO_OK) break;
      }
      const int head_rows = ns * S;
      for (int r0 = 0; r0 < head_rows && rc == RPO_OK; r0 += w.HR) {
        const int nr = std::min(w.HR, head_rows - r0);
        gather_head_rows_kernel<<<nr, 128, 0, st>>>(w.x, c->d_x_last, w.slot_idx, r0, nr, S, d, w.xh);
        c->launches++;
        if (!d_logits_dbg && fused_layers(c, 1 << 20) && (c->use_fused_lse == 2 || (c->use_fused_lse && tc2_wanted(c, nr, V, d, false)))) {
          // the output head keeps, per row and column unit, the running maximum, the sum of exponentials and the
          // target's logit: the [nr, V] logits never reach memory
          lse_targets_kernel<<<ceil_div(nr, 256), 256, 0, st>>>(r0, nr, V, S, d_tokens, d_lens, s0, w.lse_target);
          c->launches++;
          {
            ProfScope ps(c, KC_NORM);
            LAUNCH(c, norm_prep_kernel, nr, 128, 0, (const float*)w.xh, (const float*)c->gf, (bf16*)w.hh, w.ssq_h, nr, d);
          }
          TcFuse f;
          f.ssq_in = w.ssq_h; f.ssq_in_parts = 1; f.norm_dim = d; f.eps = c->shape.rms_eps;
          f.lse_parts = (float2*)w.lse_parts; f.lse_tgt = w.lse_tgt; f.lse_target = w.lse_target; f.lse_inv_T = inv_T;
          if ((rc = gemm_fused(c, (const bf16*)w.hh, (const bf16*)c->lm_head, nullptr, nr, V, d, TC_NLSE, V, f)) != RPO_OK) break;
          lse_merge_rows_kernel<<<ceil_div(nr, 8), 256, 0, st>>>((const float2*)w.lse_parts, f.ssq_out_parts, w.lse_tgt, w.lse_target,
                                                                 r0, nr, S, s0, d_out);
          c->launches++;
          continue;
        }
        if ((rc = head<T>(c, nr)) != RPO_OK) break;
        logprob_rows_kernel<<<nr, 512, 0, st>>>(w.logits, r0, nr, V, S, d_tokens, d_lens, s0, inv_T, d_out, d_logits_dbg);
        c->launches++;
      }
      if (rc == RPO_OK && cudaGetLastError() != cudaSuccess) rc = RPO_ERR_CUDA;
    } while (0);
    give_blocks(c, priv);
    if (rc != RPO_OK) return rc;
  }
  return RPO_OK;
}

extern "C" int rpo_token_logprobs(rpo_ctx* c, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                                  const int32_t* d_tokens, const int32_t* d_lens, float inv_temperature,
                                  float* d_logprobs_out, float* d_logits_dbg) {
  if (!c || n_groups <= 0 || !h_groups || G <= 0 || max_new <= 0 || !d_tokens || !d_lens || !d_logprobs_out ||
      !(inv_temperature > 0.f))
    return RPO_ERR_INVALID_ARG;
  if (!c->weights_ready) return RPO_ERR_NOT_INITIALISED;
  RPO_TRY(enter(c));
  RPO_TRY(check_groups(c, n_groups, h_groups));
  for (int g = 0; g < n_groups; ++g)
    if (h_groups[g].prefix_len + max_new > c->lim.max_positions) return RPO_ERR_LIMIT;
  c->prof_phase = 2;
  return c->bf16 ? logprobs_t<bf16>(c, n_groups, h_groups, G, max_new, d_tokens, d_lens, inv_temperature,
                                    d_logprobs_out, d_logits_dbg)
                 : logprobs_t<float>(c, n_groups, h_groups, G, max_new, d_tokens, d_lens, inv_temperature,
                                     d_logprobs_out, d_logits_dbg);
}

// ---------------------------------------------------------------------------------------------
// objective forward (Eq. 5-7, Eq. 11)
// ---------------------------------------------------------------------------------------------
extern "C" int rpo_policy_objective(rpo_ctx* c, int32_t n_groups, int32_t G, int32_t max_new, const float* d_logp_new,
                                    const float* d_logp_old, const float* d_logp_ref, const int32_t* d_lens,
                                    const int32_t* d_resp_lens, const float* d_raw_rewards, const rpo_objective_cfg* cfg,
                                    float* d_rewards_out, float* d_advantages_out, float* d_token_loss_out,
                                    float* d_group_objective_out, float* d_objective_out) {
  if (!c || n_groups <= 0 || G <= 0 || max_new <= 0 || !d_logp_new || !d_logp_old || !d_lens || !d_raw_rewards || !cfg ||
      !d_rewards_out || !d_advantages_out || !d_group_objective_out || !d_objective_out)
    return RPO_ERR_INVALID_ARG;
  if (G > OBJ_MAX_G) return RPO_ERR_LIMIT;
  if (!(cfg->clip_eps >= 0.f) || !(cfg->reward_max >= cfg->reward_min)) return RPO_ERR_INVALID_ARG;
  ObjectiveArgs a;
  memset(&a, 0, sizeof(a));
  a.logp_new = d_logp_new; a.logp_old = d_logp_old; a.logp_ref = d_logp_ref; a.lens = d_lens; a.resp_lens = d_resp_lens;
  a.raw_rewards = d_raw_rewards; a.G = G; a.S = max_new; a.clip_eps = cfg->clip_eps; a.beta = cfg->beta; a.alpha = cfg->alpha;
  a.r_min = cfg->reward_min; a.r_max = cfg->reward_max; a.length_shaping = cfg->length_shaping;
  a.rewards_out = d_rewards_out; a.adv_out = d_advantages_out; a.token_loss_out = d_token_loss_out;
  a.group_obj_out = d_group_objective_out;
  const int threads = std::max(64, std::min(1024, G * 32));
  LAUNCH(c, objective_group_kernel, n_groups, threads, 0, a);
  LAUNCH(c, objective_reduce_kernel, 1, 32, 0, (const float*)d_group_objective_out, n_groups, d_objective_out);
  return RPO_OK;
}

// ---------------------------------------------------------------------------------------------
// whole rollout with host buffers
// ---------------------------------------------------------------------------------------------
extern "C" int rpo_rollout_host(rpo_ctx* c, int32_t n_groups, const int32_t* h_tokens, const int32_t* h_offsets,
                                const int32_t* h_group_ids, int32_t G, int32_t max_new, const rpo_sampler* sp,
                                int32_t* h_tokens_out, int32_t* h_lens_out, float* h_logprobs_out,
                                int32_t want_policy, float* h_policy_out) {
  if (!c || n_groups <= 0 || !h_tokens || !h_offsets || G <= 0 || max_new <= 0 || !h_tokens_out || !h_lens_out ||
      (want_policy && !h_policy_out))
    return RPO_ERR_INVALID_ARG;
  RPO_TRY(check_sampler(sp));
  const size_t n_tok = (size_t)h_offsets[n_groups], B = (size_t)n_groups * G, BS = B * max_new;
  int32_t *d_tok = nullptr, *d_out = nullptr, *d_lens = nullptr;
  float *d_lp = nullptr, *d_pol = nullptr;
  std::vector<rpo_group> groups(n_groups);
  int rc = RPO_OK;
  bool prefilled = false;
  auto stage = [&](int slot, size_t bytes) -> void* {      // persistent device buffer of at least `bytes`
    if (c->host_stage_bytes[slot] < bytes) {
      cudaStreamSynchronize(c->stream);
      if (c->host_stage[slot]) cudaFree(c->host_stage[slot]);
      c->host_stage[slot] = nullptr; c->host_stage_bytes[slot] = 0;
      if (cudaMalloc(&c->host_stage[slot], bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
      c->host_stage_bytes[slot] = bytes;
    }
    return c->host_stage[slot];
  };
  do {
    d_tok = (int32_t*)stage(0, std::max<size_t>(n_tok, 1) * 4); d_out = (int32_t*)stage(1, BS * 4);
    d_lens = (int32_t*)stage(2, B * 4); d_lp = (float*)stage(3, BS * 4);
    if (want_policy) d_pol = (float*)stage(4, BS * 4);
    if (!d_tok || !d_out || !d_lens || !d_lp || (want_policy && !d_pol)) { rc = RPO_ERR_CUDA; break; }
    if (cudaMemcpyAsync(d_tok, h_tokens, n_tok * 4, cudaMemcpyHostToDevice, c->stream) != cudaSuccess) { rc = RPO_ERR_CUDA; break; }
    if ((rc = rpo_prefill_prefix(c, n_groups, d_tok, h_offsets, h_group_ids, groups.data())) != RPO_OK) break;
    prefilled = true;
    if ((rc = rpo_decode_suffix(c, n_groups, groups.data(), G, max_new, sp, nullptr, d_out, d_lens, d_lp, nullptr)) != RPO_OK) break;
    if (want_policy &&
        (rc = rpo_token_logprobs(c, n_groups, groups.data(), G, max_new, d_out, d_lens, 1.0f / sp->temperature, d_pol,
                                 nullptr)) != RPO_OK) break;
    cudaMemcpyAsync(h_tokens_out, d_out, BS * 4, cudaMemcpyDeviceToHost, c->stream);
    cudaMemcpyAsync(h_lens_out, d_lens, B * 4, cudaMemcpyDeviceToHost, c->stream);
    if (h_logprobs_out) cudaMemcpyAsync(h_logprobs_out, d_lp, BS * 4, cudaMemcpyDeviceToHost, c->stream);
    if (want_policy) cudaMemcpyAsync(h_policy_out, d_pol, BS * 4, cudaMemcpyDeviceToHost, c->stream);
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) { rc = RPO_ERR_CUDA; break; }
    // the call has synchronised anyway: an expired device-side wait or a bad block index means the
    // results are not to be trusted
    int word = 0;
    if ((rc = read_status(c, &word)) != RPO_OK) break;
    if (word & STATUS_TIMEOUT) rc = RPO_ERR_DEVICE_TIMEOUT;
    else if (word & STATUS_BAD_BLOCK) rc = RPO_ERR_CUDA;
  } while (0);
  if (rc != RPO_OK) { cudaStreamSynchronize(c->stream); cudaGetLastError(); }
  if (prefilled) rpo_release_groups(c, n_groups, groups.data());
  return rc;
}

// ---------------------------------------------------------------------------------------------
// test / introspection entry points
// ---------------------------------------------------------------------------------------------
extern "C" int rpo_sample_rows(rpo_ctx* c, int32_t n_rows, int32_t vocab, const float* d_logits, const rpo_sampler* sp,
                               const int64_t* d_seq_ids, int32_t step, int32_t* d_tokens_out, float* d_logprobs_out) {
  if (!c || n_rows < 0 || vocab <= 0 || vocab >= (1 << 18) || !d_logits || !d_seq_ids || !d_tokens_out || step < 0) return RPO_ERR_INVALID_ARG;
  RPO_TRY(check_sampler(sp));
  if (n_rows == 0) return RPO_OK;
  SamplerArgs a = sampler_args(c, sp);
  a.V = vocab; a.logits = d_logits; a.seq_ids = d_seq_ids; a.step = step; a.out_stride = 1; a.out_col = 0;
  a.tokens_out = d_tokens_out; a.logprobs_out = d_logprobs_out; a.eos_id = -1;
  // This test entry takes any vocabulary: its weight scratch is a stream-ordered temporary.
  void* tmp = nullptr;
  CUDA_TRY(cudaMallocAsync(&tmp, (size_t)n_rows * vocab * 4, c->stream));
  a.weights = (uint32_t*)tmp;
  const int rc = launch_sampler(c, n_rows, a);
  CUDA_TRY(cudaFreeAsync(tmp, c->stream));
  return rc;
}

extern "C" int rpo_gemm(rpo_ctx* c, int32_t impl, int32_t M, int32_t N, int32_t K, const void* d_A, const void* d_W,
                        float* d_C) {
  if (!c || M < 0 || N <= 0 || K <= 0 || !d_A || !d_W || !d_C || impl < 0 || impl > 2) return RPO_ERR_INVALID_ARG;
  int splits = 0;
  RPO_TRY(c->bf16 ? gemm<bf16>(c, (const bf16*)d_A, (const bf16*)d_W, d_C, M, N, K, EPI_STORE_F32, impl, true, &splits)
                  : gemm<float>(c, (const float*)d_A, (const float*)d_W, d_C, M, N, K, EPI_STORE_F32, impl));
  if (splits > 1) {                       // the planner (or its override) split K: reduce the planes into C
    const int64_t n = (int64_t)M * N;     // N % 16 == 0 on this path
    CUDA_TRY(cudaMemsetAsync(d_C, 0, (size_t)n * 4, c->stream));
    LAUNCH(c, reduce_partials_kernel, grid_for(n / 4, 256), 256, 0, d_C, (const float*)c->ws.partial, splits, n, n);
  }
  return RPO_OK;
}

extern "C" int rpo_gemm_bench(rpo_ctx* c, int32_t M, int32_t N, int32_t K, const void* d_A, const void* const* h_W_list,
                              int32_t n_w, int32_t iters, float* h_ms_out) {
  if (!c || !c->bf16 || M <= 0 || N <= 0 || K <= 0 || !d_A || !h_W_list || n_w <= 0 || iters <= 0 || !h_ms_out)
    return RPO_ERR_INVALID_ARG;
  if (!tc_gemm_supported<bf16>(c, M, N, K)) return RPO_ERR_SHAPE;
  if ((size_t)M * N > (size_t)c->ws.HR * c->shape.vocab) return RPO_ERR_LIMIT;   // output lands in ws.logits
  cudaStream_t st = c->stream;
  auto enqueue = [&]() -> int {
    for (int i = 0; i < iters; ++i) {
      int splits = 0;
      if (tc2_wanted(c, M, N, K, true))
        RPO_TRY(tc2_gemm_launch(c, (const bf16*)d_A, (const bf16*)h_W_list[i % n_w], c->ws.logits, M, N, K, TC_STORE_F32, N,
                                true, &splits));
      else
        RPO_TRY(tc_gemm_launch(c, (const bf16*)d_A, (const bf16*)h_W_list[i % n_w], c->ws.logits, M, N, K, TC_STORE_F32, N,
                               true, &splits));
    }
    return RPO_OK;
  };
  RPO_TRY(enqueue());                                   // warm-up: attributes, tensor maps
  cudaGraph_t graph = nullptr; cudaGraphExec_t exec = nullptr;
  CUDA_TRY(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
  const int rc = enqueue();
  const cudaError_t ce = cudaStreamEndCapture(st, &graph);
  if (rc != RPO_OK || ce != cudaSuccess) { if (graph) cudaGraphDestroy(graph); cudaGetLastError(); return rc != RPO_OK ? rc : RPO_ERR_CUDA; }
  const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
  cudaGraphDestroy(graph);
  if (ie != cudaSuccess) { cudaGetLastError(); return RPO_ERR_CUDA; }
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0); cudaEventCreate(&e1);
  cudaGraphLaunch(exec, st);
  cudaEventRecord(e0, st);
  cudaGraphLaunch(exec, st);
  cudaEventRecord(e1, st);
  const cudaError_t se = cudaStreamSynchronize(st);
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0); cudaEventDestroy(e1); cudaGraphExecDestroy(exec);
  if (se != cudaSuccess) return RPO_ERR_CUDA;
  *h_ms_out = ms / iters;
  return RPO_OK;
}

// Reads and clears the device status word (synchronises the stream).  After an expired wait the
// arrival counters of the split-K launches may be left half-counted: they are cleared too.
static int read_status(rpo_ctx* c, int* word) {
  int v = 0;
  CUDA_TRY(cudaMemcpyAsync(&v, c->d_status, 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  if (v) {
    CUDA_TRY(cudaMemsetAsync(c->d_status, 0, 4, c->stream));
    if (v & STATUS_TIMEOUT) CUDA_TRY(cudaMemsetAsync(c->ws.tile_ctr, 0, (size_t)TC_CTR_CAPACITY * 4, c->stream));
  }
  *word = v;
  return RPO_OK;
}

extern "C" int rpo_device_status(rpo_ctx* c, int32_t* out) {
  if (!c || !out) return RPO_ERR_INVALID_ARG;
  int v = 0;
  RPO_TRY(read_status(c, &v));
  *out = v;
  return (v & STATUS_TIMEOUT) ? RPO_ERR_DEVICE_TIMEOUT : RPO_OK;
}

extern "C" int rpo_debug_tap(rpo_ctx* c, float* d_buf, int64_t capacity_floats, int64_t* h_used_out) {
  if (!c || capacity_floats < 0 || (d_buf && capacity_floats == 0)) return RPO_ERR_INVALID_ARG;
  if (h_used_out) *h_used_out = c->tap_used;
  c->tap_buf = d_buf; c->tap_capacity = d_buf ? capacity_floats : 0; c->tap_used = 0;
  return RPO_OK;
}

extern "C" int rpo_counters(rpo_ctx* c, int64_t* launches, int64_t* free_blocks) {
  if (!c) return RPO_ERR_INVALID_ARG;
  if (launches) *launches = c->launches;
  if (free_blocks) *free_blocks = (int64_t)c->free_blocks.size();
  return RPO_OK;
}

extern "C" int rpo_set_option(rpo_ctx* c, const char* name, int32_t value) {
  if (!c || !name) return RPO_ERR_INVALID_ARG;
  if (!strcmp(name, "use_tcgen05")) c->use_tcgen05 = value;
  else if (!strcmp(name, "use_tc_attention")) c->use_tc_attention = value;
  else if (!strcmp(name, "use_graph")) c->use_graph = value;
  else if (!strcmp(name, "use_pdl")) c->use_pdl = value;
  else if (!strcmp(name, "use_fused_layers")) c->use_fused_layers = value;
  else if (!strcmp(name, "wait_limit_cycles")) {        // <= 0: the default; applies to the whole device (see gemm_tc.cuh)
    const long long lim = value > 0 ? (long long)value : TC_TIMEOUT_CYCLES_DEFAULT;
    CUDA_TRY(cudaMemcpyToSymbolAsync(g_wait_limit_cycles, &lim, sizeof(lim), 0, cudaMemcpyHostToDevice, c->stream));
    CUDA_TRY(cudaStreamSynchronize(c->stream));
  }
  else if (!strcmp(name, "fused_split_limit")) c->fused_split_limit = value;
  else if (!strcmp(name, "use_tc5_attention")) c->use_tc5_attention = value;
  else if (!strcmp(name, "use_fused_lse")) c->use_fused_lse = value;
  else if (!strcmp(name, "use_tc5_pipelined")) c->use_tc5_pipelined = value;
  else if (!strcmp(name, "use_tc5_decode")) c->use_tc5_decode = value;
  else if (!strcmp(name, "use_gemm_pairs")) c->use_gemm_pairs = value;
  else if (!strcmp(name, "use_cluster_merge")) c->use_cluster_merge = value;
  else if (!strcmp(name, "use_gemm_pairs_small")) c->use_gemm_pairs_small = value;
  else if (!strcmp(name, "gemm_bn")) { if (value != 0 && value != 32 && value != 64 && value != 96 && value != 128 && value != 256 && value != 384 && value != 512) return RPO_ERR_INVALID_ARG; c->gemm_bn = value; }
  else if (!strcmp(name, "gemm_splits")) c->gemm_splits = value;
  else if (!strcmp(name, "profile")) c->profile = value;
  else return RPO_ERR_INVALID_ARG;
  return RPO_OK;
}

extern "C" int rpo_profile_read(rpo_ctx* c, double* ms_out, int64_t* count_out, int32_t n) {
  if (!c || !ms_out || !count_out || n < 3 * KC_COUNT) return RPO_ERR_INVALID_ARG;
  CUDA_TRY(cudaStreamSynchronize(c->stream));
  for (int i = 0; i < n; ++i) { ms_out[i] = 0.0; count_out[i] = 0; }
  std::map<std::string, std::pair<double, int64_t>> by_label;   // option profile = 2: table on stderr
  for (auto& ev : c->prof_events) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, ev.a, ev.b);
    if (c->profile >= 2) {
      static const char* ph[] = {"prefill", "decode", "logprobs", "?"};
      auto& e = by_label[std::string(ph[std::min(ev.tag / 16, 3)]) + " " + ev.label];
      e.first += ms; e.second++;
    }
    const int phase = ev.tag / 16, k = ev.tag % 16;
    if (phase < 3 && k < KC_COUNT) { ms_out[phase * KC_COUNT + k] += ms; count_out[phase * KC_COUNT + k]++; }
    cudaEventDestroy(ev.a); cudaEventDestroy(ev.b);
  }
  c->prof_events.clear();
  for (auto& kv : by_label)
    fprintf(stderr, "[rpo profile] %-60s %8lld launches %10.3f ms  %8.2f us/launch\n", kv.first.c_str(),
            (long long)kv.second.second, kv.second.first, 1e3 * kv.second.first / kv.second.second);
  return RPO_OK;
}

// ---------------------------------------------------------------------------------------------
// sampling without any allocation
// ---------------------------------------------------------------------------------------------
// The sampler parks one 32-bit weight per (row, token) in scratch memory.  rpo_sample_rows takes
// that scratch from the stream-ordered allocator; this variant keeps a fixed array inside the
// library image instead, so it needs neither a context nor an allocator.
#define RPO_NOALLOC_SAMPLER_WORDS (4u << 20)     /* 4 Mi words = 16 MiB, held by every GPU that loads the library */
static __device__ __align__(256) uint32_t g_noalloc_sampler_scratch[RPO_NOALLOC_SAMPLER_WORDS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
uint32_t* g_noalloc_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
}  // namespace

extern "C" int rpo_sample_rows_noalloc(int32_t n_rows, int32_t vocab, const float* d_logits, const rpo_sampler* sp,
                                       const int64_t* d_seq_ids, int32_t step, int32_t* d_tokens_out,
                                       float* d_logprobs_out, void* cuda_stream) {
  if (n_rows < 0 || vocab <= 0 || vocab >= (1 << 18) || !d_logits || !d_seq_ids || !d_tokens_out || step < 0)
    return RPO_ERR_INVALID_ARG;
  RPO_TRY(check_sampler(sp));
  if ((uint64_t)n_rows * (uint64_t)vocab > (uint64_t)RPO_NOALLOC_SAMPLER_WORDS) {
    fprintf(stderr, "[rpo] rpo_sample_rows_noalloc: %d rows x %d tokens = %llu words exceed the built-in scratch of %u words\n",
            n_rows, vocab, (unsigned long long)n_rows * (unsigned long long)vocab, RPO_NOALLOC_SAMPLER_WORDS);
    return RPO_ERR_LIMIT;
  }
  if (n_rows == 0) return RPO_OK;
  int dev = -1;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return RPO_ERR_LIMIT;
  uint32_t* scratch = nullptr;
  {
    // Set-up, once per device, with that device current.  In host code the array's name is only
    // a handle: the address a kernel may use has to be asked for.
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_scratch_ptr[dev]) {
      uint32_t* ptr = nullptr;
      CUDA_TRY(cudaGetSymbolAddress((void**)&ptr, g_noalloc_sampler_scratch));
      CUDA_TRY(cudaFuncSetAttribute(sampler_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SAMPLER_SMEM));
      g_noalloc_scratch_ptr[dev] = ptr;
    }
    scratch = g_noalloc_scratch_ptr[dev];
  }
  SamplerArgs a;
  memset(&a, 0, sizeof(a));
  a.V = vocab; a.logits = d_logits; a.weights = scratch;
  a.temperature = sp->temperature;
  a.top_p24 = (uint32_t)floorf(sp->top_p * 16777216.0f);
  a.greedy = sp->greedy; a.eos_id = -1; a.seed = sp->seed;
  a.seq_ids = d_seq_ids; a.step = step; a.out_stride = 1; a.out_col = 0;
  a.tokens_out = d_tokens_out; a.logprobs_out = d_logprobs_out;
  sampler_kernel<<<n_rows, 1024, SAMPLER_SMEM, (cudaStream_t)cuda_stream>>>(a);
  CUDA_TRY(cudaGetLastError());
  return RPO_OK;
}
