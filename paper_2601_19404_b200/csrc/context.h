// Host-side state of one rollout context.
#pragma once
#include <cuda_runtime.h>
#include <map>
#include <string>
#include <vector>

#include "../../include/rpo.h"

namespace rpo {

struct TensorInfo {
  void* ptr = nullptr;     // physical base
  int rows = 0, cols = 0;  // logical [out, in]
  int row_mul = 1;         // logical row r lives at physical row r*row_mul + row_add of `ptr`
  int row_add = 0;
  bool gain = false;       // float32 vector
  uint32_t tensor_id = 0;
};

struct LayerWeights {
  void *wqkv, *wo, *wgu, *wd;  // fused [q|k|v] rows; gate/up rows interleaved
  float *g1, *g2;
};

struct GroupState {
  bool live = false;
  int32_t group_id = 0, prefix_len = 0;
  std::vector<int32_t> blocks;
  // a decode that proceeds in waves (rpo_decode_wave): the private suffix blocks and the state rows of the group's
  // sequences stay with the group between calls
  int wave_G = 0, wave_total = 0, wave_t = 0;      // sequences, reserved suffix positions, positions generated so far
  std::vector<int32_t> wave_blocks;                // wave_G x ceil(wave_total / 16) private blocks
  std::vector<int32_t> wave_rows;                  // wave_G rows of the sequence-state pool
};

struct Workspace {
  float* x = nullptr;      // [R, d] residual stream
  void* h = nullptr;       // [R, d]
  void* qkv = nullptr;     // [R, (Hq+2Hkv)*dh]
  void* attn = nullptr;    // [R, Hq*dh]
  void* gu = nullptr;      // [R, 2F]
  void* act = nullptr;     // [R, F]
  float* xh = nullptr;     // [HR, d] head input rows
  void* hh = nullptr;      // [HR, d]
  float* logits = nullptr; // [HR + max_seqs, V]: HR work rows, then the rows parked by a decode in waves
  uint32_t* sampler_w = nullptr;  // [max(max_seqs, max_groups), V] quantised sampler weights
  size_t sampler_w_rows = 0;
  float* ssq = nullptr;          // [R][ssq_stride] partial sums of squares of the residual rows (fused RMSNorm)
  int ssq_stride = 0;
  float* ssq_h = nullptr;        // [HR] the same for the rows that go into the output head
  int* tile_ctr = nullptr;       // split-K arrival counters (zero between launches)
  float* partial = nullptr;      // split-K partial sums
  size_t partial_elems = 0;
  float* attn_part = nullptr;    // decode attention partials
  size_t attn_part_elems = 0;
  void* tiles = nullptr;   // int2 (first row, rows) per 64-row attention tile
  int32_t *row_seq = nullptr, *row_t = nullptr, *row_tok = nullptr;
  int32_t* pfx_tbl = nullptr;          // decode call: the groups' prefix block ids, dense [group][pfx_stride]
  int pfx_stride = 0;
  int4* row_meta = nullptr;            // per row of the pass: (position, private KV block, slot in block, -) or x < 0: inactive
  void* seqs = nullptr;    // SeqDesc[]
  int32_t *done = nullptr, *lens = nullptr, *cur_tok = nullptr, *logit_row = nullptr, *slot_idx = nullptr;
  int32_t *t_base = nullptr, *state_idx = nullptr;      // resumed decode: positions generated before the call; state row per sequence
  void* lse_parts = nullptr;                            // float2 [HR][2 ceil(V / 256)]: the output head's per-unit (max, sum of exponentials)
  float* lse_tgt = nullptr; int32_t* lse_target = nullptr;   // [HR]
  int32_t *done_idx = nullptr;                          // resumed decode: where the finished flags are read from (-1: fresh)
  int32_t* step_ctr = nullptr;   // device counter of the decode step being computed
  int64_t* seq_ids = nullptr;
  int R = 0, HR = 0;
};

}  // namespace rpo

struct rpo_ctx {
  rpo_shape shape;
  rpo_limits lim;
  cudaStream_t stream = nullptr;
  bool own_stream = false;   // created by rpo_create because the caller passed NULL
  bool bf16 = false;
  size_t esz = 4;
  int qkv_cols = 0;
  // weights
  std::vector<void*> allocations;
  std::map<std::string, rpo::TensorInfo> tensors;
  std::vector<rpo::LayerWeights> layers;
  void *embed = nullptr, *lm_head = nullptr;
  float* gf = nullptr;
  bool weights_ready = false;
  // paged KV
  void* kv_base = nullptr;
  int64_t kv_layer_stride = 0, kv_kv_stride = 0, kv_head_stride = 0;
  std::vector<int32_t> free_blocks;
  int32_t* d_block_table = nullptr;
  int tbl_stride = 0;
  std::vector<int32_t> free_slots;
  std::vector<rpo::GroupState> groups;
  float* d_x_last = nullptr;   // [max_groups, d]
  int32_t* d_seq_done = nullptr;           // [max_seqs] finished flag per state row (decode in waves)
  std::vector<int32_t> free_state_rows;
  void* d_rope = nullptr;      // float2 [max_positions, dh/2]
  rpo::Workspace ws;
  int* d_status = nullptr;
  int64_t launches = 0;
  int sm_count = 148;
  int device = 0;                     // the CUDA device this context lives on
  int ssq_parts = 1;                  // parts per row currently in ws.ssq (set by the kernel that wrote them)
  // options
  int fused_split_limit = 1;          // ... for passes none of whose products splits K (more planes allowed: tests, sweeps)
  int use_fused_layers = 1;           // 16-bit models: RMSNorm / RoPE / KV append / SwiGLU / residual as GEMM epilogues
  int use_tcgen05 = 1, use_tc_attention = 1, use_graph = 1;
  int use_tc5_attention = 1;          // tcgen05 attention for many-row passes
  int use_tc5_pipelined = 0;          //   its pipelined variant (64-key tiles, running output in tensor memory)
  int use_fused_lse = 1;              // token log-probs: the output head keeps (max, sum exp, target) per tile instead of writing logits
  int use_tc5_decode = 0;             // tcgen05 decode attention (head_dim 128, <= 64 rows per group and KV head): parity-green, but
                                      // measured 5-25 % slower per launch than the mma.sync kernel (1.8 us per 64-key tile): off by default
  bool attn_dec5 = false;             // plan of the decode call being enqueued: prefix on tcgen05, suffix tiles in a pass of their own
  int attn_suf_splits = 1;
  int use_cluster_merge = 0;          // decode attention: splits of a work item merge inside a thread-block cluster
                                      // (measured slower than partials + merge kernel at 8 splits: off by default)
  int launch_cluster_x = 0;           // cluster width of the next launch (0: none); cleared by the launch
  int use_pdl = 1;                    // programmatic dependent launch between the library's kernels: 0 off, 1 inside the
                                      // captured decode-step graphs and in the many-row passes (prefill, log-probs), 2 on
                                      // every launch (also the eagerly launched parts of a decode call)
  bool capturing = false;             // a decode-step graph is being captured
  bool pdl_now() const { return use_pdl == 2 || (use_pdl == 1 && (capturing || prof_phase != 1)); }
  int use_gemm_pairs = 1;             // 256 x 256 tiles on CTA pairs (cta_group::2) for many-row GEMMs
  int use_gemm_pairs_small = 1;       // pair tiles with 64 rows per CTA for wide matrices at up to 128 rows
  int gemm_bn = 0, gemm_splits = 0;   // > 0: override the GEMM planner (tests, sweeps); 384 / 512 = pair tiles with 64 / 128 rows per CTA
  // attention plan of the pass being enqueued: 0 = row tiles (prefill / teacher), 1 = decode
  int attn_mode = 0, attn_tiles = 0, attn_G = 1, attn_groups = 0, attn_splits = 1, attn_split_chunk = 64;
  // device staging of rpo_rollout_host: kept between calls (stable addresses let the decode step's
  // CUDA graph be reused), grown on demand, freed with the context
  void* host_stage[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  size_t host_stage_bytes[5] = {0, 0, 0, 0, 0};
  int pending_splits = 0, pending_rows = 0;   // split-K partials of ws.x not yet reduced
  // test tap (rpo_debug_tap): residual rows entering the layer stack and leaving every layer
  float* tap_buf = nullptr;
  int64_t tap_capacity = 0, tap_used = 0;
  // optional per-kernel timing: event pairs around every launch, tagged class + 16*phase
  struct ProfEvent { cudaEvent_t a, b; int tag; const char* label; };
  int profile = 0, prof_class = 0, prof_phase = 0;
  std::vector<ProfEvent> prof_events;
  // instantiated CUDA graphs of one decode step, keyed by everything the step's launches depend on
  struct StepGraph { std::vector<uint64_t> key; cudaGraphExec_t exec; int64_t launches; };
  std::vector<StepGraph> step_graphs;
  // tcgen05 GEMM state (tensor maps are built per call; see gemm_tc.cuh)
  void* tc_state = nullptr;
};
