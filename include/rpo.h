/*
 * rpo.h -- C ABI of the B200 rollout library for RPO (Reinforcement Fine-Tuning with
 * Partial Reasoning Optimization).
 *
 * The library implements the rollout stage of the method: for every question q_k the
 * cached response a_k is truncated and the policy generates G continuations of the
 * prefix (Section 3.2 "Rollout", Eq. 3; Algorithm 1, inner loop over g = 1..G), and the
 * per-token probabilities pi_theta(o_{i,j} | q, o_{i,<j}) that the probability ratio
 * r_{i,j} of Eq. 7 is built from.  The caller hands over token arrays only: the prefix
 * is the already concatenated string q_k || a_k^{[0:-m]}.
 *
 * Conventions
 *  - Every function returns RPO_OK (0) or a negative RPO_ERR_* code; nothing throws or
 *    aborts across this boundary.  rpo_strerror() names a code.
 *  - Pointer prefixes: d_ = device memory owned by the caller (e.g. a torch tensor's
 *    data pointer), h_ = host memory owned by the caller.  The library never frees or
 *    keeps caller memory beyond the call, except that work reading/writing d_ buffers is
 *    *enqueued* on the stream given to rpo_create and may still be running on return;
 *    synchronise that stream before reading outputs or reusing inputs.
 *  - All kernels run on the one CUDA stream passed at creation.  With NULL the library creates a
 *    blocking stream of its own, which keeps the implicit ordering with work on the legacy
 *    default stream (that stream itself cannot be captured into the CUDA graphs decode uses).
 *  - There is no CPU fallback: without a CUDA device every compute call fails with
 *    RPO_ERR_CUDA.
 *  - Matrices are stored [out_features, in_features]; y = x W^T.
 *  - Sequence number of sample i of group g, for the random stream: group_id * G + i.
 */
#ifndef RPO_H_
#define RPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define RPO_OK 0
#define RPO_ERR_INVALID_ARG (-1)     /* NULL pointer, negative size, bad flag                      */
#define RPO_ERR_SHAPE (-2)           /* decoder shape not supported by the kernels                */
#define RPO_ERR_KV_POOL (-3)         /* not enough free KV blocks / group or sequence slots       */
#define RPO_ERR_CUDA (-4)            /* a CUDA runtime call failed (no device, out of memory...)  */
#define RPO_ERR_DEVICE_TIMEOUT (-5)  /* a bounded device-side wait ran out (see rpo_device_status)*/
#define RPO_ERR_NOT_INITIALISED (-6) /* weights not initialised / group handle not live           */
#define RPO_ERR_LIMIT (-7)           /* request exceeds a limit fixed at rpo_create               */

#define RPO_DTYPE_FP32 0
#define RPO_DTYPE_BF16 1

typedef struct rpo_ctx rpo_ctx; /* opaque: weights, paged KV pool, block tables, workspaces */

/* Decoder shape (the paper names the policy models only; these fields describe the
 * pre-norm GQA decoder of the benchmark configurations). */
typedef struct rpo_shape {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  float rope_base; /* theta_i = rope_base^(-2i/head_dim), rotate-half pairing           */
  float rms_eps;   /* inside the square root                                            */
  int32_t dtype;   /* RPO_DTYPE_*: storage type of matrices, K/V and GEMM inputs        */
  int32_t kv_block_tokens; /* tokens per KV block; must be 16                           */
} rpo_shape;

/* Capacity fixed at creation. */
typedef struct rpo_limits {
  int64_t kv_pool_blocks;   /* KV blocks of kv_block_tokens tokens (all layers each)      */
  int32_t max_groups;       /* live prompt groups                                         */
  int32_t max_seqs;         /* sequences decoded in one rpo_decode_suffix call (n_groups*G)*/
  int32_t max_chunk_tokens; /* rows one prefill / log-prob pass works on; a prefix must fit*/
  int32_t max_positions;    /* prefix_len + max_new upper bound (RoPE table, block tables) */
} rpo_limits;

/* Sampler of pi_theta(. | q_k, prefix, o_<j) (Eq. 3).  temperature > 0; 0 <= top_p <= 1.
 * greedy != 0: lowest token id among the maximal logits.  eos_id < 0: no early stop. */
typedef struct rpo_sampler {
  float temperature;
  float top_p;
  int32_t greedy;
  int32_t eos_id;
  uint64_t seed;
} rpo_sampler;

/* Handle of a prefilled prompt group (plain data, caller-held). */
typedef struct rpo_group {
  int32_t group_id;   /* caller's id; decides the random streams of the group's samples   */
  int32_t prefix_len; /* tokens of the cached prefix held in shared KV blocks             */
  int32_t slot;       /* library slot; do not modify                                      */
  int32_t n_blocks;   /* shared KV blocks held by the group                               */
} rpo_group;

const char* rpo_strerror(int code);

/* Fill *out with a named decoder shape: "tiny", "qwen1.5b-class", "qwen7b-class".
 * Returns RPO_ERR_INVALID_ARG for an unknown name. */
int rpo_shape_preset(const char* name, rpo_shape* out);

/* Create a context on the current CUDA device: allocates the weight arena, the paged KV
 * pool ([layer][K|V][kv_head][block][16][head_dim]), block tables and workspaces.
 * cuda_stream is a cudaStream_t (may be NULL).  *out is owned by the caller until
 * rpo_destroy.  Errors: RPO_ERR_SHAPE (vocab >= 2^18, head_dim not 64/128, d_model or d_ffn not a
 * multiple of 8, n_q_heads not a multiple of n_kv_heads, kv_block_tokens != 16),
 * RPO_ERR_CUDA (allocation failed). */
int rpo_create(rpo_ctx** out, const rpo_shape* shape, const rpo_limits* limits, void* cuda_stream);
int rpo_destroy(rpo_ctx* ctx);

/* Seeded random initialisation of the named decoder shape: every matrix element is
 * float32(std) * z with z a standard normal taken from the Philox4x32-10 block
 * (element_index / 4) of stream (seed, tensor id); bf16 models round to nearest even.
 * RMSNorm gains are set to 1.  (The paper trains DeepSeek-R1-Distill-Qwen checkpoints,
 * Section 4; random weights of the same shape stand in for them.) */
int rpo_init_weights(rpo_ctx* ctx, uint64_t seed, float std);

/* Copy one tensor to / from host memory in its storage type (float for fp32 models and
 * for gains, uint16 bf16 bit patterns otherwise), logical layout [out, in].  Names:
 * "embed", "lm_head", "gf", "layers.<l>.{wq,wk,wv,wo,wg,wu,wd,g1,g2}".  bytes must equal
 * the tensor size.  Synchronises the stream. */
int rpo_read_tensor(rpo_ctx* ctx, const char* name, void* h_dst, size_t bytes);
int rpo_write_tensor(rpo_ctx* ctx, const char* name, const void* h_src, size_t bytes);

/* Prefill: run the decoder over the cached prefix q_k || a_k^{[0:-m]} of each group ONCE
 * and keep its K/V in KV blocks that all G samples of the group will read (Eq. 3; Section 3.4
 * notes that the G samples of a group start from one and the same prefix).
 *   d_tokens   device int32, the n_groups prefixes concatenated
 *   h_offsets  host int32 [n_groups+1], prefix g = d_tokens[h_offsets[g] .. h_offsets[g+1])
 *   h_group_ids host int32 [n_groups] or NULL (ids 0..n_groups-1)
 *   h_groups_out host [n_groups], filled before return (no device sync needed)
 * Each prefix needs 1 <= len <= max_chunk_tokens and len < max_positions.
 * Errors: RPO_ERR_KV_POOL (blocks or slots exhausted; nothing is kept), RPO_ERR_LIMIT,
 * RPO_ERR_INVALID_ARG (token ids are NOT range-checked on the host; out-of-range ids are
 * clamped on the device and flagged in rpo_device_status). */
int rpo_prefill_prefix(rpo_ctx* ctx, int32_t n_groups, const int32_t* d_tokens, const int32_t* h_offsets,
                       const int32_t* h_group_ids, rpo_group* h_groups_out);

/* Decode: G continuations per group over the shared prefix KV (Eq. 3; Algorithm 1).
 * Sequence b = g_index*G + i.  Step 0 draws all G samples of a group from the logits of
 * the group's last prefix token; step j feeds token j-1.  A sequence that emits eos_id
 * stops: the EOS token and its log-prob are recorded, later slots hold eos_id / 0.0 and
 * d_lens_out counts tokens up to and including EOS.
 *   d_forced_tokens  NULL, or device int32 [B*max_new]: teacher forcing -- these tokens
 *                    are emitted instead of sampled ones (log-probs still computed)
 *   d_tokens_out     device int32 [B*max_new]
 *   d_lens_out       device int32 [B]
 *   d_logprobs_out   NULL or device float [B*max_new]: log pi(o_j | ...), full vocabulary,
 *                    at the sampler's temperature
 *   d_logits_dbg     NULL or device float [B*max_new*vocab]: the float32 logits every
 *                    step was drawn from (tests only; large)
 * Private suffix KV blocks are taken from the pool for the duration of the call.
 * Errors: RPO_ERR_LIMIT (B > max_seqs, prefix_len+max_new > max_positions),
 * RPO_ERR_KV_POOL, RPO_ERR_NOT_INITIALISED (stale handle), RPO_ERR_INVALID_ARG. */
int rpo_decode_suffix(rpo_ctx* ctx, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                      const rpo_sampler* sampler, const int32_t* d_forced_tokens, int32_t* d_tokens_out,
                      int32_t* d_lens_out, float* d_logprobs_out, float* d_logits_dbg);

/* Decode in waves: the NEXT max_new suffix tokens of each group's G sequences.  Generating the
 * cache's full-path responses (Section 3.1, Eq. 1: one response per question, sampled before
 * training) proceeds in waves so that finished sequences can leave the batch and waiting
 * questions take their place; this call keeps what a sequence needs to go on, so that a wave
 * does not run the decoder over prompt + generated tokens again:
 *   - the first call on a group reserves private KV blocks for max_total suffix tokens per
 *     sequence and one state row per sequence; later calls on the group must pass the same G
 *     and stay within max_total (RPO_ERR_LIMIT otherwise; max_total is read on the first call);
 *   - every token of a wave, the last one included, is run through the decoder before the
 *     call's work ends: its K/V joins the private blocks, and the logits its successor will
 *     be drawn from are parked in the state row (vocab floats) with the finished flag;
 *   - draw number j of a sequence is its absolute suffix position, so W calls of max_new
 *     tokens produce the tokens and log-probs of ONE rpo_decode_suffix call of W*max_new
 *     tokens on the same groups, bit for bit;
 *   - blocks and state rows return to the pool with rpo_release_groups.
 * Groups at different stages may share a call.  Outputs are relative to the wave:
 * d_tokens_out [B*max_new], d_lens_out [B] = tokens of this wave up to and including EOS
 * (0 for a sequence that had finished before), d_logprobs_out NULL or [B*max_new];
 * d_forced_tokens NULL or [B*max_new] as in rpo_decode_suffix.
 * Errors: RPO_ERR_KV_POOL (blocks or state rows exhausted; nothing is reserved),
 * RPO_ERR_LIMIT, RPO_ERR_NOT_INITIALISED, RPO_ERR_INVALID_ARG. */
int rpo_decode_wave(rpo_ctx* ctx, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                    int32_t max_total, const rpo_sampler* sampler, const int32_t* d_forced_tokens,
                    int32_t* d_tokens_out, int32_t* d_lens_out, float* d_logprobs_out);

/* Token log-probabilities log pi_theta(o_{i,j} | q, o_{i,<j}) of given suffixes (numerator
 * and denominator of r_{i,j}, Eq. 7), teacher-forced over the shared prefix KV:
 *   d_tokens [B*max_new], d_lens [B] as written by rpo_decode_suffix
 *   z = logits * inv_temperature; normalisation over the full vocabulary
 *   d_logprobs_out device float [B*max_new]; entries j >= len are 0
 *   d_logits_dbg NULL or device float [B*max_new*vocab] (tests only)
 * The [B*max_new, vocab] logits are produced in bounded row chunks, never whole. */
int rpo_token_logprobs(rpo_ctx* ctx, int32_t n_groups, const rpo_group* h_groups, int32_t G, int32_t max_new,
                       const int32_t* d_tokens, const int32_t* d_lens, float inv_temperature,
                       float* d_logprobs_out, float* d_logits_dbg);

/* Hyper-parameters of the objective (Section 4: clip as in GRPO/DAPO, m = 0.5, M = 1, alpha = 0.01). */
typedef struct rpo_objective_cfg {
  float clip_eps;          /* epsilon of clip(r, 1 - eps, 1 + eps), Eq. 6                      */
  float beta;              /* weight of the KL term of Eq. 5 (0: off)                          */
  float alpha;             /* length sensitivity of Eq. 11                                     */
  float reward_min;        /* m of Eq. 11                                                      */
  float reward_max;        /* M of Eq. 11                                                      */
  int32_t length_shaping;  /* 0: use the raw rewards as R_i                                    */
} rpo_objective_cfg;

/* Forward value of the RPO objective of one rollout batch (Section 3.2, Eq. 5-7; Section 3.4,
 * Eq. 11), on the device, from the log-probabilities rpo_token_logprobs produces:
 *   R_i  = clip(raw_i / (1 + exp(-alpha (l_ref - len_i))), m, M), l_ref = group mean of len  (Eq. 11)
 *   A_i  = (R_i - mean_R) / std_R over the sampling group (population std; 0 if std = 0)    (Eq. 7)
 *   l_ij = min(r_ij A_i, clip(r_ij, 1 +- eps) A_i), r_ij = exp(logp_new - logp_old)           (Eq. 6, 7)
 *   J    = mean over groups of 1/G sum_i 1/|o_i| sum_j [l_ij - beta k3_ij]                    (Eq. 5)
 * with k3 = exp(d) - d - 1, d = logp_ref - logp_new, the per-token KL estimator of GRPO.
 *   d_logp_new/old/ref float [B*max_new] (ref NULL: no KL term), d_lens int32 [B] = |o_i| (tokens
 *   generated in this rollout), d_resp_lens int32 [B] or NULL (= d_lens): len_i of Eq. 11,
 *   d_raw_rewards float [B]; outputs d_rewards_out [B], d_advantages_out [B], d_token_loss_out
 *   [B*max_new] or NULL (0 beyond len), d_group_objective_out [n_groups], d_objective_out [1].
 * Errors: RPO_ERR_LIMIT (G > 64), RPO_ERR_INVALID_ARG. */
int rpo_policy_objective(rpo_ctx* ctx, int32_t n_groups, int32_t G, int32_t max_new, const float* d_logp_new,
                         const float* d_logp_old, const float* d_logp_ref, const int32_t* d_lens,
                         const int32_t* d_resp_lens, const float* d_raw_rewards, const rpo_objective_cfg* cfg,
                         float* d_rewards_out, float* d_advantages_out, float* d_token_loss_out,
                         float* d_group_objective_out, float* d_objective_out);

/* Return the groups' shared KV blocks and slots to the pool (host bookkeeping; work
 * already enqueued on the stream is unaffected because later work is ordered after it). */
int rpo_release_groups(rpo_ctx* ctx, int32_t n_groups, const rpo_group* h_groups);

/* Whole rollout with HOST buffers (the call an application makes once per batch):
 * copies the prefix tokens to the device, prefills, decodes, optionally computes the
 * teacher-forced log-probs (want_policy_logprobs != 0 -> h_policy_logprobs_out), copies
 * the results back, releases the groups and synchronises the stream.
 * h_tokens_out [B*max_new], h_lens_out [B], h_logprobs_out [B*max_new] or NULL.
 * The device staging buffers belong to the context: allocated on the first call, grown
 * when a later call needs more, freed by rpo_destroy. */
int rpo_rollout_host(rpo_ctx* ctx, int32_t n_groups, const int32_t* h_tokens, const int32_t* h_offsets,
                     const int32_t* h_group_ids, int32_t G, int32_t max_new, const rpo_sampler* sampler,
                     int32_t* h_tokens_out, int32_t* h_lens_out, float* h_logprobs_out,
                     int32_t want_policy_logprobs, float* h_policy_logprobs_out);

/* The sampler alone, on caller-supplied float32 logits [n_rows, vocab] (row r belongs to
 * sequence d_seq_ids[r], draw number `step`): used to test the sampler in isolation.
 * d_tokens_out int32 [n_rows]; d_logprobs_out NULL or float [n_rows].  Takes n_rows*vocab*4
 * bytes of stream-ordered temporary device memory for the call. */
int rpo_sample_rows(rpo_ctx* ctx, int32_t n_rows, int32_t vocab, const float* d_logits, const rpo_sampler* sampler,
                    const int64_t* d_seq_ids, int32_t step, int32_t* d_tokens_out, float* d_logprobs_out);

/* The same sampler for callers that must not allocate.  (The paper has no counterpart: this is a
 * deployment variant of rpo_sample_rows, not a step of the method.)  Some hosts of this library
 * cannot obtain device memory when they sample: a serving process that gave the whole device to
 * its own memory pool at start-up, a plug-in that is handed buffers and a stream but no
 * allocator, a latency-critical loop in which the implicit synchronisation of an allocation is
 * not acceptable.  This call needs no rpo_ctx and calls no allocating routine; the per-token
 * weight scratch the sampler needs is a fixed 16 MiB array inside the library image, which every
 * GPU that loads the library holds until the process exits.
 *   n_rows * vocab must not exceed 4 * 2^20 words (e.g. 27 rows of a 151936-token vocabulary):
 *   larger requests are rejected with RPO_ERR_LIMIT and a message on stderr, nothing is launched.
 *   d_logits float32 [n_rows, vocab], d_seq_ids int64 [n_rows], d_tokens_out int32 [n_rows],
 *   d_logprobs_out NULL or float32 [n_rows]: caller-owned device memory, as in rpo_sample_rows;
 *   cuda_stream: the cudaStream_t the kernel is enqueued on (may be NULL); sampler->eos_id is
 *   ignored.  Results are identical to rpo_sample_rows.
 * The first call on a device looks up the array's device address and sets a kernel attribute
 * (once per device, for the device current at that moment); make that first call before any
 * stream capture.  All calls on a device share the one array and it keeps the previous call's
 * contents; nothing in it has to start at zero, because every row's words are rewritten before
 * they are read.  Two calls whose kernels overlap on the GPU (different streams, no ordering
 * between them) race on the array: order them. */
int rpo_sample_rows_noalloc(int32_t n_rows, int32_t vocab, const float* d_logits, const rpo_sampler* sampler,
                            const int64_t* d_seq_ids, int32_t step, int32_t* d_tokens_out, float* d_logprobs_out,
                            void* cuda_stream);

/* Dense product C[M,N] = A[M,K] * W[N,K]^T through the same GEMM kernel the layers use
 * (storage type of the context; C is float32).  For kernel-level parity tests.
 * impl: 0 = the kernel the context would choose, 1 = plain CUDA-core kernel,
 * 2 = tcgen05/TMA kernel (bf16 only; RPO_ERR_SHAPE if K % 64 != 0 or N % 16 != 0). */
int rpo_gemm(rpo_ctx* ctx, int32_t impl, int32_t M, int32_t N, int32_t K, const void* d_A, const void* d_W,
             float* d_C);

/* Kernel micro-benchmark (bf16 contexts): the tensor-core GEMM of C[M,N] = A[M,K] W^T as the layers
 * launch it (planner or its "gemm_bn"/"gemm_splits" override; split-K planes are left unreduced),
 * `iters` launches cycling through the n_w weight matrices of h_W_list (host array of device
 * pointers; use enough matrices to exceed the L2 capacity), replayed as one CUDA graph.  The output
 * goes to an internal buffer.  *h_ms_out = mean device time per launch in milliseconds.
 * Synchronises the stream.  RPO_ERR_LIMIT if M*N exceeds the internal logits buffer. */
int rpo_gemm_bench(rpo_ctx* ctx, int32_t M, int32_t N, int32_t K, const void* d_A, const void* const* h_W_list,
                   int32_t n_w, int32_t iters, float* h_ms_out);

/* Device status word, sticky until read: 0 = clean; bit 0 = a bounded wait expired
 * (TMA / MMA pipeline), bit 1 = token id out of range (clamped), bit 2 = block-table
 * index out of range (access skipped).  Synchronises the stream; *out receives the word
 * and the word is cleared.  Returns RPO_ERR_DEVICE_TIMEOUT when bit 0 was set (the results of
 * the work enqueued since the last read are not to be trusted; the context stays usable),
 * else RPO_OK.  The asynchronous entry points (prefill, decode, token log-probs) cannot
 * report an expired wait themselves: poll this call after them.  rpo_rollout_host, which
 * synchronises anyway, checks the word itself and returns RPO_ERR_DEVICE_TIMEOUT (bit 0) or
 * RPO_ERR_CUDA (bit 2). */
int rpo_device_status(rpo_ctx* ctx, int32_t* out);

/* Test tap on the residual stream (the hidden state x of the decoder the policy pi_theta of Eq. 3
 * and Eq. 7 evaluates).  While a buffer is set, every pass through the layer stack (each prefill
 * chunk, each decode forward, each chunk of rpo_token_logprobs) appends to it, in call order:
 * the rows entering layer 0 as [rows, d_model] float32; then for every layer its attention
 * output [rows, n_q_heads*head_dim] in the storage type (two bf16 values per float slot) and the
 * rows leaving the layer as [rows, d_model] float32.  A parity test can thus check every layer
 * on its own against the definition, fed with the library's own layer input, so that 16-bit
 * storage rounding does not accumulate over the depth of the model in the comparison.
 *   d_buf device float [capacity_floats], caller-owned; NULL switches the tap off.  Each call
 *   restarts the write position at 0; h_used_out (nullable) receives the number of floats written
 *   through the previous setting.  A pass that would overflow the buffer fails with RPO_ERR_LIMIT.
 * While the tap is on the decode step is not replayed as a CUDA graph. */
int rpo_debug_tap(rpo_ctx* ctx, float* d_buf, int64_t capacity_floats, int64_t* h_used_out);

/* Counters since creation: kernels launched by the library, free KV blocks. */
int rpo_counters(rpo_ctx* ctx, int64_t* kernel_launches, int64_t* free_kv_blocks);

/* Runtime switches (tests/benchmarks): name = "use_tcgen05" (bf16 GEMMs on the tensor-core
 * kernel, default 1), "use_tc_attention" (tensor-core attention kernels, default 1),
 * "use_graph" (CUDA graph per decode step, default 1), "use_pdl" (programmatic dependent launch
 * between the library's kernels: 0 off, 1 = in prefill / log-prob passes and inside the captured decode-step
 * graphs (default), 2 = also on the eagerly launched kernels of a decode call -- not recommended: with 2, a
 * rollout of 512 sequences stopped making progress about once in thirty calls on B200 / driver 580, never
 * with 0 or 1), "use_tc5_attention" (tcgen05 attention for
 * many-row passes at head_dim 128, default 1), "use_gemm_pairs" (256 x 256 GEMM tiles on CTA
 * pairs for passes of more than 128 rows, default 1), "use_cluster_merge" (decode attention:
 * the prefix splits of a work item form a thread-block cluster and merge through distributed
 * shared memory instead of a second kernel; default 0), "profile" (see rpo_profile_read),
 * "use_tc5_decode" (tcgen05 decode attention when a group's rows of one KV head fit a 64-row
 * tile; default 0: the mma.sync kernel measured faster), "use_fused_layers" (RMSNorm / RoPE / KV append / SwiGLU / residual add as GEMM
 * epilogues in passes whose products do not split K, default 1; 2 = also where they split),
 * "use_tc5_pipelined" (the pipelined variant of the tcgen05 prefill attention: 64-key tiles, running output in
 * tensor memory; default 0: measured 6-9 % slower),
 * "use_fused_lse" (rpo_token_logprobs: the output head keeps, per row and tile, the running maximum,
 * the sum of exponentials and the target's logit instead of writing the logits; default 1 = where the
 * CTA-pair kernel serves the output head, 2 = always, 0 = never; calls that ask for d_logits_dbg always
 * write the logits),
 * "wait_limit_cycles" (limit of every bounded device-side wait in SM cycles, for ALL contexts on the
 * device; <= 0 restores the default of 2e8, about 0.1 s),
 * "gemm_bn" (0 = planner, else force the tensor-core tile width: 32/64/96/128/256, or 512 / 384
 * for the CTA-pair kernel with 128 / 64 rows per CTA) and "gemm_splits" (with gemm_bn: force the split-K factor where the
 * caller can reduce planes). */
int rpo_set_option(rpo_ctx* ctx, const char* name, int32_t value);

/* Per-kernel timing.  With option "profile" = 1 every kernel launch is bracketed by a pair of
 * CUDA events on the context's stream (this serialises nothing but adds event overhead, and
 * turns CUDA-graph replay off).  rpo_profile_read synchronises, sums the elapsed times and
 * launch counts since the last read into ms_out / count_out [3 phases x 6 classes], index
 * phase*6 + class; phases: 0 prefill, 1 decode, 2 token log-probs; classes: 0 other, 1 GEMM,
 * 2 attention, 3 sampler, 4 RMSNorm, 5 RoPE + KV write.  n >= 18. */
int rpo_profile_read(rpo_ctx* ctx, double* ms_out, int64_t* count_out, int32_t n);

#ifdef __cplusplus
}
#endif
#endif /* RPO_H_ */
