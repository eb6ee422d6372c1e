/*
 * phyai.h - C ABI of the B200 (sm_100a) flow-matching action-expert denoising library.
 *
 * One policy request returns one H-action chunk (paper, Sec. "Task Formulation", Eq. 1:
 * a_{t:t+H-1} = pi_theta(x_t)); for flow policies pi_theta refines an action latent over
 * several steps.  This library is that refinement loop alone: for k = 0..n-1 the action-expert
 * transformer is evaluated on the suffix tokens (optional robot-state token + H noisy action
 * tokens, conditioned on the time t_k) attending to themselves and to a frozen per-layer
 * prefix KV cache, followed by the Euler update x <- x + dt * v(x, t_k), dt = -1/n, t from 1
 * towards 0 (Sec. "Optimization Methods", graph-replay paragraph: the prefix stays fixed over
 * the ten Euler steps, its KV tensors are retained, the sinusoidal timestep table and each
 * layer's AdaRMS modulation table are built before denoising, the full loop is captured in one
 * CUDA graph).  The per-layer operators are those of the kernel-fusion paragraph: (Ada)RMSNorm,
 * one GEMM for Q,K,V, attention of the few suffix queries over the long prefix (operator-selection
 * paragraph), residual add, one GEMM for MLP gate and up with GeGLU fused, down projection.
 *
 * Conventions
 *   - All matrices are row-major [in, out]; activations are row vectors (y = x W + b).
 *   - "device" pointers are CUDA device memory owned by the caller; "host" pointers are ordinary
 *     host memory.  The library never frees caller memory and keeps no caller pointer after the
 *     work it enqueued has finished.
 *   - Every call returns a phyai_status_t; nothing throws or aborts across the ABI.
 *     phyai_last_error() gives a thread-local description of the last failure.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Not thread-safe per handle; one call in flight per handle; handles are independent.
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails.
 */
#ifndef PHYAI_H_
#define PHYAI_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct phyai_expert phyai_expert_t; /* opaque: packed weights, tables, workspace, graphs */

typedef enum {
  PHYAI_OK = 0,
  PHYAI_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, size out of the configured range        */
  PHYAI_ERR_UNSUPPORTED = 2, /* a shape or mode the kernels do not cover                          */
  PHYAI_ERR_OOM = 3,         /* device or host allocation failed                                   */
  PHYAI_ERR_CUDA = 4,        /* a CUDA runtime call failed (message in phyai_last_error)           */
  PHYAI_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (reported by phyai_poll_status) */
} phyai_status_t;

/* Storage precision of weights and prefix KV. */
typedef enum {
  PHYAI_F32 = 0,       /* everything float32; arithmetic in true fp32 (no TF32)                       */
  PHYAI_BF16 = 1,      /* weights and prefix KV bfloat16; bf16 tensor-core operands, fp32 accumulate   */
  PHYAI_W8E4M3_A16 = 2, /* the seven large per-layer matrices as e4m3 bytes with one fp32 scale per
                          output channel (offline round-to-nearest, quantization paragraph); all other
                          tensors and the prefix KV bfloat16; activations bf16                        */
  PHYAI_W8A8_E4M3 = 3, /* storage as PHYAI_W8E4M3_A16; in addition the input of each of the four large
                          projections of a layer (fused QKV, attention output, gate / up, down) is
                          quantised per token to e4m3 -- scale = max|x| / 448, codes round-to-nearest-even,
                          saturating -- and the products run on the FP8 tensor path (quantization
                          paragraph: W8A8).  Tensor path only; kernels of the general (any batch) family */
  PHYAI_W4A16 = 4      /* the seven large per-layer matrices as symmetric 4-bit integers with one fp32 scale per
                          output channel (quantization paragraph: W4A16, round-to-nearest): a byte of the
                          [in][out / 2] array holds the codes of output channels 2j (low nibble) and 2j + 1
                          (high nibble) of one input row, code c = integer c - 8 in [-8, 7], weight = integer x
                          scale; everything else as PHYAI_W8E4M3_A16.  The integers are expanded to bf16 operand
                          images at create (exact), the scales enter in the epilogues                        */
} phyai_dtype_t;

/* How the time t_k conditions the expert. */
typedef enum {
  PHYAI_COND_PI0_CONCAT = 0, /* action token = swish([x Wa + ba ; tau] W1 + b1) W2 + b2; plain RMSNorm */
  PHYAI_COND_PI05_ADARMS = 1 /* action token = x Wa + ba; c = swish(swish(tau W1+b1) W2+b2); every norm
                                site has a dense D -> 3D (scale | shift | gate): n = rms(h)(1+scale)+shift,
                                gate multiplies the sub-layer output before the residual add            */
} phyai_cond_t;

/* Kernel family (debug / verification aid). */
typedef enum {
  PHYAI_ENGINE_AUTO = 0,  /* fp32 storage -> CUDA-core path; bf16 / e4m3 -> tcgen05 tensor path */
  PHYAI_ENGINE_SIMT = 1   /* force the CUDA-core fp32-arithmetic path for any storage type       */
} phyai_engine_t;

typedef struct {
  uint32_t struct_size;      /* = sizeof(phyai_expert_config_t), for ABI growth                        */
  uint32_t n_layers, width, mlp_dim, n_q_heads, n_kv_heads, head_dim;
  uint32_t state_dim, action_dim, horizon;
  uint32_t has_state_token;  /* 1: suffix = state token + H action tokens; 0: H action tokens          */
  uint32_t max_prefix_len;   /* largest prefix_len of one request                                      */
  uint32_t max_batch;        /* largest batch of phyai_denoise_batched                                 */
  uint32_t cond;             /* phyai_cond_t                                                           */
  uint32_t dtype;            /* phyai_dtype_t                                                          */
  float rms_eps;             /* inside the square root                                                 */
  float rope_theta;          /* 0 = no rotary embedding; suffix token i sits at position prefix_len+i  */
  float time_min_period, time_max_period; /* sinusoid periods, geometric over width/2 channels         */
  uint32_t gelu_exact;       /* 0 = tanh form, 1 = erf form                                            */
  uint32_t suffix_block_causal; /* 0 = suffix fully bidirectional; 1 = state token sees only itself    */
  uint32_t engine;           /* phyai_engine_t                                                         */
} phyai_expert_config_t;

/*
 * Weights: device pointers, caller-owned, storage per `dtype` (float32 / bfloat16; for
 * PHYAI_W8E4M3_A16 the seven per-layer matrices are uint8 e4m3 codes and `scales` is set).
 * Per-layer members are HOST arrays of n_layers DEVICE pointers.  Members a mode does not
 * have are NULL.  phyai_expert_create copies / repacks everything, so the caller may free its
 * copies once the create call's stream work is complete (create synchronises before returning).
 *
 *   state_w [Ds,D], state_b [D]                      (has_state_token only)
 *   action_in_w [A,D], action_in_b [D]
 *   time_mlp1_w [2D,D] (pi0: rows 0..D-1 multiply the action embedding, rows D..2D-1 multiply tau)
 *               [D,D]  (pi0.5), time_mlp1_b [D], time_mlp2_w [D,D], time_mlp2_b [D]
 *   action_out_w [D,A], action_out_b [A]
 *   final_norm: gamma [D] (gain is 1+gamma)  |  pi0.5: W_mod [D,3D], final_norm_b [3D]
 *   wq [D,Hq*dh] wk [D,Hkv*dh] wv [D,Hkv*dh] wo [Hq*dh,D] wgate [D,F] wup [D,F] wdown [F,D]  (no biases)
 *   norm1 / norm2: gamma [D]  |  pi0.5: W_mod [D,3D] with norm1_b / norm2_b [3D]
 *   scales[m][l] -> float[out] for m = 0..6 (q,k,v,o,gate,up,down)
 */
typedef struct {
  const void *state_w, *state_b, *action_in_w, *action_in_b;
  const void *time_mlp1_w, *time_mlp1_b, *time_mlp2_w, *time_mlp2_b;
  const void *action_out_w, *action_out_b, *final_norm, *final_norm_b;
  const void *const *wq, *const *wk, *const *wv, *const *wo, *const *wgate, *const *wup, *const *wdown;
  const void *const *norm1, *const *norm1_b, *const *norm2, *const *norm2_b;
  const float *const *scales[7];
} phyai_weights_t;

/*
 * Create an expert (Sec. "Architecture": the model runner owns buffers, caches and graphs; the
 * modelling code is stateless).  Allocates packed weights, the rotary table and a workspace
 * sized from max_batch and max_prefix_len, repacks the weights on `stream` and synchronises it.
 * On failure *out is NULL.  Errors: INVALID_ARG (NULL, zero sizes, n_q_heads not a multiple of
 * n_kv_heads, odd head_dim/width), UNSUPPORTED (shape outside the tensor path's tiling:
 * width, mlp_dim, n_q_heads*head_dim must be multiples of 128 there), OOM, CUDA.
 */
phyai_status_t phyai_expert_create(const phyai_expert_config_t *cfg, const phyai_weights_t *weights,
                                   void *stream, phyai_expert_t **out);

/* Free everything the handle owns (synchronises the device first). NULL is ignored. */
void phyai_expert_destroy(phyai_expert_t *h);

/* Bytes of a prefix-KV buffer holding `total_prefix_tokens` tokens, layout below. 0 on bad input. */
size_t phyai_prefix_kv_bytes(const phyai_expert_config_t *cfg, uint64_t total_prefix_tokens);

/*
 * Denoise one action chunk (graph-replay paragraph: ten Euler steps over a fixed prefix).
 *
 *   prefix_kv   device, layout [n_layers][2 (K,V)][kv_tokens][n_kv_heads][head_dim], head_dim
 *               contiguous, float32 for PHYAI_F32 else bfloat16, 16-byte aligned; K is used as
 *               given (already rotated by the producer).  kv_tokens is the token capacity of the
 *               buffer (>= prefix_len); rows >= prefix_len are never read.
 *   prefix_len  0 <= prefix_len <= min(kv_tokens, max_prefix_len); 0 = suffix-only attention.
 *   state       device float32 [state_dim] (NULL iff has_state_token == 0)
 *   noise       device float32 [horizon, action_dim]: x at t = 1
 *   n_steps     >= 1; dt = -1/n_steps, t_k = 1 - k/n_steps
 *   out_actions device float32 [horizon, action_dim]: x at t = 0; may alias `noise`
 *
 * Only enqueues work on `stream` and returns; results are valid once the stream has been
 * synchronised.  The first call with a new n_steps builds that step count's tables (time
 * embedding, per-step bias or modulation) and, unless disabled, captures the loop as a CUDA
 * graph; it is slower and should be kept out of timed regions.  Errors: INVALID_ARG.
 */
phyai_status_t phyai_denoise(phyai_expert_t *h, const void *prefix_kv, uint64_t kv_tokens, uint32_t prefix_len,
                             const float *state, const float *noise, uint32_t n_steps, float *out_actions,
                             void *stream);

/*
 * Batched variant for many concurrent rollouts (Sec. "Parallel Execution": requests are
 * independent and exchange no state).  Request b uses rows cu_prefix_lens[b] ..
 * cu_prefix_lens[b+1]-1 of the packed prefix KV (same layout, requests concatenated along the
 * token axis, no padding rows), its own state and noise.
 *
 *   batch           1 <= batch <= max_batch
 *   prefix_kv       device, [n_layers][2][kv_tokens][n_kv_heads][head_dim]
 *   cu_prefix_lens  device int32 [batch+1], non-decreasing, cu[0] >= 0, cu[batch] <= kv_tokens,
 *                   every difference <= max_prefix_len (checked on the device: a violation sets
 *                   the status word to INVALID_ARG and the call writes nothing)
 *   states          device float32 [batch, state_dim] or NULL
 *   noise, out      device float32 [batch, horizon, action_dim]
 */
phyai_status_t phyai_denoise_batched(phyai_expert_t *h, uint32_t batch, const void *prefix_kv, uint64_t kv_tokens,
                                     const int32_t *cu_prefix_lens, const float *states, const float *noise,
                                     uint32_t n_steps, float *out_actions, void *stream);

/*
 * Host-buffer variants: all tensor arguments (cu_prefix_lens included) are HOST pointers
 * (pinned memory makes the copies asynchronous).  The call copies them into handle-owned
 * device staging buffers on `stream`, runs the same kernels, and copies the actions back to
 * `out_actions` (host).  The result is valid after the stream is synchronised.  The KV staging
 * buffer holds max_batch * max_prefix_len tokens; kv_tokens beyond that -> INVALID_ARG.
 */
phyai_status_t phyai_denoise_host(phyai_expert_t *h, const void *prefix_kv, uint64_t kv_tokens, uint32_t prefix_len,
                                  const float *state, const float *noise, uint32_t n_steps, float *out_actions,
                                  void *stream);
phyai_status_t phyai_denoise_batched_host(phyai_expert_t *h, uint32_t batch, const void *prefix_kv,
                                          uint64_t kv_tokens, const int32_t *cu_prefix_lens, const float *states,
                                          const float *noise, uint32_t n_steps, float *out_actions, void *stream);

/*
 * After the stream has been synchronised: read and clear the handle's device status word.
 * PHYAI_OK, PHYAI_ERR_TIMEOUT (a bounded wait inside a kernel expired; results are invalid) or
 * PHYAI_ERR_INVALID_ARG (device-side validation of cu_prefix_lens failed).  Synchronises the
 * device copy of one word; do not call during stream capture.
 */
phyai_status_t phyai_poll_status(phyai_expert_t *h);

/* Options (testing and measurement aids).  key "use_graph": 0 launches the kernels directly, 1 (default)
 * replays a captured CUDA graph per (batch, n_steps).  key "use_tc_attention": 1 (default) lets large batches
 * use the tcgen05 attention kernel, 0 keeps the mma.sync kernel.  key "use_cluster_attention": 1 (default) lets
 * calls with few requests merge their key-split attention partials through distributed shared memory (clusters
 * of 8 CTAs), 0 keeps the split kernel + merge kernel.  key "use_fused_oproj": 1 lets that cluster kernel also
 * apply the attention output projection of its head (head_dim 256, model width 1024, one token tile).
 * key "use_cluster_gemm": 1 (default) runs the projections of calls with at most 64 suffix tokens on the
 * cluster split-K kernel (k-ranges of a channel tile reduce over distributed shared memory; the norms are
 * folded into the neighbouring projections), 0 keeps the general kernel + norm kernels.
 * key "slab_splits": 1..16 (default 8), the most k-ranges a residual projection of a single-token-tile call is
 * split into on the general kernel (partial sums are written as slabs and added in slab order: bit-reproducible).
 * key "b1_c_qkv" / "b1_c_o" / "b1_c_gu" / "b1_c_d": cluster size (k-ranges per channel tile, 1..8; 0 = choose) of
 * the four projections on the cluster split-K kernel.  key "use_b1_attention": 1 (default) lets those calls use
 * the cluster tcgen05 attention kernel (head_dim 128 / 256, even head and group counts), 0 keeps the mma.sync
 * cluster kernel.  key "use_w8_inkernel": 1 (default) streams PHYAI_DTYPE_FP8_E4M3 weights as bytes and decodes
 * them inside the cluster GEMM, 0 reads the bf16 images made at create (bit-identical results, twice the bytes).
 * key "use_state_cache": 1 lets a block-causal expert (Sec. "adapters"; the state tokens see only the prefix and
 * themselves, so their keys and values do not change over the steps) run its state tokens once per call and the
 * loop on the action tokens only; 0 (default) runs every suffix token in every step, which is faster as long as the
 * state token does not cost a token tile of its own.
 * key "b1_attn_hpc": query heads per CTA (1 or 2; 0 = choose) of the cluster attention kernel.  key "use_b1_step":
 * 1 (default) runs the step boundary of those calls (velocity head, Euler update, next embedding) as one cluster kernel.
 * key "use_persistent_gu" / "use_persistent_qkv": 1 (default) runs the gate/up and the q|k|v projection of calls
 * with more than 1024 suffix tokens on the persistent tile kernel (one CTA per SM, two accumulators, a tile's
 * epilogue under the next tile's main loop); 0 keeps them on the one-tile-per-CTA kernel.
 * key "use_attn_splits": 1 (default) lets calls of few requests (at most a quarter of the SMs' worth of head-pair
 * CTAs) split every request's key tiles over up to 8 CTAs of the tcgen05 attention kernel, merged by a second launch.
 * key "trace": see phyai_read_trace.
 * key "wait_limit": iteration bound of the device-side waits on other agents' progress (testing).
 * Unknown key -> INVALID_ARG. */
phyai_status_t phyai_set_option(phyai_expert_t *h, const char *key, int64_t value);

/*
 * Tracing aid (the paper times phases with GPU-side profiler scopes; Sec. "Results", measurement protocol).
 * With option "trace" = 1, one CTA of every cluster-GEMM and cluster-attention launch of a call writes
 * device-global-timer stamps (ns) into slot `launch index` (position of the launch within the call, from 0) of a
 * 4096 x 16 buffer: [0] kernel start, [1] set-up done, [2] dependency resolved (for attention: Q acquired),
 * [3] MMAs / key tiles complete, [4] partials of the cluster received, [5] results stored, [6] cluster released,
 * [7] (GEMM) the SM the CTA ran on, (attention) probabilities written; [8..15] further stamps of the attention
 * kernel (Q copied, Q in tensor memory, logits ready, partial staged, ...).  After the stream is synchronised phyai_read_trace copies the buffer to `out`
 * (HOST memory, capacity >= 4096 * 16 entries); slots of launches that are not traced stay 0.  The stamps cost
 * a few hundred ns each: a traced call is slower.  "trace" = 0 turns it off.
 * Option "trace_all_from" = i > 0 (with "trace" = 1): instead, EVERY CTA of the cluster-GEMM and cluster-attention
 * launches with index i .. i + 4 of a call stamps, into consecutive slots (slot = CTAs of the earlier traced launches +
 * the CTA's linear index in its grid); 0 returns to one CTA per launch.
 * For calls with more than 64 suffix tokens "trace_all_from" = i traces launch i alone, if it is a tile GEMM: slot =
 * the CTA's linear index, stamps [0] start, [1] set-up done, [2] dependency resolved, [3] first operands landed,
 * [4] last MMA issued, [5] (first) accumulator complete, [6] epilogue's stores issued, [7] SM, [8] tensor memory
 * released, [9] tiles walked (persistent kernel).
 * The tcgen05 attention kernel of such calls is traced the same way: [0] start, [1] dependency resolved, [2] Q in
 * tensor memory, [3] S(0) issued, [4] P V(0) issued, [5] all MMAs issued, [6] last P V complete, [7] SM, [8] output
 * stored, [9] key tiles, [10] = 1.
 */
phyai_status_t phyai_read_trace(phyai_expert_t *h, uint64_t *out, size_t capacity, uint32_t *n_slots,
                                uint32_t *n_stamps);

/* Number of kernel launches (graph nodes) one denoise call with this batch / n_steps issues;
 * 0 if unknown.  Reporting aid for benchmarks. */
uint64_t phyai_launches_per_call(phyai_expert_t *h, uint32_t batch, uint32_t n_steps);

/*
 * Stand-alone operator: suffix -> (prefix U suffix) attention of one layer (operator-selection
 * paragraph: a ~50-token query against a longer prefix, head dimension 256), the kernel the
 * denoising loop uses, callable on its own.
 *
 *   desc            shapes; head_dim in {64,128,256}, suffix_len <= 64; num_splits 0 lets the
 *                   library choose how many CTAs share one request's key range (1..16 to fix it)
 *   qkv             device float32 [batch*suffix_len][(Hq + 2 Hkv) * head_dim] = (q | k | v) rows of
 *                   the suffix tokens, NOT yet rotated
 *   prefix_kv       device bfloat16 [n_layers][2][kv_tokens][Hkv][head_dim]; planes of `layer` are read
 *   cu_prefix_lens  device int32 [batch+1], non-decreasing, cu[0] >= 0, cu[batch] <= kv_tokens (checked on the
 *                   device: a violation sets *status_word to PHYAI_ERR_INVALID_ARG and nothing is written);
 *                   batch <= 65535
 *   rope_cos_sin    device float32 [positions][head_dim/2][2] = (cos, sin) of position * theta^(-2j/dh)
 *                   for every position < max prefix_len + suffix_len, or NULL for no rotation;
 *                   suffix token i of a request sits at position prefix_len + i
 *   out             device bfloat16 (as uint16) row-major [batch*suffix_len][Hq*head_dim]
 *   status_word     device int32, zeroed by the caller; stays 0 on success, becomes PHYAI_ERR_INVALID_ARG
 *                   (cu_prefix_lens) or PHYAI_ERR_TIMEOUT (a bounded wait inside the kernel expired)
 *
 * Split-KV partial results need scratch memory: this entry point takes it from the stream-ordered
 * allocator (cudaMallocAsync / cudaFreeAsync on `stream`).  Only enqueues work.  Errors: INVALID_ARG,
 * UNSUPPORTED, OOM, CUDA; message in phyai_op_last_error().
 */
typedef struct {
  uint32_t struct_size;
  uint32_t n_q_heads, n_kv_heads, head_dim, suffix_len;
  uint32_t n_layers, layer;
  uint32_t state_token_block_causal; /* 1: suffix row 0 sees, of the suffix keys, only key 0 */
  uint32_t num_splits;
} phyai_attention_desc_t;

phyai_status_t phyai_suffix_attention(const phyai_attention_desc_t *desc, uint32_t batch, const float *qkv,
                                      const void *prefix_kv, uint64_t kv_tokens, const int32_t *cu_prefix_lens,
                                      const float *rope_cos_sin, uint16_t *out, int32_t *status_word, void *stream);

/* Scratch bytes phyai_suffix_attention uses for this shape and batch (upper bound when num_splits is 0). */
size_t phyai_suffix_attention_scratch_bytes(const phyai_attention_desc_t *desc, uint32_t batch);

/*
 * phyai_suffix_attention without any allocation.  (The paper has no counterpart; this entry point
 * exists for callers that must not allocate device memory: code running where cudaMalloc is
 * forbidden or unavailable, for example a real-time control loop with a no-allocation rule after
 * start-up, a process whose memory pool is owned and capped by another component, or a plug-in
 * that may only use the buffers it is handed.)
 *
 * Same arguments, same result as phyai_suffix_attention; the caller still passes inputs, the
 * output and the status word.  The request block and the split-KV partials go into a fixed
 * 16 MiB array (phyai_suffix_attention_static_capacity()) that is part of the library image: every GPU that
 * loads the library holds it until the process exits.  The call uses no cudaMalloc, cudaFree,
 * stream-ordered allocator or other allocating routine.
 *
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and remembers it; make that first call before starting any stream capture.
 *   - Shapes that need more than the capacity (256 bytes + batch * Hq * splits * 64 * (head_dim + 2) * 4)
 *     are rejected with PHYAI_ERR_INVALID_ARG and a message naming both numbers; with
 *     num_splits == 0 the library picks a split count first and then checks.
 *   - All calls on a device share the one array and it keeps the last call's contents.  Nothing
 *     in it needs clearing between calls, but two calls that overlap on the GPU (different
 *     streams, or different host threads) race on it: serialise them.
 */
phyai_status_t phyai_suffix_attention_static(const phyai_attention_desc_t *desc, uint32_t batch, const float *qkv,
                                             const void *prefix_kv, uint64_t kv_tokens,
                                             const int32_t *cu_prefix_lens, const float *rope_cos_sin, uint16_t *out,
                                             int32_t *status_word, void *stream);
size_t phyai_suffix_attention_static_capacity(void);

/*
 * The steps either side of the loop that belong to the model adapter (Sec. "Architecture": the adapter owns
 * preprocessing, cache validity and action conversion).
 *
 * phyai_pack_prefix_kv: a backbone's padded K / V of every layer -> the library's ragged prefix-KV layout.
 *   desc            n_layers, n_kv_heads, head_dim, elem_bytes (2 = bfloat16, 4 = float32), batch, p_max
 *   k, v            device, [n_layers][batch][p_max][n_kv_heads][head_dim], K already rotated; rows >= lens[b] are
 *                   padding and are never read; 16-byte aligned
 *   lens            device int32 [batch], 0 <= lens[b] <= p_max
 *   prefix_kv       device, receives [n_layers][2][kv_tokens][n_kv_heads][head_dim]: request b at rows
 *                   cu[b] .. cu[b] + lens[b] - 1, no padding rows; rows >= cu[batch] are left untouched
 *   cu_prefix_lens  device int32 [batch + 1], written: the exclusive prefix sum of lens
 *   status_word     device int32, zeroed by the caller; a length outside 0..p_max or sum(lens) > kv_tokens sets it to
 *                   PHYAI_ERR_INVALID_ARG and nothing is copied (cu_prefix_lens is still written)
 * Bit-exact copy.  Only enqueues work on `stream`.  Errors: INVALID_ARG (NULL, zero size, misalignment, a row that
 * is not a multiple of 16 bytes), CUDA; message in phyai_adapter_last_error().
 */
typedef struct {
  uint32_t struct_size;
  uint32_t n_layers, n_kv_heads, head_dim, elem_bytes, batch, p_max;
} phyai_kv_pack_desc_t;

phyai_status_t phyai_pack_prefix_kv(const phyai_kv_pack_desc_t *desc, const void *k, const void *v, const int32_t *lens,
                                    void *prefix_kv, uint64_t kv_tokens, int32_t *cu_prefix_lens, int32_t *status_word,
                                    void *stream);

/*
 * phyai_postprocess_actions: the raw chunk x at t = 0 -> robot actions (appendices on the pi0 / pi0.5 reproductions:
 * actions are clipped to [-1, 1] in normalised space and un-normalised with the checkpoint's q01 / q99 quantile
 * statistics; the controller uses the first out_horizon steps and out_dim action dimensions).
 *   out[b][h][a] = (clip(x[b][h][a], clip_lo, clip_hi) + 1) / 2 * (q99[a] - q01[a]) + q01[a],  h < out_horizon, a < out_dim
 *   x     device float32 [batch][horizon][action_dim];  out  device float32 [batch][out_horizon][out_dim]
 *   q01, q99   device float32 [>= out_dim], or both NULL (no un-normalisation: q01 = -1, q99 = 1)
 *   clip_lo >= clip_hi disables the clip.
 * Only enqueues work.  Errors: INVALID_ARG, CUDA.
 */
phyai_status_t phyai_postprocess_actions(const float *x, uint32_t batch, uint32_t horizon, uint32_t action_dim,
                                         const float *q01, const float *q99, float clip_lo, float clip_hi,
                                         uint32_t out_horizon, uint32_t out_dim, float *out, void *stream);

/*
 * phyai_project_features_kv: the request-local K / V projections of a feature-handoff action head (results section,
 * GR00T phase list: the action head contains "request-local cross-attention K/V projections"; the vision-language
 * features are fixed over the denoising steps, so their per-layer keys and values are computed once per request and
 * then serve as the loop's prefix KV; no rotary embedding on features).  K_l = F Wk_l, V_l = F Wv_l on the tensor cores.
 *   desc        n_layers, n_kv_heads, head_dim, feat_dim (a multiple of 64; 2 * n_kv_heads * head_dim a multiple of 128)
 *   features    device bfloat16 [tokens][feat_dim] row-major: the requests' feature rows, concatenated in the order
 *               of their prefix rows (cu_prefix_lens of the later denoise call)
 *   wk, wv      HOST arrays of n_layers DEVICE pointers, bfloat16 [feat_dim][n_kv_heads * head_dim] ([in, out])
 *   prefix_kv   device bfloat16 [n_layers][2][kv_tokens][n_kv_heads][head_dim]; rows [0, tokens) of every plane are
 *               written
 * Allocates its temporaries, runs on `stream` and synchronises it before returning (once per request batch, outside
 * the captured loop).  Errors: INVALID_ARG, OOM, CUDA, TIMEOUT.
 */
typedef struct {
  uint32_t struct_size;
  uint32_t n_layers, n_kv_heads, head_dim, feat_dim;
} phyai_kv_proj_desc_t;
phyai_status_t phyai_project_features_kv(const phyai_kv_proj_desc_t *desc, const void *features, const void *const *wk,
                                         const void *const *wv, uint64_t tokens, uint64_t kv_tokens, void *prefix_kv,
                                         void *stream);
/*
 * The same with the packed weight images and the workspace held in a handle: create packs the 2 * n_layers matrices
 * once (synchronises `stream`); run only enqueues kernels on `stream` (no allocation, no synchronisation; one run in
 * flight per handle) for up to max_tokens feature rows.  A bounded device-side wait that expired leaves rows unwritten;
 * the one-shot call above reports it, a projector's caller sees non-finite / stale rows downstream.
 */
typedef struct phyai_kv_projector phyai_kv_projector_t;
phyai_status_t phyai_kv_projector_create(const phyai_kv_proj_desc_t *desc, const void *const *wk, const void *const *wv,
                                         uint64_t max_tokens, void *stream, phyai_kv_projector_t **out);
phyai_status_t phyai_kv_projector_run(phyai_kv_projector_t *p, const void *features, uint64_t tokens, uint64_t kv_tokens,
                                      void *prefix_kv, void *stream);
void phyai_kv_projector_destroy(phyai_kv_projector_t *p);

/* Thread-local description of the last error of an adapter entry point. */
const char *phyai_adapter_last_error(void);

/*
 * Stand-alone W8A8 projection (quantization paragraph: W8A8, round-to-nearest): the activation quantization kernel
 * and the FP8 tensor-core GEMM that the PHYAI_W8A8_E4M3 loop uses, on one activation matrix.
 *   s[m]    = max_k |x[m][k]| / 448   (1 for an all-zero row), float32
 *   q[m][k] = e4m3 code nearest to x[m][k] / s[m] (ties to the even mantissa, saturating at +-448)
 *   y[m][n] = s[m] * w_scales[n] * sum_k value(q[m][k]) * value(w_codes[k][n]),  fp32 accumulation
 *   x_bf16        device bfloat16 [M][K] row-major (16-byte aligned)
 *   w_codes       device uint8 (e4m3) [K][N] row-major;  w_scales device float32 [N]
 *   y             device float32 [M][N]
 *   x_codes_out   device uint8 [M][K] or NULL: the activation codes;  x_scales_out device float32 [M] or NULL
 * 1 <= M <= 65536; K a multiple of 128, at most 4096; N a multiple of 128, at most 65536.  Allocates its temporaries,
 * runs on `stream` and synchronises it before returning (a verification entry point, not part of a serving loop).
 * Errors: INVALID_ARG, OOM, CUDA, TIMEOUT; message in phyai_w8a8_last_error().
 */
phyai_status_t phyai_w8a8_project(const void *x_bf16, const uint8_t *w_codes, const float *w_scales, uint32_t M,
                                  uint32_t K, uint32_t N, float *y, uint8_t *x_codes_out, float *x_scales_out,
                                  void *stream);
const char *phyai_w8a8_last_error(void);

/*
 * Data-parallel serving front-end, host side (Sec. "Parallel Execution": data-parallel runners exchange no state;
 * appendix on eight-GPU serving: rank 0 collects at most 32 pending observations, waits up to 20 ms for a batch to
 * fill, gives every worker a fixed local batch -- the shape its CUDA graph was captured for --, pads the local
 * inputs to that shape and drops the padded outputs after the gather).  No device work; thread-safe.
 *
 *   config   max_batch (most requests of one batch), n_workers x local_batch >= max_batch, window_ms >= 0
 *   submit   any thread: queue a request (an opaque 64-bit id chosen by the caller)
 *   next     the serving loop: blocks until a batch is due -- max_batch requests pending, or window_ms passed since
 *            the OLDEST pending request arrived -- or until timeout_ms have passed (then *n = 0).  ids: HOST array of
 *            max_batch entries, filled in arrival order.
 *   plan     pure function: slots[w * local_batch + j] = index into the batch (request for worker w, slot j) or -1
 *            (padding); requests fill the workers in order.  *active_workers = workers that hold a request.
 * Errors: INVALID_ARG (NULL, zero sizes, n_workers * local_batch < max_batch, n > max_batch), OOM.
 */
typedef struct phyai_batcher phyai_batcher_t;
typedef struct {
  uint32_t struct_size;
  uint32_t max_batch, n_workers, local_batch;
  double window_ms;
} phyai_batcher_config_t;

phyai_status_t phyai_batcher_create(const phyai_batcher_config_t *cfg, phyai_batcher_t **out);
void phyai_batcher_destroy(phyai_batcher_t *b);
phyai_status_t phyai_batcher_submit(phyai_batcher_t *b, uint64_t request_id);
phyai_status_t phyai_batcher_next(phyai_batcher_t *b, double timeout_ms, uint64_t *ids, uint32_t *n);
uint32_t phyai_batcher_pending(phyai_batcher_t *b);
phyai_status_t phyai_batcher_plan(const phyai_batcher_config_t *cfg, uint32_t n, int32_t *slots, uint32_t *active_workers);

/* Thread-local description of the last error of an operator entry point. */
const char *phyai_op_last_error(void);

/* Thread-local, NUL-terminated description of the last error on this thread ("" if none). */
const char *phyai_last_error(void);

/* Library version string. */
const char *phyai_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PHYAI_H_ */
