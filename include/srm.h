/*
 * srm.h — C ABI of the B200-native Structured Recurrent Mixer (SRM) decode library.
 *
 * What the library computes (paper sections in brackets):
 *   - the recurrent-form decode step over a batch of B independent samples: per layer a
 *     token-mixer cache update [Method/Architecture, Eq. 2 (row-repeat heads) and Eq. 3
 *     (column-repeat heads), "mixed" heads], then the channel-mixing feed-forward, then
 *     the LM head and token selection [Recurrent Throughput and Concurrency];
 *   - the sequence-parallel form over a prompt, which yields the same cache: the two forms
 *     share parameters and cache layout, so a model can switch between them at any position
 *     [Method/Architecture, Eq. 1 and Eq. 3].
 *
 * Conventions
 *   - Every pointer named d_* is a DEVICE pointer, 16-byte aligned unless stated; h_* is a
 *     HOST pointer. The library allocates no device memory: weights, state, workspace and
 *     token buffers are allocated by the caller and only borrowed. They must stay valid
 *     until the handle that borrowed them is destroyed (weights: srm_destroy; state buffer:
 *     srm_state_destroy; workspace and token buffers: until the stream work of the call ends).
 *   - `stream` is a cudaStream_t passed as void*. All device work is enqueued on it and the
 *     calls return without synchronising, except where stated.
 *   - All functions return 0 (SRM_OK) or a negative srm_error. No exceptions, no global
 *     mutable state besides the last CUDA error code and the launch counter (atomic). Handles
 *     are not thread-safe; distinct handles may be used from distinct threads.
 *   - Matrices are row-major [out, in]. Positions are absolute, 0-based; all samples of a
 *     state share one position counter.
 *   - The CUDA device current at srm_create is the one the handles belong to.
 */
#ifndef SRM_H_
#define SRM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct srm_model srm_model;   /* opaque host object; borrows the weight blob      */
typedef struct srm_state srm_state;   /* opaque host object; borrows the state buffer     */

enum srm_error {
  SRM_OK = 0,
  SRM_ERR_INVALID_ARG = -1,          /* null pointer, non-positive size, bad enum          */
  SRM_ERR_UNSUPPORTED = -2,          /* shape outside what the kernels support             */
  SRM_ERR_ALIGNMENT = -3,            /* a device pointer is not 16-byte (blob: 256) aligned */
  SRM_ERR_BUFFER_TOO_SMALL = -4,     /* weights / state / workspace smaller than required  */
  SRM_ERR_CTX_OVERFLOW = -5,         /* position would reach n_ctx (alpha, beta end there) */
  SRM_ERR_CUDA = -6,                 /* a CUDA call failed; see srm_last_cuda_error        */
  SRM_ERR_DEVICE_STATUS = -7,        /* srm_status found device-side flags set             */
  SRM_ERR_STATIC_SCRATCH = -8        /* batch needs more scratch than the built-in array holds */
};

/* Bits of the device status word (srm_status). Kernels never trap: they clamp, flag, go on. */
enum srm_status_bits {
  SRM_STATUS_TOKEN_RANGE = 1u,       /* a token id was outside [0, vocab); it was clamped  */
  SRM_STATUS_WAIT_TIMEOUT = 2u,      /* a bounded pipeline wait inside a GEMM gave up      */
  SRM_STATUS_NONFINITE = 4u          /* the sampler met a non-finite logit                 */
};

enum { SRM_DTYPE_FP32 = 0, SRM_DTYPE_BF16 = 1, SRM_DTYPE_FP16 = 2 /* cache storage only */ };
enum { SRM_SELECT_GREEDY = 0, SRM_SELECT_TOPK = 1, SRM_SELECT_TOPP = 2 };
enum {
  SRM_FLAG_NO_GRAPH = 4,             /* srm_generate never replays a captured step                     */
  SRM_FLAG_GRAPH = 8,                /* srm_generate always replays a captured step (default: only for
                                        batches small enough to be bound by the host's launch rate)     */
  SRM_FLAG_SIMT_GEMM = 1,            /* debug: run the bf16 GEMMs on the plain SIMT kernel  */
  SRM_FLAG_NO_SPLITK = 16,           /* the down projection of a decode step always gives whole output tiles to a CTA
                                        pair (see srm_k_gemm_splitk); for comparison and measurement */
  SRM_FLAG_NO_FUSED_TOPK = 32,       /* top-k selection always from fp32 logits written to the workspace (default: the
                                        candidates are collected inside the LM-head epilogue and no logits are written
                                        when the caller does not ask for them); for comparison and measurement */
  SRM_FLAG_NO_SMALL_BATCH = 64,      /* batches of at most 64 samples also run one kernel per operation (default: such a
                                        batch, on a bf16 mixed-head model of at most 1024 channels, runs its whole
                                        decode step in ONE cooperative kernel that streams the weights with all SMs;
                                        results agree with the other path to rounding, not bit for bit) */
  SRM_FLAG_NO_TAIL_SPLIT = 128,      /* tensor-core projections process every 256 x 256 tile whole (default: the tiles of a
                                        last, partly filled round run as two 256 x 128 pieces each, which keeps nearly all
                                        CTA pairs busy to the end); for comparison and measurement */
  SRM_FLAG_NO_FUSED_FFN = 256,       /* the feed-forward block of a decode step always runs as two launches, up projection
                                        then down projection (default, bf16 models whose d is a multiple of 256, passes
                                        of at most 16384 rows with at least two 256 x 256 tiles per CTA pair:
                                        ONE kernel computes the tiles of both projections, see srm_k_ffn; same results
                                        bit for bit); for comparison and measurement */
  SRM_FLAG_NO_KSLICE = 512,          /* the down projection of a small decode pass always adds whole tiles into x (default,
                                        where its tiles fill less than half of the CTA pairs, bf16 mixed-head models: the
                                        K dimension is cut into up to 8 ranges, one CTA pair each, and the next layer's
                                        mixer adds the partial products in a fixed order; results then differ in the
                                        last bits from those of a pass large enough not to be cut); for comparison */
  SRM_FLAG_HEAD_PROJ = 2             /* token mixer with head projections [Method/Architecture, Eq. 10]:
                                        q = W_in LN1(x) (W_in stacks the per-head I_g), heads of q mixed, and
                                        x += W_out (concatenated heads); the cache holds projected values.
                                        Adds W_in, W_out [d, d] per layer to the blob and 4 L d^2 flop per token */
};

/* Token mixer of the model [Method/Architecture].
 *   SRM_MIXER_MIXED     mixed heads: heads g < n_heads/2 row-repeat [Eq. 2], the rest column-repeat [Eq. 3], outputs
 *                       concatenated; the cache is d values per sample and layer (the default, and the hot path);
 *   SRM_MIXER_COMBINED  linearly combined heads: every head holds one row-repeat and one column-repeat matrix and
 *                       outputs w[g][0] * (row-repeat product) + w[g][1] * (column-repeat product) + beta; the cache
 *                       is both sum terms, 2 d values ("double the cache");
 *   SRM_MIXER_KERNEL    non-unitary kernels [Eq. 11]: kernel_size column-repeat filters over the whole hidden
 *                       dimension, filter i reading the channels shifted by i (zero past the last channel); the
 *                       cache is one sum term per filter, kernel_size * d values; alpha is [kernel_size, n_ctx] and
 *                       lambda [kernel_size] (n_heads is not used by the mixing).
 * The two further mixers run through fused step kernels of their own (warp per row); their sequence form is
 * evaluated through the recurrence, one launch per position over all prompts of a pass. They take the cache in
 * fp32 or fp16, d_model <= 1024, no head projections and no per-sample positions (srm_prefill_ragged). */
enum { SRM_MIXER_MIXED = 0, SRM_MIXER_COMBINED = 1, SRM_MIXER_KERNEL = 2 };

/* Model description. */
typedef struct {
  int32_t n_layers;      /* L >= 1                                                        */
  int32_t d_model;       /* d, multiple of 64, <= 2048                                    */
  int32_t n_heads;       /* h, even, 2 <= h <= 8, d % (4h) == 0                           */
  int32_t ffn_mult;      /* F = ffn_mult * d                                              */
  int32_t vocab;         /* V, multiple of 8                                              */
  int32_t n_ctx;         /* positions for which alpha/beta exist                          */
  int32_t dtype;         /* SRM_DTYPE_FP32: fp32 weights, plain fp32 FMA everywhere;
                            SRM_DTYPE_BF16: bf16 matrices and GEMM inputs, fp32 accumulate,
                            fp32 residual stream, norms and mixer arithmetic              */
  int32_t state_dtype;   /* storage type of the cache [Method/Architecture: the cache may be kept in half
                            precision]: SRM_DTYPE_FP32; SRM_DTYPE_FP16 (half the bytes per sample; values are
                            clamped to +-65504 when stored); SRM_DTYPE_BF16 (half the bytes; 8 significant bits:
                            in a decay-free head the rounding errors add up as a random walk, about 2^-9 sqrt(t)
                            of the cache after t steps, which leaves the bf16 logit tolerance after a few hundred
                            positions; for short contexts only)                           */
  float   ln_eps;        /* LayerNorm epsilon                                             */
  int32_t flags;         /* SRM_FLAG_* (0 in production)                                  */
  int32_t mixer;         /* SRM_MIXER_*                                                   */
  int32_t kernel_size;   /* SRM_MIXER_KERNEL: number of filters k, 1 <= k <= 16; else ignored */
} srm_config;

/* Token selection. Greedy: smallest id among the maxima. Top-k: keep the top_k largest logits
 * ordered by (logit desc, id asc), weights exp((l - l_max)/temperature), inverse-CDF draw with
 * u = (r >> 8) * 2^-24 where r is the first word of Philox4x32-10 with key (seed lo, seed hi)
 * and counter (sample_idx_base + b, step, 0, 0); 1 <= top_k <= 256.
 * Top-p (nucleus sampling, the sampler of the paper's GRPO rollouts [Training details: top-p 0.9,
 * temperature 0.7]): probabilities softmax(l / temperature); the nucleus is the shortest prefix of the
 * (logit desc, id asc) order whose probability reaches top_p; the token is drawn from the nucleus by
 * inverse CDF over ids in ascending order with the same u. Masses are summed as 64-bit fixed-point
 * integers (weight of the most probable token = 2^31), so the result does not depend on scheduling;
 * 0 < top_p <= 1. */
typedef struct {
  int32_t  mode;             /* SRM_SELECT_*                                               */
  int32_t  top_k;
  float    temperature;
  float    top_p;            /* SRM_SELECT_TOPP only                                       */
  uint64_t seed;
  uint64_t sample_idx_base;  /* Philox sample index of row 0 of the state                  */
} srm_sampling;

/* ---- sizes and weight-blob layout ------------------------------------------------------- */

/* Tensors of the weight blob, in blob order. Small vectors are always fp32; the four matrices
 * (E, W1, W2, W_LM) are fp32 or bf16 per config.dtype. Every tensor starts 256-byte aligned. */
enum srm_tensor {
  SRM_T_E = 0,        /* [V, d]    embedding (global: layer = -1)                          */
  SRM_T_LN1_G, SRM_T_LN1_B,          /* [d]  norm before the token mixer                   */
  SRM_T_ALPHA,        /* [h, n_ctx] repeated mixing weights alpha                          */
  SRM_T_BETA,         /* [n_ctx, d] per-position bias beta                                 */
  SRM_T_LAMBDA,       /* [h]       decay constants in (0.9, 1]                             */
  SRM_T_LN2_G, SRM_T_LN2_B,          /* [d]  norm before the feed-forward                  */
  SRM_T_W1,           /* [F, d]    up projection                                           */
  SRM_T_B1,           /* [F]                                                               */
  SRM_T_W2,           /* [d, F]    down projection                                         */
  SRM_T_B2,           /* [d]                                                               */
  SRM_T_LNF_G, SRM_T_LNF_B,          /* [d]  final norm (global)                           */
  SRM_T_W_LM,         /* [V, d]    LM head, no bias (global)                               */
  SRM_T_W_IN,         /* [d, d]    per layer, only with SRM_FLAG_HEAD_PROJ: rows g*d_h.. are I_g; placed
                                   after B2 in the layer's part of the blob                          */
  SRM_T_W_OUT,        /* [d, d]    per layer, only with SRM_FLAG_HEAD_PROJ: P_out                   */
  SRM_T_ALPHA_COL,    /* [h, n_ctx] SRM_MIXER_COMBINED only: weights of the column-repeat matrices (SRM_T_ALPHA then
                                   holds those of the row-repeat matrices); placed after the tensors above        */
  SRM_T_LAMBDA_COL,   /* [h]       SRM_MIXER_COMBINED only: decays of the column-repeat matrices                  */
  SRM_T_W_COMB,       /* [h, 2]    SRM_MIXER_COMBINED only: combination weights (row-repeat, column-repeat)       */
  SRM_T_COUNT
};

/* Total bytes of the weight blob, 0 if the config is invalid. */
size_t srm_weights_bytes(const srm_config* cfg);
/* Byte offset, byte size and element size of one tensor inside the blob (layer ignored for
 * the global tensors). Lets a caller fill the blob without knowing the layout rule. */
int srm_weight_slot(const srm_config* cfg, int32_t layer, int32_t tensor,
                    size_t* offset, size_t* nbytes, int32_t* elem_bytes);
/* Bytes of the state buffer for B samples: a 256-byte header (status word, counters), the
 * last selected token int32[B], the per-sample position int32[B] (used after srm_prefill_ragged), the
 * per-sample candidate threshold float[B] of the fused top-k selection, each rounded up to 256 bytes, then the
 * cache [L, C, B, d] in state_dtype, C = srm_cache_planes(cfg). */
size_t srm_state_bytes(const srm_config* cfg, int64_t B);
/* d-vectors of cache per sample and layer: 1 (mixed heads), 2 (combined heads), kernel_size (kernels). 0: bad config. */
int32_t srm_cache_planes(const srm_config* cfg);
/* Workspace bytes so that decode processes `B_chunk` samples per pass and prefill handles
 * prompts of up to `n_prefill_max` tokens in one pass of at least one sample. Calls accept any
 * workspace at least this large for B_chunk = 1 and split the batch into as many passes as
 * the given workspace requires. Decode never uses more than 12288 rows of it in one pass: a larger
 * batch runs as equal passes of at most 10240 rows (whole 256-row tiles), which keeps a layer's
 * activations in L2 between its kernels; results do not depend on the split, with two exceptions in the last bits:
 * a batch of at most 64 samples whose workspace holds it in one pass takes the single-kernel step (see
 * SRM_FLAG_NO_SMALL_BATCH), whose sums run in another order than those of the kernel-per-operation path; and a pass
 * small enough for its down projection to be cut along K (see SRM_FLAG_NO_KSLICE) adds that projection's partial
 * products in another order than a large pass, whatever batch it is part of. */
size_t srm_workspace_bytes(const srm_config* cfg, int64_t B_chunk, int32_t n_prefill_max);
/* Workspace bytes with which srm_prefill (and its variants) processes `samples` prompts of up to n tokens in one
 * pass [Eq. 1, Eq. 3: the sequence-parallel form over all positions of a pass]. A workspace for both calls is the
 * larger of this and srm_workspace_bytes(cfg, B_chunk, 0). 0: bad arguments. */
size_t srm_prefill_workspace_bytes(const srm_config* cfg, int64_t samples, int32_t n);
/* Rows per decode pass that a batch of B samples is processed in when the workspace has room for
 * `ws_rows` rows (the rule stated above; host only, no device work). 0 if B < 1 or ws_rows < 1. */
int64_t srm_decode_pass_rows(int64_t B, int64_t ws_rows);

/* ---- handles ------------------------------------------------------------------------------ */

/* Validates cfg, records tensor addresses inside the caller's blob (256-byte aligned,
 * nbytes >= srm_weights_bytes) and prepares TMA descriptors for the weight matrices. */
int srm_create(const srm_config* cfg, const void* d_weights, size_t nbytes, srm_model** out);
int srm_destroy(srm_model* m);

/* Binds a caller buffer of >= srm_state_bytes(cfg, B) bytes as the state of B samples and
 * enqueues its zero-fill (cache = 0, position = 0) on `stream`. */
int srm_state_create(srm_model* m, int64_t B, void* d_state, size_t nbytes, void* stream,
                     srm_state** out);
int srm_state_destroy(srm_state* s);
int srm_state_reset(srm_state* s, void* stream);
/* Position bookkeeping (host side): number of tokens consumed so far. */
int64_t srm_state_pos(const srm_state* s);
int srm_state_set_pos(srm_state* s, int64_t pos);
/* For a state whose buffer was copied from a state left by srm_prefill_ragged (checkpoint / resume): declares
 * that the per-sample position vector inside the buffer is valid and that the longest sample stands at
 * max_pos (what srm_state_pos reported for the source state). From then on the state behaves as the source. */
int srm_state_adopt_positions(srm_state* s, int64_t max_pos);
/* 1 when the state keeps one position per sample (after srm_prefill_ragged or srm_state_adopt_positions). */
int srm_state_is_ragged(const srm_state* s);
/* Device address of the cache slab of one layer, [C, B, d] in state_dtype (for checkpointing
 * and tests), and of the last-token vector int32[B]. */
void* srm_state_layer_ptr(const srm_state* s, int32_t layer);
int32_t* srm_state_last_token_ptr(const srm_state* s);
/* Fused top-k selection [Recurrent Throughput and Concurrency: choosing the next tokens from the logits is the
 * step the paper measures as its large-batch bottleneck]. With SRM_SELECT_TOPK, top_k <= 160, V >= 2048, the
 * tensor-core path and no logits requested, srm_decode_step / srm_generate collect, inside the LM-head epilogue,
 * every logit of a row at or above that row's threshold and select among those: no logits reach HBM. The set is
 * exact whenever it holds at least top_k logits. The threshold of a sample is carried from one selection to its
 * next (float[B] in the state buffer; all-zero bits = none yet) and aims at about max(192, 3 top_k) candidates. A
 * row with no threshold, fewer than top_k candidates or more than 1024 is handed back: its logits alone are
 * recomputed into the workspace and it goes through the same kernels as the logits path, so ids are identical to
 * that path in every case. The two calls below expose the threshold vector (device pointer, for tests and
 * checkpoints) and the number of rows handed back since the state was last reset (synchronises `stream`). */
float* srm_state_topk_threshold_ptr(const srm_state* s);
int srm_state_topk_handed_back(srm_state* s, void* stream, uint64_t* rows);
/* Synchronises `stream`, copies the device status word to *flags and clears it.
 * Returns SRM_ERR_DEVICE_STATUS when any bit was set. */
int srm_status(srm_state* s, void* stream, uint32_t* flags);

/* ---- the hot path ------------------------------------------------------------------------- */

/* Sequence-parallel prefill [Eq. 1, Eq. 3]: consumes d_tokens[B, n] (row-major int32) at
 * positions 0..n-1 of a freshly reset state, leaves the cache that position n reads and
 * pos = n, and selects generated token 0 from the logits of position n-1 (Philox step 0).
 * d_first_tok int32[B] and d_logits_last float[B, V] may be NULL. */
int srm_prefill(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n,
                const srm_sampling* sampling, int32_t* d_first_tok, float* d_logits_last,
                void* d_ws, size_t ws_bytes, void* stream);

/* Prefill of prompts of different lengths (a serving batch). d_tokens int32[B, n_max] holds the prompts
 * left-aligned, sample b uses its first d_lengths[b] tokens (1 <= length <= n_max; the rest of the row must
 * still hold valid token ids, they are not used). Each sample's cache is the one its own length leaves
 * [Eq. 1, Eq. 3 on its own positions], its first generated token comes from the logits of its last prompt
 * position, and from here on the state keeps ONE POSITION PER SAMPLE on the device: srm_decode_step,
 * srm_generate and the other step calls read alpha_t, beta_t at each sample's own t and advance it, so
 * sample b behaves exactly as if it had been prefilled and decoded alone. srm_state_pos then reports the
 * position of the longest sample (the one that reaches n_ctx first) and srm_state_set_pos is refused.
 * Lengths outside [1, n_max] are clamped to that range (the prefill and the positions kept for the decode
 * steps use the clamped value) and reported through srm_status (SRM_STATUS_TOKEN_RANGE). */
int srm_prefill_ragged(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n_max,
                       const int32_t* d_lengths, const srm_sampling* sampling, int32_t* d_first_tok,
                       float* d_logits_last, void* d_ws, size_t ws_bytes, void* stream);

/* Prefill for replicated prompts [Inference Compute Scaling: many samples per question, as in the
 * GRPO rollouts]: d_tokens holds n_prompts DISTINCT prompts [n_prompts, n]; the state has
 * B = n_prompts * replicas samples and sample p * replicas + j is replica j of prompt p. Every prompt runs
 * through the sequence-parallel form once, its cache is copied to the rows of its replicas, and each
 * replica selects its own first token from the prompt's last-position logits (Philox sample index
 * sample_idx_base + state row, step 0), which is what srm_prefill on the replicated token matrix gives, bit
 * for bit. d_first_tok int32[B] and d_logits_last float[n_prompts, V] may be NULL. Needs, on top of the
 * prefill workspace, L * d * state element bytes (rounded up to 256) per prompt of a pass at the end of d_ws. */
int srm_prefill_replicated(srm_model* m, srm_state* s, const int32_t* d_tokens, int32_t n_prompts, int32_t n,
                           int32_t replicas, const srm_sampling* sampling, int32_t* d_first_tok,
                           float* d_logits_last, void* d_ws, size_t ws_bytes, void* stream);

/* One recurrent decode step [Eq. 2, Eq. 3]: consumes d_tok_in[B] (NULL: the token selected
 * by the previous call) at position pos, updates the cache, pos += 1, and selects the next
 * token with Philox step `step`. d_tok_out int32[B] and d_logits_out float[B, V] may be NULL. */
int srm_decode_step(srm_model* m, srm_state* s, const int32_t* d_tok_in,
                    const srm_sampling* sampling, int32_t step, int32_t* d_tok_out,
                    float* d_logits_out, void* d_ws, size_t ws_bytes, void* stream);

/* Generation loop [Recurrent Throughput and Concurrency; the paper moved its loop inside the compiled graph
 * to escape a per-call driver delay]: `steps` decode steps, each consuming the previously selected token
 * (the one left by srm_prefill or the previous step). Step j (0-based) writes its selection
 * to d_out[b * out_stride + j] and uses Philox step first_step + j. No host synchronisation
 * between steps. Fails with SRM_ERR_CTX_OVERFLOW before enqueuing anything if
 * pos + steps > n_ctx. For batches small enough to be bound by the host's kernel-launch rate one step is
 * captured once as a CUDA graph (on a stream the model owns; position, Philox step and store column live
 * in device-side counters of the state header that a one-thread kernel advances) and replayed `steps`
 * times on `stream`; the graph is kept and reused while state, workspace, sampling and output buffer stay
 * the same. Results are identical to the launch-by-launch loop. */
int srm_generate(srm_model* m, srm_state* s, int32_t steps, int32_t first_step,
                 const srm_sampling* sampling, int32_t* d_out, int64_t out_stride,
                 void* d_ws, size_t ws_bytes, void* stream);

/* Same step as srm_decode_step with HOST token buffers (pinned memory recommended):
 * copies h_tok_in[B] to the device, runs the step, copies the selection to h_tok_out[B], all
 * on `stream`; the caller synchronises the stream before reading h_tok_out. */
int srm_decode_step_host(srm_model* m, srm_state* s, const int32_t* h_tok_in,
                         const srm_sampling* sampling, int32_t step, int32_t* h_tok_out,
                         void* d_ws, size_t ws_bytes, void* stream);

/* Decode step for callers that cannot allocate device memory. (The paper has no counterpart:
 * this is a packaging variant of srm_decode_step, not a step of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plug-in inside a host
 * application that reserved the whole device up front, a latency-critical loop that must not
 * take cudaMalloc's implicit device-wide synchronisation, a callback that is only allowed to
 * enqueue work. Such a caller still owns its inputs and outputs (weights, state, token buffers);
 * what it cannot provide is the per-step workspace (residual stream, activations, hidden layer,
 * logits). Here that workspace is an array of SRM_STATIC_SCRATCH_BYTES that is part of the
 * library image itself: every GPU that loads libsrm.so holds these bytes until the process
 * exits, whether or not this call is ever used.
 *
 * Same arguments and results as srm_decode_step, minus the workspace. Differences:
 *   - the whole batch must fit in one pass: if srm_workspace_bytes(cfg, B, 0) exceeds
 *     SRM_STATIC_SCRATCH_BYTES the call enqueues nothing and returns SRM_ERR_STATIC_SCRATCH
 *     (e.g. the mid model, 142 KB per row next to 10.6 MB of fixed scratch, takes up to about 160 rows; the tiny
 *     model about 13 000);
 *   - the device that is current must be the model's device (else SRM_ERR_INVALID_ARG);
 *   - the first call on each device looks up the array's device address (cudaGetSymbolAddress).
 *     Make that first call outside of any stream capture; later calls only enqueue kernels;
 *   - no cudaMalloc, cudaFree or other allocating routine is called, on any call;
 *   - every call on a device shares the one array. It keeps whatever the previous call left
 *     there; the step overwrites (or clears, on the stream) every byte it later reads, so the caller has nothing to clear. Two
 *     calls whose GPU work can overlap (different streams, or different host threads without
 *     ordering) race on the array and produce garbage: serialise them on one stream. */
#define SRM_STATIC_SCRATCH_BYTES (32u << 20)
int srm_decode_step_static(srm_model* m, srm_state* s, const int32_t* d_tok_in,
                           const srm_sampling* sampling, int32_t step, int32_t* d_tok_out,
                           float* d_logits_out, void* stream);

/* ---- single kernels, exported for unit parity tests and profiling ------------------------- */

/* Fused token-mixer step of one layer on R rows at position t [Eq. 2, Eq. 3]:
 *   x <- (d_tok != NULL ? E[tok] : x);  z = LN1(x);  y, S' = mixer(z, S, t);  x <- x + y;
 *   a = LN2(x) in the activation type of cfg.dtype.
 * d_x float[R, d] in/out, d_S [R, d] in state_dtype in/out ([C, R, d] for the further mixers), d_a [R, d] out. */
int srm_k_mixer_step(srm_model* m, int32_t layer, int32_t t, int64_t R, const int32_t* d_tok,
                     float* d_x, void* d_S, void* d_a, uint32_t* d_status, void* stream);
/* Recurrent step of a layer with LINEARLY COMBINED heads [Architecture: every head holds one row-repeat and
 * one column-repeat matrix, the two products are combined linearly; twice the cache] on R rows of normed
 * inputs at position t, fp32, no model handle (all arrays are the caller's device memory, 16-byte aligned):
 *   y     = w[g][0] (alpha_row[g][t] z + S_row) + w[g][1] alpha_col[g][t] (z + S_col) + beta[t]   [Eq. 2, Eq. 3]
 *   S_row <- lam_row[g] (S_row + alpha_row[g][t] z);   S_col <- lam_col[g] (S_col + z)
 * for head g = channel / (d / n_heads). d_z, d_y float[R, d]; d_S_row, d_S_col float[R, d] in/out;
 * d_alpha_row, d_alpha_col float[n_heads, n_ctx]; d_beta float[n_ctx, d]; d_lam_row, d_lam_col float[n_heads];
 * d_w float[n_heads, 2]. d / n_heads must be a multiple of 4 (SRM_ERR_UNSUPPORTED); t >= n_ctx is
 * SRM_ERR_CTX_OVERFLOW. Asynchronous on `stream`. */
int srm_k_mixer_combined_step(int64_t R, int32_t d, int32_t n_heads, int32_t t, int32_t n_ctx, const float* d_z,
                              float* d_S_row, float* d_S_col, const float* d_alpha_row, const float* d_alpha_col,
                              const float* d_beta, const float* d_lam_row, const float* d_lam_col, const float* d_w,
                              float* d_y, void* stream);
/* Recurrent step of a layer with a NON-UNITARY KERNEL of size k [Eq. 11: k column-repeat filters, filter i
 * applied to the hidden channels shifted by i, X zero-padded past its last channel, stride 1], fp32:
 *   v_i = z + P_i;   y[c] = sum_{i < k, c + i < d} alpha[i][t] v_i[c + i] + beta[t][c];   P_i <- lam[i] v_i
 * d_z, d_y float[R, d]; d_P float[k, R, d] in/out (the sum term of Eq. 3 per filter: k times the cache);
 * d_alpha float[k, n_ctx]; d_beta float[n_ctx, d]; d_lam float[k]. Needs d % 4 == 0, k <= 16, k <= d and
 * k * d * 4 bytes of shared memory within 200 KB, else SRM_ERR_UNSUPPORTED. Asynchronous on `stream`. */
int srm_k_mixer_kernel_step(int64_t R, int32_t d, int32_t k, int32_t t, int32_t n_ctx, const float* d_z, float* d_P,
                            const float* d_alpha, const float* d_beta, const float* d_lam, float* d_y, void* stream);
/* The same two variants over whole sequences (the prefill form, evaluated through the recurrence): d_Z, d_Y
 * float[Bp, n, d] hold positions t0 .. t0 + n - 1 of Bp samples; the caches (d_S_row, d_S_col float[Bp, d];
 * d_P float[k, Bp, d]) enter as the sum terms for position t0 (zeros for a fresh prompt) and leave as those for
 * position t0 + n. Equal to the product with the explicit n x n matrices [Eq. 1, Eq. 3, Eq. 11] up to rounding
 * order. Parameters as in the step calls; t0 + n > n_ctx is SRM_ERR_CTX_OVERFLOW; the kernel-size-k call needs
 * (2 k + 8) d * 4 bytes of shared memory within 200 KB (SRM_ERR_UNSUPPORTED). */
int srm_k_mixer_combined_scan(int64_t Bp, int32_t n, int32_t t0, int32_t d, int32_t n_heads, int32_t n_ctx, const float* d_Z,
                              float* d_S_row, float* d_S_col, const float* d_alpha_row, const float* d_alpha_col,
                              const float* d_beta, const float* d_lam_row, const float* d_lam_col, const float* d_w,
                              float* d_Y, void* stream);
int srm_k_mixer_kernel_scan(int64_t Bp, int32_t n, int32_t t0, int32_t d, int32_t k, int32_t n_ctx, const float* d_Z, float* d_P,
                            const float* d_alpha, const float* d_beta, const float* d_lam, float* d_Y, void* stream);
/* out = LN_f(x) in the activation type: d_x float[R, d] -> d_a [R, d]. */
int srm_k_final_norm(srm_model* m, int64_t R, const float* d_x, void* d_a, void* stream);
/* Dense projection D[M, N] = A[M, K] * W[N, K]^T with one of three epilogues:
 *   0: out_act[M, N] = gelu_erf(D + bias)      (activation type)
 *   1: out_f32[M, N] += D + bias               (fp32 residual stream; d_bias may be NULL: no bias)
 *   2: out_f32[M, N] = D                       (fp32 logits)
 * A, W in the activation type of cfg.dtype; bf16 runs on the tcgen05 tensor-core kernel
 * (or the SIMT kernel when cfg.flags has SRM_FLAG_SIMT_GEMM), fp32 on the SIMT kernel. */
int srm_k_gemm(srm_model* m, int32_t epilogue, int64_t M, int64_t N, int64_t K, const void* d_A,
               const void* d_W, const float* d_bias, void* d_out, uint32_t* d_status,
               void* stream);
/* Epilogue 1 of srm_k_gemm (out_f32[M, N] += A W^T + bias, bf16 tensor-core path) with the K dimension shared out
 * between CTA pairs: the (256 x 256 tile, 64-wide k-block) sequence is cut into one contiguous range per pair, so
 * that no pair idles when the tile count is not a multiple of the pair count [the down projection of the
 * feed-forward: x += H W2^T + b2]. A tile is cut at most once; its two partial products are added in a fixed
 * order (upper k-range first), so the result is reproducible; it differs from srm_k_gemm's in the last bits.
 * This is what srm_decode_step and srm_generate run for the down projection when it is the faster kernel (a long
 * K and a partly empty last round: 192 tiles of 96 k-blocks on 74 pairs, the rollout model; with 64 or 128
 * tiles of 64 k-blocks the extra epilogues cost more than the shorter ranges save, and the unsplit kernel stays). d_order: scratch of srm_k_gemm_splitk_order_bytes(M, N) bytes, 256-byte aligned,
 * cleared by the call. SRM_ERR_UNSUPPORTED when the shape does not call for a split (the tiles fill whole
 * rounds, or there are fewer than half as many tiles as pairs): use srm_k_gemm then. */
size_t srm_k_gemm_splitk_order_bytes(int64_t M, int64_t N);
int srm_k_gemm_splitk(srm_model* m, int64_t M, int64_t N, int64_t K, const void* d_A, const void* d_W,
                      const float* d_bias, float* d_out, void* d_order, size_t order_bytes,
                      uint32_t* d_status, void* stream);
/* The work list of CTA pair `pair` of `pairs` in srm_k_gemm_splitk: up to max_pieces entries of four int64
 * {tile row, tile column, first k-block, end k-block} written to the HOST array `pieces`. Returns the number
 * of pieces of that pair, or a negative SRM_ERR_* (SRM_ERR_UNSUPPORTED: no split for this shape). Pure host
 * arithmetic: needs no device. */
int64_t srm_k_gemm_splitk_plan(int64_t M, int64_t N, int64_t K, int32_t pairs, int32_t pair,
                               int64_t* pieces, int64_t max_pieces);
/* The feed-forward block of layer `layer` on M rows as one kernel [Method/Architecture: the channel-mixing
 * feed-forward that follows the token mixer]: H = gelu(a W1^T + b1), x += H W2^T + b2. d_a [M, d] bf16 in, d_H [M, F]
 * bf16 out (scratch of the block), d_x [M, d] fp32 in/out. The 256 x 256 tiles of BOTH projections are dealt to the
 * CTA pairs by a host-made plan (srm_k_ffn_plan); a down tile reads H column tile after column tile along its K
 * dimension and waits, per column tile, for a counter the epilogue warps of that up tile raise, so pairs with a down
 * tile start it while other pairs still compute up tiles of the same rows, and no pair idles through the down
 * projection. Results equal srm_k_gemm (epilogue 0) followed by srm_k_gemm (epilogue 1) bit for bit. d_ready: scratch
 * of srm_k_ffn_ready_bytes(M, F) bytes, 256-byte aligned, cleared by the call. The CTA pairs of the launch wait for
 * one another: do not run it concurrently with other work on the same device (it then may time out: status bit
 * SRM_STATUS_WAIT_TIMEOUT, result invalid). SRM_ERR_UNSUPPORTED: not a bf16 tensor-core model, d or F not a multiple of
 * 256, more than 16384 rows or more than 2048 tiles. This is what srm_decode_step and srm_generate run per layer
 * for passes with at least two tiles per CTA pair (mid model: from 2048 rows), unless
 * SRM_FLAG_NO_FUSED_FFN is set. */
size_t srm_k_ffn_ready_bytes(int64_t M, int64_t F);
int srm_k_ffn(srm_model* m, int32_t layer, int64_t M, const void* d_a, void* d_H, float* d_x, void* d_ready,
              size_t ready_bytes, uint32_t* d_status, void* stream);
/* The work lists of srm_k_ffn for M rows of a model of width d and hidden width F on `pairs` CTA pairs, written to
 * HOST arrays: off[pairs + 1] (pair c owns items off[c] .. off[c + 1] - 1, in this order) and up to max_items items
 * of three int32 {0 = up tile / 1 = down tile / 2, 3 = first, second 256 x 128 half of an up tile, row block, column
 * tile}. Returns the number of items (every tile of both projections exactly once, some up tiles as two halves), or a negative SRM_ERR_*. *makespan / *ideal (may be NULL): the plan's length and
 * the even-share lower bound under the cost model of the planner, in k-block times. Pure host arithmetic: needs no
 * device. */
int64_t srm_k_ffn_plan(int64_t M, int32_t d, int32_t F, int32_t pairs, int32_t* off, int32_t* items, int64_t max_items,
                       double* makespan, double* ideal);
/* LM head with greedy selection fused into the GEMM epilogue (bf16 models only): d_tok[r] =
 * argmax_v (a[r, :] . W_lm[v, :]), lowest id among equal maxima - the token srm_k_gemm (epilogue 2)
 * followed by greedy srm_k_select gives, without writing the R x V logits. d_a [R, d] in the
 * activation type; d_part is scratch of part_bytes >= ceil(V / 256) * 4 * R * 8 bytes, 16-byte aligned.
 * This is the path srm_decode_step, srm_generate and srm_prefill take for greedy sampling when the
 * caller does not ask for logits [Recurrent Throughput and Concurrency: finding the next tokens from the
 * logits is the bottleneck the paper measures at large batch]. */
int srm_k_lm_head_greedy(srm_model* m, int64_t R, const void* d_a, void* d_part, size_t part_bytes,
                         int32_t* d_tok, uint32_t* d_status, void* stream);
/* Token selection on d_logits float[R, V] -> d_tok int32[R]; row r uses sample index
 * sampling->sample_idx_base + r. */
int srm_k_select(srm_model* m, int64_t R, const float* d_logits, const srm_sampling* sampling,
                 int32_t step, int32_t* d_tok, uint32_t* d_status, void* stream);
/* Sequence-parallel token mixing of one layer for Bp samples of n positions [Eq. 1, Eq. 3]:
 * x[Bp*n, d] in/out (row = b*n + position), a[Bp*n, d] out, cache S[Bp, d] out (the sum term
 * position n reads). d_tok (int32[Bp*n]) non-NULL: rows start from the embedding. */
int srm_k_prefill_mixer(srm_model* m, int32_t layer, int64_t Bp, int32_t n, const int32_t* d_tok,
                        float* d_x, void* d_S, void* d_a, uint32_t* d_status, void* stream);

/* Failure-detection check without a fault: launches one thread that waits, with the bounded wait all pipelines of
 * this library use, on a barrier that nothing completes. After limit_cycles (1 .. 2^31 SM clock cycles) the wait
 * gives up, SRM_STATUS_WAIT_TIMEOUT is raised in *d_status, *d_gave_up (may be NULL) is set to 1 and the kernel ends;
 * the context stays usable. Asynchronous on `stream`. */
int srm_k_wait_probe(uint32_t* d_status, int64_t limit_cycles, int32_t* d_gave_up, void* stream);

/* ---- measurement -------------------------------------------------------------------------- */
enum srm_kernel_class {
  SRM_KERNEL_MIXER = 0,          /* fused recurrent token-mixer step                           */
  SRM_KERNEL_GEMM_UP,            /* feed-forward up projection (+bias, GELU)                   */
  SRM_KERNEL_GEMM_DOWN,          /* feed-forward down projection (+bias, residual)             */
  SRM_KERNEL_GEMM_LM,            /* LM head                                                    */
  SRM_KERNEL_NORM,               /* final norm                                                 */
  SRM_KERNEL_SELECT,             /* token selection                                            */
  SRM_KERNEL_PREFILL_MIXER,      /* sequence-parallel token mixing                             */
  SRM_KERNEL_GEMM_PROJ,          /* head projections W_in, W_out (SRM_FLAG_HEAD_PROJ)          */
  SRM_KERNEL_STEP_SMALL,         /* the single-kernel decode step of a small batch             */
  SRM_KERNEL_FFN,                /* feed-forward block as one kernel (up and down projection)  */
  SRM_KERNEL_CLASS_COUNT
};
/* While enabled, every kernel launch of this model is bracketed by two CUDA events recorded on the
 * launching stream (events are created on first need and reused; no device memory). */
int srm_profile_enable(srm_model* m, int on);
/* Waits for the recorded events, folds them into per-class totals and returns the number of
 * launches and the summed device time (ms) of one class since the last reset. */
int srm_profile_read(srm_model* m, int32_t kernel_class, uint64_t* launches, double* total_ms);
int srm_profile_reset(srm_model* m);
/* Number of kernels this library has launched since it was loaded (all models). */
uint64_t srm_kernel_launches(void);

/* ---- diagnostics -------------------------------------------------------------------------- */
const char* srm_strerror(int code);
int srm_last_cuda_error(void);        /* cudaError_t of the most recent SRM_ERR_CUDA       */
const char* srm_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SRM_H_ */
