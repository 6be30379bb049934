/*
 * sps.h -- C ABI of the B200 speculative-sampling library (libsps_b200.so).
 *
 * The library implements the hot path of speculative sampling (Chen et al.,
 * "Accelerating Large Language Model Decoding with Speculative Sampling"):
 * K single-row draft-model steps, one (K+1)-row target-model scoring pass and
 * the modified rejection sampler, as CUDA kernels for sm_100a.  Notation is
 * the paper's: q = TARGET model, p = DRAFT model, K = lookahead.
 *
 * Conventions
 *   - every function returns an int status: SPS_OK (0) or a negative error.
 *     Nothing throws, aborts or prints.  sps_last_error() describes the last
 *     failure on a handle (or, with a NULL handle, of the handle-less calls).
 *   - "host" / "device" in a comment says where the pointer must point.
 *   - weight and logit buffers passed in are caller-owned and never written
 *     unless stated; the handle owns its KV caches, work buffers and graphs.
 *   - one handle = one CUDA stream; calls on a handle are not re-entrant.
 *
 * Random numbers.  Algorithm 2 draws r ~ U[0,1] and samples tokens; this
 * library fixes the generator so results can be reproduced elsewhere:
 * Philox4x32-10, key = (seed low 32, seed high 32), counter =
 * (t, s, b, 0) with t the position inside the loop (0..K-1 drafts, K the extra
 * token), s the loop index, b the sequence index.  Word 0 -> u_draft (draw of
 * draft token t), word 1 -> u_acc (accept test), word 2 -> u_res (resample at
 * t, or extra-token draw at t = K).  u = (word >> 8) * 2^-24.
 * Every draw is an inverse-CDF draw in index order on unnormalised weights.
 */
#ifndef SPS_B200_H
#define SPS_B200_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPS_OK 0
#define SPS_EINVAL (-1)   /* bad argument or unsupported shape                     */
#define SPS_ENOMEM (-2)   /* device or host allocation failed                      */
#define SPS_ECUDA (-3)    /* a CUDA call failed; sps_last_error has its message    */
#define SPS_ERANGE (-4)   /* token id >= vocab, or sequence would exceed max_seq   */
#define SPS_ESTATE (-5)   /* call order (e.g. step before prefill)                 */
#define SPS_ETIMEOUT (-6) /* a bounded device-side wait ran out                    */

#define SPS_MAX_K 15      /* K + 1 rows <= 16 per sequence                         */

/* sps_accept / sps_step flag bits (per sequence) */
#define SPS_FLAG_RESAMPLED 1u /* a draft was rejected; token drawn from norm(max(0, q - p)) */
#define SPS_FLAG_BONUS 2u     /* all K drafts accepted; extra token drawn from q_{K+1}       */
#define SPS_FLAG_FALLBACK 4u  /* rejected with sum max(0, q - p) == 0: token drawn from q_t  */
#define SPS_FLAG_TIMEOUT 8u   /* sps_accept only: a bounded wait inside the kernel ran out; this
                                 sequence's outputs are meaningless (handle calls return SPS_ETIMEOUT) */

/* sps_cfg.flags */
#define SPS_CFG_NO_GRAPH 1u   /* launch kernels one by one instead of replaying CUDA graphs  */
#define SPS_CFG_TENSOR_PARALLEL 2u /* the weights are one rank's shard of both models (see sps_tp_attach) */

typedef struct sps_handle sps_handle;

/* One decoder-only transformer: pre-RMSNorm, multi-head attention with
 * n_heads * d_head == d_model, rotary positions on adjacent pairs over the
 * whole head, non-gated FFN with tanh-GeLU, no biases, untied (un)embedding.
 * (The paper's Hyperparams table fixes d_model / heads / layers only.)
 * n_kv_heads: key / value heads; 0 or n_heads = one per query head.  A divisor
 * of n_heads below it gives grouped-query attention, 1 multi-query attention
 * (Related Work: multi-query attention shrinks the key / value cache;
 * Conclusion: it combines with this method, which leaves the transformer
 * body alone): query head h attends
 * over key / value head h / (n_heads / n_kv_heads), wk and wv have
 * n_kv_heads * d_head rows, and the cache holds that many numbers per position.
 * dtype: 0 = fp32, 1 = bf16; it is the storage type of the weight matrices,
 * the embeddings and the KV cache.  Norm gains are always fp32.
 * dtype 2 = weight-only int8: the linear layers' matrices (wq .. w_down and the
 * unembedding) are signed bytes with one fp32 scale per output row,
 * w[n][k] = scale[n] * byte[n][k] (sps_weights' *_scale members); the token
 * embedding and the KV cache stay bf16.  (The paper notes that quantisation
 * composes with speculative sampling, since the method does not touch the
 * transformer body; half the bytes per weight halve the floor of every pass.)
 * bf16 / int8 models need d_model and d_ff to be multiples of 128; d_head is 64 or 128. */
typedef struct {
  int32_t n_layers, d_model, n_heads, d_head, d_ff, vocab;
  int32_t dtype;
  float rms_eps, rope_base;
  int32_t n_kv_heads;
} sps_model_cfg;

typedef struct {
  sps_model_cfg target, draft;
  int32_t max_seq;   /* longest sequence (prompt + generated + K) a cache row exists for */
  int32_t max_batch; /* sequences decoded together, <= 8; max_batch * (max_K + 1) <= 16,
                        or <= 128 when the target is bf16 (passes above 16 rows run
                        their linear layers as tensor-core GEMMs)                        */
  int32_t max_K;     /* largest lookahead that will be asked for, <= SPS_MAX_K           */
  int32_t device;    /* CUDA device ordinal                                              */
  void* stream;      /* cudaStream_t to run on; NULL = the library creates its own       */
  uint32_t flags;    /* SPS_CFG_*                                                        */
} sps_cfg;

/* Weights of one model.  All pointers are DEVICE pointers, borrowed for the
 * life of the handle and never written.  Matrices are row-major [out, in]
 * (y = W x), in the model's dtype.  The per-layer members are HOST arrays of
 * n_layers device pointers. */
typedef struct {
  const void* tok_embed;  /* [vocab, d_model]            */
  const void* unembed;    /* [vocab, d_model]            */
  const void* final_norm; /* [d_model] fp32              */
  const void* const* attn_norm; /* each [d_model] fp32   */
  const void* const* ffn_norm;  /* each [d_model] fp32   */
  const void* const* wq;        /* each [d_model, d_model] */
  const void* const* wk;        /* each [n_kv_heads * d_head, d_model] */
  const void* const* wv;
  const void* const* wo;
  const void* const* w_up;      /* each [d_ff, d_model]  */
  const void* const* w_down;    /* each [d_model, d_ff]  */
  /* dtype 2 only (NULL otherwise): fp32 row scales, 16-byte aligned, one per output row of the matrix */
  const float* unembed_scale;        /* [vocab]               */
  const float* const* wq_scale;      /* each [d_model]        */
  const float* const* wk_scale;      /* each [n_kv_heads * d_head] */
  const float* const* wv_scale;
  const float* const* wo_scale;
  const float* const* w_up_scale;    /* each [d_ff]           */
  const float* const* w_down_scale;  /* each [d_model]        */
} sps_weights;

/* What a generation did (the Results section counts the tokens each
 * speculative loop produced; so does this). */
typedef struct {
  int32_t loops;         /* target calls                                             */
  int32_t draft_calls;   /* draft forward passes                                     */
  int32_t emitted;       /* tokens produced before truncation to n_new               */
  int32_t accepted;      /* draft tokens accepted                                    */
  int32_t resampled;     /* loops that ended in a residual resample                  */
  int32_t bonus;         /* loops that accepted all K drafts and drew the extra token */
  int32_t fallback;      /* loops that took the sum max(0, q-p) == 0 fallback         */
  int32_t overshoot;     /* tokens of the last loop dropped to return exactly n_new  */
  int32_t hist_emitted[SPS_MAX_K + 2]; /* hist_emitted[j] = loops that emitted j tokens */
  float ms_prefill;      /* device time of the prompt pass                           */
  float ms_decode;       /* device time from the first loop's start to the last loop's end,
                            host turnaround between loops included                   */
  float ms_draft, ms_verify, ms_accept; /* device time inside the three phases       */
  int32_t kernel_launches; /* kernels the loops launched (graph nodes counted per replay) */
} sps_stats;

/* Build a handle for a (target, draft) pair: the target model q and the draft
 * model p of Algorithm 2's preamble.  draft_w may be NULL, then
 * only K = 0 (Algorithm 1) is available.  Allocates the KV caches
 * [layer][sequence][head][position][d_head] in the model dtype, work buffers
 * and rotary tables on cfg->device.  *out receives the handle. */
int sps_create(const sps_weights* target_w, const sps_weights* draft_w, const sps_cfg* cfg, sps_handle** out);
int sps_destroy(sps_handle* h);
/* NUL-terminated text owned by the handle (or by the library when h is NULL). */
const char* sps_last_error(sps_handle* h);

/* Algorithm 2 (K >= 1) or Algorithm 1 (K == 0) for one sequence: ingest the
 * prompt, then loop { draft K tokens; score K+1 positions; accept / resample /
 * extra token } until n_new tokens exist.  "T" of the algorithms is a minimum
 * length: the last loop may overshoot and is truncated to exactly n_new.
 *   prompt      host  [prompt_len], prompt_len >= 1, ids < vocab
 *   out_tokens  host  [n_new]
 *   out_stats   host, may be NULL
 * temperature > 0 scales both models' logits before the rejection scheme
 * (section Modified Rejection Sampling: a temperature changes the
 * probabilities the scheme is applied to);
 * temperature == 0 is greedy decoding (top-k with k = 1 on both models, see
 * sps_set_sampling).  SPS_ERANGE if prompt_len + n_new + K > max_seq. */
int sps_generate(sps_handle* h, const int32_t* prompt, int32_t prompt_len, int32_t n_new, int32_t K,
                 float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats);

/* Top-k and nucleus filtering of BOTH models' distributions ahead of the
 * rejection scheme.  The section Modified Rejection Sampling says these
 * methods are handled by changing the probabilities before the scheme is
 * applied and gives no formula; this library's:
 * after softmax(l / temperature), top_k >= 1 keeps every token whose logit is
 * at least the k-th largest (tokens tied with it stay; 0 = off); then
 * 0 < top_p < 1 keeps, of those, the tokens whose logit is at least v, v the
 * largest logit value such that the tokens with logit >= v hold at least top_p
 * of the mass top-k kept (1 = off); the rest weigh nothing and what is left is
 * renormalised.  The setting stays on the handle for every later sps_generate*,
 * sps_step; no device work.  SPS_EINVAL for top_k < 0 or top_p outside (0, 1]. */
int sps_set_sampling(sps_handle* h, int32_t top_k, float top_p);

/* sps_generate with the lookahead adapted from loop to loop.  The paper fixes K
 * per experiment and finds that the best value depends on the domain (the K
 * trade-off figure); the rule here is this library's: K starts at
 * (K_min + K_max) / 2, grows by one after a loop that accepted every draft,
 * shrinks by one after a loop that rejected its first draft, within
 * [K_min, K_max], 1 <= K_min <= K_max <= max_K.  K depends on the past only, so
 * every loop is an exact iteration of Algorithm 2 and the output law is the
 * target's.  With K_min == K_max it is sps_generate.  out_stats->draft_calls /
 * loops is the mean lookahead used. */
int sps_generate_adaptive(sps_handle* h, const int32_t* prompt, int32_t prompt_len, int32_t n_new, int32_t K_min,
                          int32_t K_max, float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats);

/* Same for B sequences with equal prompt lengths, advanced in lock-step with
 * ragged progress; sequence b uses Philox sequence index index0 + b, index0
 * being 0 unless sps_set_sequence_index0 changed it.  A sequence that has its
 * n_new tokens keeps its rows in the later passes (their shape is fixed) but
 * is no longer advanced, and its overshoot never counts against max_seq:
 * prompt_len + n_new + K <= max_seq is all that is required.
 *   prompts host [B, prompt_len]; out_tokens host [B, n_new]; out_stats host [B] or NULL. */
int sps_generate_batch(sps_handle* h, const int32_t* prompts, int32_t B, int32_t prompt_len, int32_t n_new,
                       int32_t K, float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats);

/* Sequence b of the following sps_generate*, sps_step calls draws its random
 * numbers as Philox sequence index0 + b (counter word c2; the paper runs one
 * sequence and names no generator -- this is how independent sequences get
 * independent uniforms here).  With it a batch, or a replica on another GPU,
 * can carry global sequence numbers and reproduce exactly what each sequence
 * would have produced alone.  Stays on the handle until changed; default 0. */
int sps_set_sequence_index0(sps_handle* h, uint32_t index0);

/* Measurement mode (not part of the method): every draft is accepted with the
 * fixed probability alpha instead of min(1, q/p), so that tokens per loop --
 * (1 - alpha^(K+1)) / (1 - alpha) in expectation -- can be swept independently
 * of how well a draft model happens to agree with its target (the Results
 * section's speed-ups depend on that agreement; random-init models have
 * little).  The emitted tokens then follow no particular law; every kernel
 * runs exactly as otherwise.  alpha in (0, 1]; 0 switches the mode off (the
 * default).  Applies to the generate / step calls of this handle. */
int sps_set_forced_acceptance(sps_handle* h, float alpha);

/* Per-loop record of the last sps_generate / sps_generate_adaptive /
 * sps_generate_batch call, for latency percentiles (the Results section
 * reports mean per-token latency; a loop delivers its tokens together, so the
 * distribution of per-loop times is what a serving system sees).
 *   loop_ms      host [cap], device time of loop i (draft + scoring + accept), may be NULL
 *   loop_emitted host [cap], tokens loop i emitted for sequence 0 (before truncation to n_new), may be NULL
 *   loop_K       host [cap], lookahead loop i ran with, may be NULL
 *   *out_loops   loops the call ran (may exceed cap: only the first cap are copied)
 * SPS_ESTATE before the first generation. */
int sps_last_loop_trace(sps_handle* h, float* loop_ms, int32_t* loop_emitted, int32_t* loop_K, int32_t cap, int32_t* out_loops);

/* Pieces of sps_generate, for tests that drive the loop themselves. */
/* forget every sequence and both caches' lengths */
int sps_reset(sps_handle* h);
/* make toks[0..n-1] (host) the sequence so far of a batch-1 run; both caches take positions 0..n-2 */
int sps_prefill(sps_handle* h, const int32_t* toks, int32_t n);
/* the same for B sequences of their own lengths: sequence b is toks[b * ld .. b * ld + lens[b]) (host, lens[b] >= 1,
 * lens[b] <= ld); both caches take positions 0 .. lens[b] - 2 of each.  What follows a sequence's length in its
 * row of toks is ignored.  B <= max_batch. */
int sps_prefill_batch(sps_handle* h, const int32_t* toks, const int32_t* lens, int32_t B, int32_t ld);
/* one loop iteration (Algorithm 2's while-body) with loop index `step`, for every sequence the last prefill set:
 * out_tokens host [B, K+1] (emitted first, -1 after), out_n_emitted host [B] = n_accepted + 1,
 * out_flags host [B] SPS_FLAG_* (may be NULL); B = 1 after sps_prefill */
int sps_step(sps_handle* h, int32_t K, float temperature, uint64_t seed, uint32_t step, int32_t* out_tokens,
             int32_t* out_n_emitted, uint32_t* out_flags);
/* copy what the last sps_step saw to HOST buffers (any may be NULL):
 * q_logits [B, K+1, V], p_logits [B, K, V], drafts [B, K] */
int sps_last_logits(sps_handle* h, int32_t K, float* q_logits, float* p_logits, int32_t* drafts);

/* The scoring step of Algorithm 2 alone (section Conditional Scoring): one
 * target pass that yields the K+1 conditional logit rows for the K drafts and
 * the position after them.  Feeds rows[0..K] (host) to the TARGET at positions
 * len..len+K where len is the target cache's valid length, appends their
 * keys/values, and writes logits.  Does not move the valid length (calling it
 * again overwrites the same positions), so it can be timed repeatedly.
 *   out_logits DEVICE fp32 [K+1, vocab], caller-owned; out_ms host, device time, may be NULL. */
int sps_verify(sps_handle* h, const int32_t* rows, int32_t K, float* out_logits, float* out_ms);
/* The same pass over n_rows rows (1..16) of either model; which: 0 = target, 1 = draft. */
int sps_score(sps_handle* h, int32_t which, const int32_t* rows, int32_t n_rows, float* out_logits, float* out_ms);

/* The modified rejection sampler alone (Algorithm 2's second for-loop and its
 * extra-token line; section "Modified Rejection Sampling"), one fused kernel:
 * softmax statistics of q_0..q_K and p_0..p_{K-1} at `temperature`; for
 * t = 0..K-1 accept draft t iff u_acc < min(1, q_t(d_t) / p_t(d_t)); at the
 * first rejection draw from max(0, q_t - p_t) / sum max(0, q_t - p_t) and stop;
 * if none, draw from q_K.
 *   q_logits      device fp32 [B, K+1, V]
 *   p_logits      device fp32 [B, K, V]   (the logits the drafts were drawn from)
 *   draft_tokens  device int32 [B, K]
 *   stream        cudaStream_t (NULL = default stream); the call only enqueues
 *   out_n_accepted device int32 [B]
 *   out_tokens    device int32 [B, K+1]: accepted drafts, then the resampled / extra token, then -1
 *   out_flags     device uint32 [B], SPS_FLAG_*
 * Sequence b uses Philox counter (t, step, b, 0).  0 <= K <= SPS_MAX_K, V >= 1. */
int sps_accept(const float* q_logits, const float* p_logits, const int32_t* draft_tokens, int32_t B, int32_t K,
               int32_t V, float temperature, uint64_t seed, uint32_t step, void* stream, int32_t* out_n_accepted,
               int32_t* out_tokens, uint32_t* out_flags);

/* sps_accept with both distributions filtered as sps_set_sampling describes
 * (top_k 0 and top_p 1 = plain sps_accept; temperature 0 = greedy). */
int sps_accept_filtered(const float* q_logits, const float* p_logits, const int32_t* draft_tokens, int32_t B, int32_t K,
                        int32_t V, float temperature, int32_t top_k, float top_p, uint64_t seed, uint32_t step,
                        void* stream, int32_t* out_n_accepted, int32_t* out_tokens, uint32_t* out_flags);

/* One inverse-CDF draw per row from softmax(logits / temperature) with
 * u_draft of counter (t, step, b, 0): the draft draw of Algorithm 2's first
 * for-loop, for given logits.  logits device fp32 [B, V];
 * out_tokens device int32 [B]. */
int sps_sample(const float* logits, int32_t B, int32_t V, float temperature, uint64_t seed, uint32_t step, uint32_t t,
               void* stream, int32_t* out_tokens);

/* sps_sample from the filtered distribution (see sps_set_sampling). */
int sps_sample_filtered(const float* logits, int32_t B, int32_t V, float temperature, int32_t top_k, float top_p,
                        uint64_t seed, uint32_t step, uint32_t t, void* stream, int32_t* out_tokens);

/* The memory-bound linear layer alone (section Conditional Scoring: at small
 * batch the linear layers are bound by memory): Y[M, N] = X[M, D] W[N, D]^T with fp32
 * accumulation.  W device, row-major [N, D], dtype 0 fp32 / 1 bf16; X device
 * fp32 [M, D]; Y device fp32 [M, N]; 1 <= M <= 16.  bf16 needs D % 128 == 0 and
 * 16-byte aligned W.  workspace: device scratch of sps_linear_workspace_bytes()
 * bytes for the same (dtype, M, N, D), zero-filled once before its first use
 * (the kernel leaves it ready for the next call).
 * out_ms: host, device time of the kernel, may be NULL; when given the call
 * waits for the kernel and returns SPS_ETIMEOUT if a bounded wait inside it ran out
 * (Y is then meaningless; the workspace stays usable for the next call).
 * sps_linear_scaled also takes dtype 2: W device int8 [N, D] (signed bytes) with
 * row_scale device fp32 [N], Y[m, n] = row_scale[n] * sum_k X[m, k] W[n, k] -- the
 * weight-only quantisation the paper's closing remark on quantisation refers to
 * (it composes with speculative sampling because the transformer body is not
 * touched): half the bytes per weight.  row_scale must be NULL for dtypes 0, 1.
 * The same workspace size function serves all three. */
int sps_linear_scaled(const void* W, int32_t dtype, const float* row_scale, const float* X, int32_t M, int32_t N, int32_t D,
                      float* Y, void* workspace, void* stream, float* out_ms);
int sps_linear(const void* W, int32_t dtype, const float* X, int32_t M, int32_t N, int32_t D, float* Y,
               void* workspace, void* stream, float* out_ms);
int64_t sps_linear_workspace_bytes(int32_t dtype, int32_t M, int32_t N, int32_t D);

/* The linear layer of the prompt pass (Algorithm 2 starts from a prompt of t
 * tokens whose keys and values both models must hold before the first loop):
 * the same product Y[M, N] = X[M, D] W[N, D]^T for up to 128 rows at once, so
 * that the weights are read once for the whole prompt chunk.  bf16 weights
 * only; W device row-major [N, D], 16-byte aligned; X device fp32 [M, D]; Y
 * device fp32 [M, N]; 1 <= M <= 128; D a multiple of 64.  The activations enter
 * the tensor cores as two bf16 halves (about 16 significant bits), products
 * accumulate in fp32.  workspace: device scratch of
 * sps_linear_wide_workspace_bytes(N, D) bytes, contents irrelevant.  The call
 * waits for the result; out_ms (host, may be NULL) receives the device time.
 * Returns SPS_ETIMEOUT if a bounded wait inside the kernel ran out. */
int sps_linear_wide(const void* W, const float* X, int32_t M, int32_t N, int32_t D, float* Y, void* workspace, void* stream,
                    float* out_ms);
int64_t sps_linear_wide_workspace_bytes(int32_t N, int32_t D);

/* The same linear layer for callers that cannot allocate device memory (the
 * paper has no counterpart: this is a service of the library, not a step of
 * the method).  A host that runs inside a stream capture, or serves under a
 * frozen memory budget, or is a plugin that only ever receives buffers, has no
 * workspace to hand to sps_linear; here the split-K scratch is a fixed array
 * inside the library's device image (about 16 MiB on every GPU that loads the
 * library, held until the process exits).  The call makes no cudaMalloc /
 * cudaFree and uses no allocating library routine.
 *   W, X, Y, dtype, M, N, D: as for sps_linear (all device pointers).
 *   stream: cudaStream_t, NULL = default stream; the call only enqueues.
 * Limit: sps_linear_static_floats_needed(dtype, M, N, D) <=
 * sps_linear_static_max_floats() (4 Mi floats).  The need is N * 16 * splits,
 * where splits is how many ranges the kernel cuts D into on the current device
 * (1 for fp32; for bf16 D over the largest multiple of 128 that divides D and
 * is at most 2048 -- 1024 for M > 8 or for layers with few rows); ask the
 * helper rather than redoing that rule.  Larger shapes return SPS_EINVAL with
 * a message.  The first call on a device looks up the array's device address
 * (cudaGetSymbolAddress) with that device current; make that first call
 * before any stream capture begins.
 * All calls share the one array: two calls whose kernels overlap on the GPU
 * (different streams) race on it -- keep them on one stream or order them.
 * Each call clears the array's counters before its kernel, so a call that
 * follows an aborted one starts clean.  The call only enqueues and cannot
 * report a bounded wait that ran out inside the kernel (sps_linear with
 * out_ms can); Y is then meaningless. */
int sps_linear_static(const void* W, int32_t dtype, const float* X, int32_t M, int32_t N, int32_t D, float* Y,
                      void* stream);
int64_t sps_linear_static_max_floats(void);
/* floats of split-K scratch the shape needs on the current device; -1 for arguments sps_linear_static rejects */
int64_t sps_linear_static_floats_needed(int32_t dtype, int32_t M, int32_t N, int32_t D);

/* Tensor-parallel passes (section Conditional Scoring: the models are served Megatron-style over several chips, the
 * attention and feed-forward blocks sharded and each followed by an all-reduce of (K + 1) x d_model numbers, which
 * is latency-bound and about as costly for K + 1 rows as for one; section Choice of Draft Models: the draft is shaped
 * to be served on the same chips).  One process per GPU; rank r of `world` (<= 8) creates its handle with
 * SPS_CFG_TENSOR_PARALLEL and ITS SHARD of both models:
 *   wq, wk, wv, w_up : the shard's output rows -- n_heads / world query heads, n_kv_heads / world key / value heads,
 *                      d_ff / world feed-forward features (contiguous blocks, rank r the r-th);
 *   wo, w_down       : the matching input COLUMNS, stored densely: [d_model, n_heads * d_head / world],
 *                      [d_model, d_ff / world];
 *   embeddings, unembedding, norm gains: whole, on every rank.
 * sps_model_cfg then describes the shard: d_model as in the whole model, n_heads / n_kv_heads / d_ff the shard's
 * (n_heads * d_head < d_model is allowed under this flag).  After every output projection the ranks exchange their
 * partial updates of the residual stream: each rank stores its partial into a slot of every rank's inbox (plain
 * stores into peer memory) and raises a flag there; each rank then sums the slots of its OWN inbox in rank order, so
 * every rank holds the same bits and runs the same loop.  No library collective, no multicast.
 *
 * sps_tp_buffers returns this rank's inbox and flag array (device pointers, with their sizes) for export to the
 * peers (e.g. as CUDA IPC handles, which the caller exchanges however it talks to its peers).
 * sps_tp_attach gives the handle every rank's inbox and flag array as THIS device addresses them (entry `rank`: its
 * own); attach every rank before any of them runs a pass.  Afterwards the handle's calls (sps_prefill, sps_step,
 * sps_generate, ...) are collective: every rank makes the same calls with the same arguments.  Waits on peers are
 * bounded like every other wait (SPS_ETIMEOUT). */
int sps_tp_buffers(sps_handle* h, void** inbox, void** flags, int64_t* inbox_bytes, int64_t* flags_bytes);
int sps_tp_attach(sps_handle* h, int32_t rank, int32_t world, void* const* peer_inbox, void* const* peer_flags);
/* A whole group emulated on ONE GPU, for checking the sharded arithmetic and the exchange kernels without `world`
 * GPUs: ranks[r] is rank r's handle, all created on one device with the same cfg.stream and attached to one another
 * with plain device pointers.  The calls enqueue what the `world` processes would, phase by phase (every rank's
 * store phase of an exchange before any rank's sum), so nothing ever waits for a kernel that is launched later.
 * sps_tp_group_prefill: as sps_prefill on every rank.  sps_tp_group_score: as sps_score on every rank; out_logits
 * host array of `world` DEVICE buffers [n_rows, vocab], which come out identical.  sps_tp_group_generate: below. */
int sps_tp_group_prefill(sps_handle* const* ranks, int32_t world, const int32_t* toks, int32_t n);
/* sps_generate for the emulated group (one sequence): every rank drafts, scores and runs the accept kernel on its own
 * copy of the logits; the ranks' decisions are compared after every loop (SPS_ESTATE if they ever differ) and rank 0's
 * tokens are returned.  out_stats: counts and the decode time only. */
int sps_tp_group_generate(sps_handle* const* ranks, int32_t world, const int32_t* prompt, int32_t prompt_len, int32_t n_new,
                          int32_t K, float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats);
int sps_tp_group_score(sps_handle* const* ranks, int32_t world, int32_t which, const int32_t* rows, int32_t n_rows,
                       float* const* out_logits, float* out_ms);

/* Test hook for the give-up path of the kernels' waits.  Every wait inside a
 * kernel (on a copy, on another CTA, on a tile queue) is bounded by the global
 * timer: when the bound runs out the kernel records an error, lets the copies
 * it has in flight land, frees what it holds and returns, and the host call
 * reports SPS_ETIMEOUT.  limit_us shortens that bound (0 = the default of 2 s;
 * at most 2 s), and drop_stage >= 0 makes the copy producer of the first CTA
 * of sps_linear / sps_linear_wide leave out that stage of its ring, so that a
 * wait runs out on purpose with nothing left in flight (-1 = leave nothing
 * out).  Process-wide; not thread-safe; meant for tests only. */
int sps_debug_set_wait(int64_t limit_us, int32_t drop_stage);

/* Philox4x32-10 on the device, for known-answer tests: ctr device uint32 [n,4],
 * key device uint32 [n,2], out device uint32 [n,4]. */
int sps_philox(const uint32_t* ctr, const uint32_t* key, int32_t n, void* stream, uint32_t* out);

#ifdef __cplusplus
}
#endif
#endif
