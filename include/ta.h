/*
 * ta.h — C ABI of the Transactional Attention (TA) KV-cache compaction library for NVIDIA B200 (sm_100a).
 *
 * The library implements one thing: the retention step of TA (Algorithm 1), run once over a prefilled KV cache,
 * per layer and per KV head:
 *
 *   1. anchor detection + voucher allocation   (Section 3.2, Eq. 2, Algorithm 1 steps 1-6)   ta_sponsor_mask
 *   2. attention part of the utility           (Eq. 1 terms alpha*A_i and delta*P_i)           ta_score
 *   3. budget-K selection                      (Algorithm 1 step 8, Section 3.3)               ta_select_topk
 *   4. eviction = gather of retained rows      (Algorithm 1 step 9, Section 3.2)               ta_compact_kv
 *   all four in one enqueue                    (Algorithm 1)                                   ta_compress
 *
 * Conventions shared by every entry point
 *   - Positions are 0-based; the paper's 1-based position i is i0 + 1.
 *   - "DEVICE" pointers are CUDA device memory owned by the caller and must stay valid until the stream has
 *     executed the call. "HOST" pointers are read before the call returns.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL = the legacy default stream),
 *     allocate no memory, never throw and never abort. Host-detectable problems are returned as ta_status
 *     and nothing is enqueued. Problems only the device can see (a token id outside the vocabulary, a sequence
 *     longer than max_n, a pipeline wait that ran out) are recorded in the context and returned by ta_ctx_poll();
 *     the kernels skip the offending access and still terminate.
 *   - A batch holds B sequences. Uniform batches give every sequence n_uniform tokens; ragged batches pack
 *     all tokens back to back and give cu_seqlens (B+1 ascending offsets, cu_seqlens[0] = 0). In both cases
 *     token (b, i) has the packed index tok = cu_seqlens[b] + i (uniform: b*n_uniform + i). Per-token
 *     arrays are indexed by tok; per-(layer, KV head, token) arrays are laid out [L][Hkv][total_tokens].
 *   - A "unit" is one (layer l, sequence b, KV head g); units are independent.
 *   - Supported shapes: head_dim d = 128; G = Hq/Hkv and observation window W with G*W <= 256 and W <= 64;
 *     budget K <= 4096... see ta_limits below. Anything else returns TA_ERR_UNSUPPORTED: there is no fallback
 *     path.
 */
#ifndef TA_H_
#define TA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ta_status {
  TA_OK = 0,
  TA_ERR_INVALID_ARG = 1,       /* NULL where data is required, negative size, inconsistent batch description   */
  TA_ERR_UNSUPPORTED = 2,       /* shape or device outside the supported set                                     */
  TA_ERR_ALIGNMENT = 3,         /* a bf16 view whose base or strides are not 16-byte multiples                   */
  TA_ERR_SCRATCH_TOO_SMALL = 4, /* the context's scratch cannot hold this call (see ta_scratch_bytes)            */
  TA_ERR_CUDA = 5,              /* a CUDA runtime / driver call failed; ta_ctx_last_cuda_error() has the code     */
  TA_ERR_TIMEOUT = 6,           /* device: a bounded pipeline wait ran out                                       */
  TA_ERR_DEVICE_BOUNDS = 7      /* device: token id >= vocab_size, or a sequence longer than max_n                */
} ta_status;

enum { TA_MODE_SCORED = 0, TA_MODE_FAST = 1 };

/* bits of the per-token flag byte written by ta_sponsor_mask */
enum {
  TA_FLAG_ANCHOR_TOKEN = 1, /* S_i of Eq. 1: the token belongs to a matched anchor pattern            */
  TA_FLAG_ANCHOR_END = 2,   /* the token is the last token of a match: "the anchor i" of Eq. 2        */
  TA_FLAG_SPONSORED = 4     /* V_i > 0                                                                */
};

/* hard limits of the library (validated on every call) */
enum {
  TA_MAX_PATTERNS = 256,    /* patterns in one set                                                     */
  TA_MAX_PATTERN_LEN = 8,   /* token ids per pattern                                                   */
  TA_MAX_SPAN = 64,         /* sponsorship span L per pattern                                          */
  TA_MAX_WINDOW = 64,       /* observation window W                                                    */
  TA_MAX_SCORE_ROWS = 256,  /* G * W                                                                   */
  TA_MAX_BUDGET = 4096,     /* K                                                                       */
  TA_MAX_SEQ_LEN = 1 << 20, /* tokens per sequence                                                     */
  TA_HEAD_DIM = 128,        /* d                                                                       */
  TA_MAX_CONCEPTS = 8,      /* anchor-concept embeddings of the embedding detector                     */
  TA_MAX_EMBED_DIM = 8192   /* embedding width of the embedding detector                               */
};

/*
 * Hyper-parameters of Eq. 1 / Eq. 2 / Section 3.3. Paper defaults in brackets.
 *   alpha, beta, gamma, delta, lambda  weights of Eq. 1                       [1.0 0.5 0.3 0.2 0.1]
 *   voucher_decay                      base of the per-token voucher decay    [0.8]  (Eq. 2)
 *   budget_decay, age_steps            B_i = B_p * budget_decay^age_steps     [0.9, 0] (Section 3.2, budgets decay per step)
 *   n_sink, n_recent                   mandatory first / last tokens, taken from the main pool (Section 3.3)
 *   k_protected                        slots reserved for sponsored tokens; < 0 means K_eff - n_sink - n_recent
 *                                      (the K_p = K - 1 - W of Theorems 2-4)
 *   obs_window                         W: number of trailing query positions whose attention is summed into A_i
 *   pension_rho                        P_i is an exponential moving average over the W window rows with this
 *                                      coefficient: P_i = sum_t (1-rho) rho^(W'-1-t) a_{t,i}
 *   softmax_scale                      0 means 1/sqrt(d)
 *   causal                             1: query row t (position n-W+t) sees keys i <= n-W+t
 *   mode                               TA_MODE_SCORED (Eq. 1) or TA_MODE_FAST (Eq. 3: alpha = delta = 0, no Q/K read)
 *   vocab_size                         token ids must lie in [0, vocab_size); sizes the frequency histogram of F_i
 */
typedef struct ta_policy {
  float alpha, beta, gamma, delta, lambda;
  float voucher_decay;
  float budget_decay;
  int32_t age_steps;
  int32_t n_sink, n_recent, k_protected;
  int32_t obs_window;
  float pension_rho;
  float softmax_scale;
  int32_t causal;
  int32_t mode;
  int32_t vocab_size;
} ta_policy;

/* Named budget partitions. The paper states three that disagree; all are expressible in ta_policy:
 *   TA_PRESET_THEOREM  1 sink, 4 recent, protected = the rest   (Theorems 2-4, Corollary on the minimum budget)
 *   TA_PRESET_SEC33    1 sink, 2 recent, protected = K/4        (Section 3.3: K=16 -> 12 + 4)
 *   TA_PRESET_AUDIT    4 sinks, 6 recent, 6 protected           (baseline-audit table, K=16)
 * ta_policy_default fills every field with the paper's defaults for budget K and the given preset. */
enum { TA_PRESET_THEOREM = 0, TA_PRESET_SEC33 = 1, TA_PRESET_AUDIT = 2 };
ta_status ta_policy_default(int preset, int K, ta_policy* out /*HOST*/);

typedef struct ta_batch {
  int32_t n_layers;          /* L >= 1: layers handled by this call (independent; a launch-batching dimension) */
  int32_t batch;             /* B >= 1                                                                       */
  int32_t n_uniform;         /* tokens per sequence when cu_seqlens == NULL                                  */
  int32_t max_n;             /* >= every sequence length (sizes the launch)                                  */
  int64_t total_tokens;      /* sum of lengths (B * n_uniform when uniform)                                  */
  const int32_t* cu_seqlens; /* DEVICE, B+1 entries, or NULL for a uniform batch                             */
} ta_batch;

/* A bf16 tensor with head_dim contiguous. Element (l, b, h, i, c) lives at
 *   uniform batch: ptr + l*stride_l + b*stride_b + h*stride_h + i*stride_n + c
 *   ragged batch : ptr + l*stride_l + h*stride_h + (cu_seqlens[b] + i)*stride_n + c        (stride_b unused)
 * Strides are in elements and must be multiples of 8 (16 bytes); ptr must be 16-byte aligned.
 * For q_obs the position axis is the window row t in [0, W) (row t is the query at position n - W + t; when
 * n < W the first W - n rows are ignored) and the tensor is always dense per sequence (stride_b is used for
 * ragged batches too). */
typedef struct ta_bf16_view {
  const void* ptr; /* DEVICE */
  int64_t stride_l, stride_b, stride_h, stride_n;
} ta_bf16_view;

typedef struct ta_ctx ta_ctx;           /* opaque; one per device; owns scratch and the device status word      */
typedef struct ta_patterns ta_patterns; /* opaque; device-resident matcher tables                               */

/* ---- context ---------------------------------------------------------------------------------------------- */

/* Creates a context on `device` (must be compute capability 10.x) with `scratch_bytes` of device scratch.
 * The only entry points that allocate or free device memory are ta_ctx_create/destroy and
 * ta_patterns_create/destroy. */
ta_status ta_ctx_create(int device, size_t scratch_bytes, ta_ctx** out);
void ta_ctx_destroy(ta_ctx* ctx);

/* Scratch needed by the largest of the entry points for this problem size (ta_compress needs the most). */
ta_status ta_scratch_bytes(const ta_batch* batch, int Hq, int Hkv, int d, int K, const ta_policy* policy,
                           size_t* out_bytes);

/* Synchronises the context's device, then returns and clears the first device-detected error (TA_OK if none). */
ta_status ta_ctx_poll(ta_ctx* ctx);
int ta_ctx_last_cuda_error(const ta_ctx* ctx);
const char* ta_status_string(ta_status s);

/* Limit of every device-side wait of the kernels launched through this context, in nanoseconds of wall time
 * (default and 0: two seconds). A wait that runs out makes its kernel return early; ta_ctx_poll then reports
 * TA_ERR_TIMEOUT once and the outputs of that call are undefined. Meant for callers with their own watchdog and for
 * tests. */
ta_status ta_ctx_set_wait_limit(ta_ctx* ctx, uint64_t nanoseconds);
/* Diagnostic for the time-out path: enqueues a kernel of one warp that waits, with a limit of limit_ns (at most one
 * second), on a barrier that nothing completes, with no copy or tensor-core operation in flight. The kernel returns
 * when the limit is reached, sets bit 2 of *outcome (DEVICE int32; bits 0 and 1 would mean a wait succeeded), and
 * the next ta_ctx_poll reports TA_ERR_TIMEOUT once. The context stays usable. */
ta_status ta_ctx_selftest_wait(ta_ctx* ctx, uint64_t limit_ns, int32_t* outcome, void* stream);
/* Tuning: CTAs that share one (layer, sequence, KV head) unit in the score kernel: 1, 2, 4 or 8; 0 (default) lets
 * the library choose per launch from the unit count, the sequence length and the L2 size. */
ta_status ta_ctx_set_score_cluster(ta_ctx* ctx, int ctas_per_unit);

/* What the most recent ta_compress (or variant) call on this context launched: out[0] = CTAs per unit of the score
 * kernel, out[1] = its clusters, out[2] = 1 when the selection kernel gathered the retained rows itself (small
 * budgets; no separate gather kernel), out[3] = kernels of this library the call enqueued. */
ta_status ta_ctx_last_launch_info(const ta_ctx* ctx, int32_t out[4] /*HOST*/);

/* Every entry point that enqueues work opens an NVTX range of its own name around its host side (visible in timeline
 * tools; free when no tool is attached). */

/* Optional per-kernel timing of ta_compress: when enabled, CUDA events are recorded on the call's stream around
 * each kernel of the next ta_compress calls. ta_ctx_read_timing synchronises on those events and returns the
 * milliseconds of the most recent call in out_ms[0..4] = {mask+static utility, score, select, compact, total}.
 * Stages that did not run report 0. */
ta_status ta_ctx_enable_timing(ta_ctx* ctx, int enable);
ta_status ta_ctx_read_timing(ta_ctx* ctx, float out_ms[5] /*HOST*/);

/* ---- anchor patterns (Section 3.2: the pattern set P; passing only allow-listed patterns is the allowlist
 *      defence of Section 5.3) ------------------------------------------------------------------------------- */

/* n_pat patterns; pattern p is ids_flat[offsets[p] .. offsets[p+1]) (1..TA_MAX_PATTERN_LEN token ids, all >= 0).
 * budget[p] is the sponsor budget B (NULL: 15 for all), span[p] the span L in [1, TA_MAX_SPAN] (NULL: 6).
 * All arrays HOST. n_pat may be 0 (no anchors: TA degenerates to plain score-based top-K). */
ta_status ta_patterns_create(ta_ctx* ctx, int n_pat, const int32_t* ids_flat, const int32_t* offsets,
                             const float* budget, const int32_t* span, ta_patterns** out);
void ta_patterns_destroy(ta_patterns* pats);

/* ---- step 1: sponsorship mask, vouchers and the attention-free utility ------------------------------------
 * Algorithm 1 steps 1-6 and the attention-free part of step 7 (which is the whole TA-Fast score, Eq. 3).
 * For every token: a pattern ends at position e when ids[e-len+1..e] equals it and the match does not cross
 * the start of the sequence; if several patterns end at e the longest wins, then the lowest index. Every token of
 * a match gets TA_FLAG_ANCHOR_TOKEN, its last token TA_FLAG_ANCHOR_END. Vouchers follow Eq. 2 with the winning
 * pattern's budget (decayed age_steps times) and span, clipped at the end of the sequence; contributions of several
 * anchors add, nearest anchor first. u_static = ((beta*R + gamma*S) - lambda*F) + V with R = (i0+1)/n and
 * F = (occurrences of the token's id in its sequence)/n, every operation rounded to fp32.
 *   token_ids  DEVICE int32 [total_tokens]
 *   flags      DEVICE uint8 [total_tokens]   out
 *   voucher    DEVICE float [total_tokens]   out
 *   u_static   DEVICE float [total_tokens]   out
 * Uses B*vocab_size*4 bytes of context scratch. batch->n_layers is ignored. */
ta_status ta_sponsor_mask(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                          const int32_t* token_ids, uint8_t* flags, float* voucher, float* u_static, void* stream);

/* ---- embedding-based anchor detector (Section 3.2 "Anchor detection", third instantiation; Section 5.4) ---------
 * "Cosine similarity between input embeddings and anchor concept embeddings": conf[i] is the largest cosine
 * similarity between token i's input embedding and the n_concepts concept embeddings (a zero vector has similarity
 * 0 with everything; a NaN anywhere in a token's embedding gives NaN, which no threshold accepts). The result is a
 * per-token confidence for ta_sponsor_mask_conf.
 *   emb       DEVICE bf16, token i at emb + i*stride_tok, D contiguous values (the model's input-embedding rows of
 *             the prompt tokens); 16-byte aligned, stride_tok a multiple of 8 and >= D
 *   concepts  DEVICE bf16 [n_concepts][D]
 *   conf      DEVICE float [total_tokens] out
 * D a multiple of 32, at most TA_MAX_EMBED_DIM; 1 <= n_concepts <= TA_MAX_CONCEPTS. bf16 products accumulated in
 * fp32 on the tensor cores; the embeddings are read exactly once. */
ta_status ta_detect_embedding(ta_ctx* ctx, int64_t total_tokens, const void* emb, int64_t stride_tok, int D,
                              const void* concepts, int n_concepts, float* conf, void* stream);

/* ---- step 1 with a learned anchor detector (Section 5.1, "Learned Anchor Detection") ----------------------
 * The detector itself (an MLP on hidden states, or an embedding similarity) runs in the caller's model; its
 * per-token confidence f(h_i) is the input here. Token i is an anchor iff conf[i] > threshold (NaN: no anchor).
 * Anchors are single tokens: TA_FLAG_ANCHOR_TOKEN and TA_FLAG_ANCHOR_END are set together, all anchors share the
 * span L = span, and vouchers, flags and u_static follow exactly as in ta_sponsor_mask (Eq. 2, Eq. 3) with the
 * per-anchor budget
 *   rank_by_confidence == 0 : B_i = budget                  TA-Learned   (paper: threshold 0.5, B = 15)
 *   rank_by_confidence != 0 : B_i = budget * conf[i]        TA-LearnRank (paper: threshold 0.3, budget = 1, i.e.
 *                             V_j = sum_i f(h_i) 0.8^(j-i) 1[f(h_i) > 0.3, i < j <= i+L])
 * decayed age_steps times like a pattern's budget; every product rounded to fp32.
 *   conf  DEVICE float [total_tokens]
 * span in [1, TA_MAX_SPAN]. Other arguments, outputs and scratch use as ta_sponsor_mask. The outputs feed
 * ta_select_topk / ta_compact_kv unchanged. */
ta_status ta_sponsor_mask_conf(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, const int32_t* token_ids,
                               const float* conf, float threshold, float budget, int span, int rank_by_confidence,
                               uint8_t* flags, float* voucher, float* u_static, void* stream);

/* ---- step 2: attention mass over the observation window ---------------------------------------------------
 * Eq. 1's A_i and P_i, read as a one-shot compaction after prefill: for unit (l, b, g) the score rows are the
 * last W' = min(W, n) query positions of the G = Hq/Hkv query heads of KV group g;
 *   a_{h,t,i} = softmax_i( scale * <q_{h,t}, k_i> )   over the keys the row may see,
 *   A_i = sum_{h,t} a_{h,t,i},      P_i = sum_{h,t} (1-rho) rho^(W'-1-t) a_{h,t,i}.
 *   q_obs   bf16 view, positions = window rows, heads = Hq query heads
 *   k       bf16 view, positions = context tokens, heads = Hkv
 *   lse_obs DEVICE float [L][B][Hq][W] natural-log softmax normalisers of the same rows, or NULL. When given
 *           (a prefill attention kernel has them), the keys are read once instead of twice.
 *   A, P    DEVICE float [L][Hkv][total_tokens], out; P may be NULL.
 * The contraction runs on the tensor cores (bf16 inputs, fp32 accumulation). */
ta_status ta_score(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                   ta_bf16_view q_obs, ta_bf16_view k, const float* lse_obs, float* A, float* P, void* stream);

/* The attention part of Eq. 1 with its weights applied, u_att_i = alpha*A_i + delta*P_i, as ta_compress computes it
 * before the attention-free terms are added: the same rows, keys and arguments as ta_score, one output.
 *   u_att   DEVICE float [L][Hkv][total_tokens], out.
 * When every row weight alpha + delta*(1-rho)*rho^(W-1-t) is positive (true for the paper's alpha = 1, delta = 0.2)
 * the weights are folded into the softmax exponents and a key costs a single sum; the result equals
 * alpha*A + delta*P up to fp32 rounding (relative 1e-3 + absolute 1e-5 against exact arithmetic, as for A and P). */
ta_status ta_score_weighted(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                            ta_bf16_view q_obs, ta_bf16_view k, const float* lse_obs, float* u_att, void* stream);

/* ---- step 3: budget-K selection (Algorithm 1 step 8 with the partition of Section 3.3) --------------------
 * Per unit: K_eff = min(K, n). If K_eff == n everything is kept. Otherwise p = k_protected (auto when < 0,
 * clipped to [0, K_eff]) slots are protected and K_main = K_eff - p are main slots. Mandatory tokens (sinks
 * 0.., then recents n-1, n-2, ..) are taken in that order while main slots last; the protected pool takes the
 * sponsored tokens (voucher > 0) with the largest vouchers, lower position first among equals; what is left of
 * the budget goes to the tokens with the largest u = (alpha*A + delta*P) + u_static (TA_MODE_SCORED) or
 * u = u_static (TA_MODE_FAST), lower position first among equals (+0 and -0 compare equal; inputs must be finite).
 *   flags, voucher, u_static  DEVICE, per token, as written by ta_sponsor_mask
 *   A, P                      DEVICE float [L][Hkv][total_tokens] (scored mode; P may be NULL; both NULL in fast mode)
 *   idx    DEVICE int32 [L][B][Hkv][K]  out: retained positions, ascending, padded with -1
 *   count  DEVICE int32 [L][B][Hkv]     out: K_eff
 * Uses total_tokens + 8*B bytes of context scratch. */
ta_status ta_select_topk(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hkv, int K,
                         const uint8_t* flags, const float* voucher, const float* u_static, const float* A,
                         const float* P, int32_t* idx, int32_t* count, void* stream);

/* ---- step 3 without any allocation -------------------------------------------------------------------------
 * (No counterpart in the paper: this entry point exists for a deployment constraint, not for the method.)
 * Same computation and same results as ta_select_topk, for callers that are not allowed to allocate device memory
 * and therefore cannot create a ta_ctx: code running inside an inference server whose memory pool already owns the
 * whole GPU, a plugin loaded into someone else's process under a fixed memory budget, or a latency-critical loop
 * where cudaMalloc's implicit device synchronisation is unacceptable. It takes no context. Its working memory (one
 * byte per token plus a few words per sequence; in fast mode also B*K indices) lives in a fixed array inside the
 * library image, so every GPU that loads this library gives up TA_STATIC_SCRATCH_BYTES for it until the process
 * exits. The call issues no cudaMalloc/cudaFree and uses no allocating library routine.
 *   - Limit: 256 + total_tokens + 8*B (+ 4*B*K in fast mode), each piece rounded up to 256 bytes, must fit in
 *     TA_STATIC_SCRATCH_BYTES; larger problems are rejected with TA_ERR_SCRATCH_TOO_SMALL and nothing is enqueued.
 *   - It works on the CUDA device that is current when it is called. The first call on each device looks up the
 *     array's device address (a one-time runtime query, no allocation); make that first call outside of any stream
 *     capture.
 *   - All calls share the one array, which still holds the previous call's data: the call clears the part that has
 *     to start at zero itself, but two calls whose kernels can overlap on the GPU (different streams without an
 *     ordering between them, or two host threads) race on it. Serialise them.
 *   - There is no context to poll: a sequence longer than batch->max_n gets count 0 and an all -1 index row instead
 *     of an error code.
 * Arguments are those of ta_select_topk without the context. */
enum { TA_STATIC_SCRATCH_BYTES = 4 << 20 };
ta_status ta_select_topk_static(const ta_policy* policy, const ta_batch* batch, int Hkv, int K, const uint8_t* flags,
                                const float* voucher, const float* u_static, const float* A, const float* P,
                                int32_t* idx, int32_t* count, void* stream);

/* ---- step 4: compaction (Algorithm 1 step 9: index_select along the sequence axis) ------------------------
 *   k, v          bf16 views over the full cache
 *   idx, count    as written by ta_select_topk
 *   k_out, v_out  DEVICE bf16 [L][B][Hkv][K][d] out; rows at and beyond count are zero-filled. */
ta_status ta_compact_kv(ta_ctx* ctx, const ta_batch* batch, int Hkv, int d, int K, ta_bf16_view k, ta_bf16_view v,
                        const int32_t* idx, const int32_t* count, void* k_out, void* v_out, void* stream);

/* ---- all steps in one enqueue (Algorithm 1) ---------------------------------------------------------------
 * Steps 1-4 for batch->n_layers layers. The per-sequence results of step 1 (and, in fast mode, of step 3, which
 * then does not depend on layer or head) are kept in the context and reused when seq_epoch is non-zero and equal
 * to the previous call's: pass the same non-zero epoch for successive layers of one batch, a new one (or 0:
 * never reuse) for a new batch. Under one epoch the token ids and cu_seqlens must stay the same; a change of the
 * pattern set, of K, of the mode or of any policy field that the per-sequence steps read is noticed and recomputed.
 * In scored mode the utilities stay in context scratch; A and P are not materialised. q_obs and k are not read in fast mode (their ptr may be NULL). */
ta_status ta_compress(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch, int Hq,
                      int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs, ta_bf16_view k,
                      ta_bf16_view v, uint64_t seq_epoch, void* k_out, void* v_out, int32_t* idx, int32_t* count,
                      void* stream);

/* The same when the softmax normalisers of the observation-window rows are already known (a prefill attention kernel
 * computes the log-sum-exp of every query row): lse_obs is DEVICE float [L][B][Hq][W], natural log, as for ta_score.
 * The keys are then read once instead of twice and the scoring costs about half. Scored mode only. */
ta_status ta_compress_lse(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch, int Hq,
                          int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs, ta_bf16_view k,
                          ta_bf16_view v, const float* lse_obs, uint64_t seq_epoch, void* k_out, void* v_out,
                          int32_t* idx, int32_t* count, void* stream);

/* ---- one selection per layer, shared by its KV heads (Eq. 1: A_i "across heads") -----------------------------
 * Eq. 1 and Appendix A Definition 1 define A_i as attention accumulated over ALL heads, which gives one retained
 * set per layer. ta_compress reads them per KV head (every head keeps its own K tokens); this entry point takes
 * the literal reading: A_i and P_i are summed over the Hq query heads of the layer (each attending to the keys of
 * its own KV head), u = (alpha*A + delta*P) + u_static is formed once per (layer, sequence), one selection is
 * made from it, and every KV head of the layer gathers the same positions: idx[l][b][g][:] is the same for all g.
 * The head sum is taken in fp32 over the per-head fused terms, KV head 0 first.
 * Arguments, outputs and scratch as ta_compress; policy->mode must be TA_MODE_SCORED. */
ta_status ta_compress_allheads(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                               int Hq, int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs,
                               ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch, void* k_out, void* v_out,
                               int32_t* idx, int32_t* count, void* stream);

/* The same for a layer whose heads are sharded over several GPUs (tensor-parallel attention), as a pair of calls
 * with the caller's all-reduce in between (Eq. 1 and Appendix A Definition 1: A_i is summed "across heads"):
 *   ta_score_headsum          u_heads[l][tok] = sum over THIS shard's KV heads g (ascending, fp32) of
 *                             alpha*A_g + delta*P_g; Hq and Hkv are the shard's head counts, q_obs and k its views.
 *                             u_heads is DEVICE float [L][total_tokens], out.
 *   (caller)                  sums u_heads over the shards, e.g. an fp32 sum all-reduce of L*total_tokens floats
 *   ta_compress_from_headsum  adds the attention-free terms, selects once per (layer, sequence) exactly as
 *                             ta_compress_allheads does, and gathers the rows of this shard's Hkv heads.
 * Every shard passes the same token ids, patterns, policy and K and therefore retains the same positions. The
 * library performs no communication itself. */
ta_status ta_score_headsum(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                           ta_bf16_view q_obs, ta_bf16_view k, float* u_heads, void* stream);
ta_status ta_compress_from_headsum(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy,
                                   const ta_batch* batch, int Hkv, int d, int K, const int32_t* token_ids,
                                   const float* u_heads, ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch,
                                   void* k_out, void* v_out, int32_t* idx, int32_t* count, void* stream);

/* ---- composition with another eviction score (Section 4.5 "Composability") ---------------------------------
 * TA changes the scoring function, not the eviction policy: sponsorship is added on top of whatever importance
 * score a pipeline already has (accumulated attention of H2O, the pooled prefill-window attention of SnapKV, a
 * per-layer or per-head budgeted score, ...). This entry point is ta_compress with the attention terms of Eq. 1
 * supplied by the caller instead of computed from Q and K:
 *   u = (alpha*score + delta*score2) + u_static,  then selection (Section 3.3) and the gather, as in ta_compress.
 *   score   DEVICE float [L][Hkv][total_tokens]   the caller's per-token importance (takes the place of A_i)
 *   score2  DEVICE float, same shape, or NULL     a second term weighted by delta (takes the place of P_i)
 * policy->mode must be TA_MODE_SCORED; obs_window and the softmax fields are ignored. Values must be finite.
 * Everything else (patterns, seq_epoch reuse of the per-sequence step, outputs, scratch) as ta_compress. */
ta_status ta_compress_scores(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                             int Hkv, int d, int K, const int32_t* token_ids, const float* score,
                             const float* score2, ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch, void* k_out,
                             void* v_out, int32_t* idx, int32_t* count, void* stream);

/* Composition with methods that give every layer or every head its own budget (Section 2 names PyramidKV, whose
 * budgets shrink from layer to layer, and Ada-KV, which sets one per head; Section 4.5 claims TA composes with
 * them): as ta_compress_scores, but (layer l, KV head g) keeps budgets[l*Hkv + g] tokens of every sequence.
 *   budgets  HOST int32 [n_layers][Hkv], each in 1..K_max; at most TA_MAX_BUDGET_CLASSES distinct values and
 *            n_layers*Hkv <= 4096 (else TA_ERR_UNSUPPORTED). Read before the call returns.
 *   K_max    stride of the outputs: idx [L][B][Hkv][K_max], k_out/v_out [L][B][Hkv][K_max][d]; rows at and beyond a
 *            unit's count = min(budget, n) are -1 / zero as in ta_compress.
 * The budget partition of Section 3.3 (sinks, recents, protected pool) is taken per budget value, so a unit's result
 * equals that of ta_compress_scores called with K = its own budget. The per-sequence step is not cached between
 * calls. Scratch: ta_scratch_bytes_budgets (n_budget_classes = number of distinct budget values, or an upper bound). */
#define TA_MAX_BUDGET_CLASSES 64
ta_status ta_scratch_bytes_budgets(const ta_batch* batch, int Hkv, int K_max, const ta_policy* policy,
                                   int n_budget_classes, size_t* out_bytes);
ta_status ta_compress_scores_budgets(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy,
                                     const ta_batch* batch, int Hkv, int d, int K_max, const int32_t* budgets,
                                     const int32_t* token_ids, const float* score, const float* score2,
                                     ta_bf16_view k, ta_bf16_view v, void* k_out, void* v_out, int32_t* idx,
                                     int32_t* count, void* stream);
/* The same budgets with TA's own attention terms (scored mode of ta_compress: A_i and P_i of Eq. 1 from q_obs and k).
 * Scratch: ta_scratch_bytes_budgets (it covers what ta_compress needs). */
ta_status ta_compress_budgets(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                              int Hq, int Hkv, int d, int K_max, const int32_t* budgets, const int32_t* token_ids,
                              ta_bf16_view q_obs, ta_bf16_view k, ta_bf16_view v, void* k_out, void* v_out,
                              int32_t* idx, int32_t* count, void* stream);

/* ---- Algorithm 1 in the decode loop: per-step retention --------------------------------------------------------
 * (Section 3.1: the policy selects S, |S| <= K, "after each generation step"; Algorithm 1 steps 1-10.)
 * Every step brings one new token per sequence. Per unit (layer l, sequence b, KV head g; unit index
 * (l*B + b)*Hkv + g) the library keeps the state of the at most K+1 cached tokens IN POSITION ORDER and decides
 * which one to evict; it never touches key/value rows. The caller owns a cache of K+1 rows per unit: the new token's
 * keys and values go to row next_slot[unit], and an evicted token's row is handed out as the next next_slot.
 * The paper does not say what persists between steps; this library takes these readings: an anchor is detected
 * once, when the token that completes a pattern arrives (Algorithm 1 step 1 on the stream of ids: evicted tokens were
 * seen); a token's voucher is fixed at its arrival (Eq. 2, steps 2-6) and afterwards only decays (step 10); A_i
 * accumulates and P_i averages the per-step attention mass (Eq. 1; Appendix A Definition 1); R_i and F_i use the count
 * of tokens seen so far; nothing is evicted while at most K tokens are cached (Section 3.1).
 * What one step computes:
 *   - the new token completes a pattern (longest wins, then lowest index) -> it becomes an anchor with that pattern's
 *     budget and span; every cached token of the match gets S = 1;
 *   - the new token's voucher (Eq. 2) from the anchors of the last TA_MAX_SPAN positions, whose budgets have decayed
 *     by budget_decay once per step since detection; nearest anchor first;
 *   - A += a and P = rho*P + (1-rho)*a for every cached token, a = this step's attention mass on it;
 *   - u = (alpha*A + delta*P) + ((beta*R + gamma*S) - lambda*F) + V with R = (i0+1)/n, F = count(id)/n over the n
 *     tokens seen so far; if K+1 tokens are cached, the budget partition of Section 3.3 keeps K of them
 *     (sinks = earliest cached tokens, recents = latest);
 *   - every voucher is multiplied by budget_decay (Algorithm 1 step 10).
 * All arrays DEVICE, owned, allocated and zero-initialised by the caller before the first step (next_slot: 0);
 * to continue from a prefilled cache fill them from the outputs of the one-shot calls instead (cache_len = number of
 * cached tokens, rows 0..cache_len-1 in position order, next_slot = cache_len, n_seen / hist / rings from the prompt).
 * Every unit holds the same number of tokens (cache_len); the call updates cache_len. policy->age_steps is ignored. */
typedef struct ta_stream {
  int32_t n_layers, batch, Hkv, K; /* U = n_layers*batch*Hkv units of K+1 slots; 1 <= K <= TA_MAX_BUDGET          */
  int32_t cache_len;               /* HOST scalar: tokens cached per unit before the step, 0..K; updated          */
  int32_t *pos, *slot, *tok;       /* [U][K+1] position, cache row and token id of the r-th cached token          */
  float *A, *P, *V;                /* [U][K+1] accumulated attention, pension average, voucher                    */
  uint8_t* S;                      /* [U][K+1] anchor-token indicator                                             */
  int32_t* next_slot;              /* [U] cache row for the next new token                                        */
  int32_t* n_seen;                 /* [B] tokens seen so far                                                      */
  int32_t* hist;                   /* [B][vocab_size] occurrences of every token id so far                        */
  int32_t* tok_ring;               /* [B][TA_MAX_PATTERN_LEN] the latest token ids, position t at index t % len   */
  float* anc_B;                    /* [B][TA_MAX_SPAN] budget of the anchor at position t (index t % span), else 0 */
  int32_t* anc_L;                  /* [B][TA_MAX_SPAN] its span, 0: no anchor                                      */
} ta_stream;

/* Context scratch one ta_stream_step needs. */
ta_status ta_stream_scratch_bytes(const ta_stream* st, size_t* out_bytes);

/*   new_ids      DEVICE int32 [B]        the new token of every sequence
 *   attn         DEVICE float [U][K+1]   attention mass of this step's query (summed over the unit's G query heads)
 *                                        on each CACHE ROW, the new token's own row (next_slot) included; rows that
 *                                        hold no token are not read
 *   evicted_pos  DEVICE int32 [U] out    position of the evicted token, -1 when nothing was evicted */
ta_status ta_stream_step(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, ta_stream* st /*HOST*/,
                         const int32_t* new_ids, const float* attn, int32_t* evicted_pos, void* stream);

/* ---- host-buffer variant of ta_compress --------------------------------------------------------------------
 * Same computation with every data pointer on the HOST (pinned memory makes the copies asynchronous):
 * token_ids, cu_seqlens (inside batch: HOST here), the q_obs / k / v views, and the four outputs. The caller lends
 * `workspace` (DEVICE, workspace_bytes >= ta_compress_host_workspace_bytes(...)) for the staged copies. Host to
 * device copies, kernels and device to host copies are all enqueued on `stream`. A V cache (and, in fast mode, a K
 * cache) that lies in pinned or registered host memory is not copied at all: only its retained rows are read, directly
 * over the bus, by the gather kernel. Views must be dense in the
 * order [L][B][Hkv or Hq][n or W][d] (ragged: [L][Hkv][total_tokens][d]); other strides return
 * TA_ERR_UNSUPPORTED. */
ta_status ta_compress_host_workspace_bytes(const ta_batch* batch, int Hq, int Hkv, int d, int K,
                                           const ta_policy* policy, size_t* out_bytes);
ta_status ta_compress_host(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                           int Hq, int Hkv, int d, int K, const int32_t* token_ids, const void* q_obs,
                           const void* k, const void* v, void* k_out, void* v_out, int32_t* idx, int32_t* count,
                           void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TA_H_ */
