// Host side of libta.so: argument validation, scratch carving and launch sequencing for the entry points declared
// in ta.h. Nothing here computes any part of the method; every step runs in the kernels of ta_mask.cu, ta_score.cu,
// ta_select.cu and ta_compact.cu.
#include <cuda.h>
#include <math.h>
#include <nvtx3/nvToolsExt.h>
#include <new>
#include <string.h>

#include "ta_internal.cuh"

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Carve {  // hands out aligned pieces of the context scratch
  uint8_t* base;
  size_t off = 0;
  explicit Carve(uint8_t* b) : base(b) {}
  template <class T>
  T* take(size_t count) {
    T* p = reinterpret_cast<T*>(base + off);
    off += align_up(count * sizeof(T));
    return p;
  }
};

struct Layout {  // scratch layout of ta_compress (a superset of what the single-step entry points need)
  size_t hist, flags, voucher, u_static, forced, r_main, idx_seq, count_seq, u, u_all, idx_lb, count_lb, order;
  size_t forced_cls, r_main_cls, class_K, class_of;  // budgets per (layer, head) only (n_classes > 0)
  size_t end;
};

Layout make_layout(const ta_batch& b, int Hkv, int K, const ta_policy& pol, int n_classes = 0) {
  Layout L;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes);
    return o;
  };
  const size_t total = (size_t)b.total_tokens, B = (size_t)b.batch;
  L.hist = take(B * (size_t)pol.vocab_size * 4);
  L.flags = take(total);
  L.voucher = take(total * 4);
  L.u_static = take(total * 4);
  L.forced = take(total);
  L.r_main = take(B * 4);
  L.idx_seq = take(B * (size_t)K * 4);
  L.count_seq = take(B * 4);
  L.u = take(pol.mode == TA_MODE_FAST ? 0 : (size_t)b.n_layers * Hkv * total * 4);
  // selection shared by the heads of a layer (ta_compress_allheads): head sums and the per-(layer, sequence) result
  const bool scored = pol.mode != TA_MODE_FAST;
  L.u_all = take(scored ? (size_t)b.n_layers * total * 4 : 0);
  L.idx_lb = take(scored ? (size_t)b.n_layers * B * K * 4 : 0);
  L.count_lb = take(scored ? (size_t)b.n_layers * B * 4 : 0);
  L.order = take(scored && b.cu_seqlens ? (size_t)b.n_layers * B * Hkv * 4 : 0);  // unit order of the score kernel
  L.forced_cls = take((size_t)n_classes * total);
  L.r_main_cls = take((size_t)n_classes * B * 4);
  L.class_K = take((size_t)n_classes * 4);
  L.class_of = take(n_classes > 0 ? (size_t)b.n_layers * Hkv * 4 : 0);
  L.end = off;
  return L;
}

ta_status check_batch(const ta_batch* b) {
  if (!b) return TA_ERR_INVALID_ARG;
  if (b->n_layers < 1 || b->batch < 1 || b->max_n < 0 || b->total_tokens < 0) return TA_ERR_INVALID_ARG;
  if (b->max_n > TA_MAX_SEQ_LEN) return TA_ERR_UNSUPPORTED;
  if (!b->cu_seqlens) {
    if (b->n_uniform < 0 || b->n_uniform > b->max_n) return TA_ERR_INVALID_ARG;
    if (b->total_tokens != (int64_t)b->batch * b->n_uniform) return TA_ERR_INVALID_ARG;
  }
  if (b->total_tokens > 0x7fffffffLL) return TA_ERR_UNSUPPORTED;
  return TA_OK;
}

ta_status check_policy(const ta_policy* p) {
  if (!p) return TA_ERR_INVALID_ARG;
  if (p->mode != TA_MODE_SCORED && p->mode != TA_MODE_FAST) return TA_ERR_INVALID_ARG;
  if (p->vocab_size < 1 || p->age_steps < 0 || p->n_sink < 0 || p->n_recent < 0) return TA_ERR_INVALID_ARG;
  if (p->softmax_scale < 0.0f || !(p->pension_rho >= 0.0f && p->pension_rho <= 1.0f)) return TA_ERR_INVALID_ARG;
  return TA_OK;
}

ta_status check_heads(int Hq, int Hkv, int d, const ta_policy* p, bool scored) {
  if (Hkv < 1 || Hq < Hkv || Hq % Hkv) return TA_ERR_INVALID_ARG;
  if (d != TA_HEAD_DIM) return TA_ERR_UNSUPPORTED;
  if (scored) {
    if (p->obs_window < 1) return TA_ERR_INVALID_ARG;
    if (p->obs_window > TA_MAX_WINDOW || (Hq / Hkv) * p->obs_window > TA_MAX_SCORE_ROWS || Hq / Hkv > 256)
      return TA_ERR_UNSUPPORTED;
  }
  return TA_OK;
}

ta_status check_view(const ta_bf16_view& v, bool need_b) {
  if (!v.ptr) return TA_ERR_INVALID_ARG;
  if ((uintptr_t)v.ptr % 16) return TA_ERR_ALIGNMENT;
  const int64_t s[4] = {v.stride_l, v.stride_b, v.stride_h, v.stride_n};
  for (int i = 0; i < 4; ++i) {
    if (i == 1 && !need_b) continue;
    if (s[i] < 0) return TA_ERR_INVALID_ARG;
    if (s[i] % 8) return TA_ERR_ALIGNMENT;
  }
  if (v.stride_n < TA_HEAD_DIM) return TA_ERR_INVALID_ARG;
  return TA_OK;
}

ta_seq_desc seq_desc(const ta_batch& b) {
  ta_seq_desc s;
  s.cu = b.cu_seqlens;
  s.n_uniform = b.n_uniform;
  s.batch = b.batch;
  s.max_n = b.max_n;
  s.total = b.total_tokens;
  return s;
}

ta_status cuda_fail(ta_ctx* ctx, cudaError_t e) {
  ctx->last_cuda_error = (int)e;
  return TA_ERR_CUDA;
}

struct Range {  // NVTX range around the host side of an entry point (what a timeline tool shows per call)
  explicit Range(const char* name) { nvtxRangePushA(name); }
  ~Range() { nvtxRangePop(); }
};

// What the per-sequence results cached under a seq_epoch depend on besides the token ids: every policy field that
// the mask, the static utility and the forced set read, and the pattern set.
uint64_t reuse_key(const ta_policy& p, const ta_patterns* pats) {
  uint64_t h = 1469598103934665603ull;
  auto mix = [&](const void* data, size_t n) {
    const unsigned char* b = static_cast<const unsigned char*>(data);
    for (size_t i = 0; i < n; ++i) h = (h ^ b[i]) * 1099511628211ull;
  };
  mix(&p.beta, sizeof p.beta);
  mix(&p.gamma, sizeof p.gamma);
  mix(&p.lambda, sizeof p.lambda);
  mix(&p.voucher_decay, sizeof p.voucher_decay);
  mix(&p.budget_decay, sizeof p.budget_decay);
  mix(&p.age_steps, sizeof p.age_steps);
  mix(&p.n_sink, sizeof p.n_sink);
  mix(&p.n_recent, sizeof p.n_recent);
  mix(&p.k_protected, sizeof p.k_protected);
  mix(&p.mode, sizeof p.mode);
  mix(&p.vocab_size, sizeof p.vocab_size);
  mix(&pats, sizeof pats);
  return h;
}

struct DeviceGuard {  // makes the context's device current for the duration of a call
  int prev = -1;
  bool ok;
  explicit DeviceGuard(int dev) {
    ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess);
    if (prev == dev) prev = -1;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

}  // namespace

extern "C" {

const char* ta_status_string(ta_status s) {
  switch (s) {
    case TA_OK: return "ok";
    case TA_ERR_INVALID_ARG: return "invalid argument";
    case TA_ERR_UNSUPPORTED: return "unsupported shape or device";
    case TA_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case TA_ERR_SCRATCH_TOO_SMALL: return "context scratch too small";
    case TA_ERR_CUDA: return "CUDA call failed";
    case TA_ERR_TIMEOUT: return "device wait timed out";
    case TA_ERR_DEVICE_BOUNDS: return "device-side bounds check failed";
  }
  return "unknown";
}

ta_status ta_policy_default(int preset, int K, ta_policy* out) {
  if (!out || K < 0) return TA_ERR_INVALID_ARG;
  ta_policy p;
  memset(&p, 0, sizeof p);
  p.alpha = 1.0f;
  p.beta = 0.5f;
  p.gamma = 0.3f;
  p.delta = 0.2f;
  p.lambda = 0.1f;
  p.voucher_decay = 0.8f;
  p.budget_decay = 0.9f;
  p.age_steps = 0;
  p.obs_window = 32;
  p.pension_rho = 0.9f;
  p.softmax_scale = 0.0f;
  p.causal = 1;
  p.mode = TA_MODE_SCORED;
  p.vocab_size = 32000;
  switch (preset) {
    case TA_PRESET_THEOREM: p.n_sink = 1; p.n_recent = 4; p.k_protected = -1; break;
    case TA_PRESET_SEC33: p.n_sink = 1; p.n_recent = 2; p.k_protected = K / 4; break;
    case TA_PRESET_AUDIT: p.n_sink = 4; p.n_recent = 6; p.k_protected = 6; break;
    default: return TA_ERR_INVALID_ARG;
  }
  *out = p;
  return TA_OK;
}

ta_status ta_ctx_create(int device, size_t scratch_bytes, ta_ctx** out) {
  if (!out) return TA_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return TA_ERR_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return TA_ERR_CUDA;
  if (prop.major != 10) return TA_ERR_UNSUPPORTED;  // the kernels are built for sm_100a only
  DeviceGuard guard(device);
  if (!guard.ok) return TA_ERR_CUDA;
  ta_ctx* c = new (std::nothrow) ta_ctx();
  if (!c) return TA_ERR_CUDA;
  memset(c, 0, sizeof *c);
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->scratch_bytes = scratch_bytes;
  cudaError_t e = cudaMalloc(&c->d_status, sizeof(ta_dev_status));
  if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, sizeof(ta_dev_status));
  if (e == cudaSuccess && scratch_bytes) e = cudaMalloc(&c->scratch, scratch_bytes);
  for (int i = 0; e == cudaSuccess && i < 8; ++i) e = cudaEventCreate(&c->ev[i]);
  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
  if (e == cudaSuccess) {
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &q);
    if (e == cudaSuccess && (q != cudaDriverEntryPointSuccess || !c->encode_tiled)) e = cudaErrorNotSupported;
  }
  if (e != cudaSuccess) {
    ta_ctx_destroy(c);
    return TA_ERR_CUDA;
  }
  *out = c;
  return TA_OK;
}

void ta_ctx_destroy(ta_ctx* c) {
  if (!c) return;
  DeviceGuard guard(c->device);
  for (int i = 0; i < 8; ++i)
    if (c->ev[i]) cudaEventDestroy(c->ev[i]);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->side) cudaStreamDestroy(c->side);
  if (c->scratch) cudaFree(c->scratch);
  if (c->d_status) cudaFree(c->d_status);
  delete c;
}

ta_status ta_scratch_bytes(const ta_batch* batch, int Hq, int Hkv, int d, int K, const ta_policy* policy,
                           size_t* out_bytes) {
  (void)Hq;
  (void)d;
  if (!out_bytes) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (K < 1 || Hkv < 1) return TA_ERR_INVALID_ARG;
  *out_bytes = make_layout(*batch, Hkv, K, *policy).end + kAlign;
  return TA_OK;
}

ta_status ta_scratch_bytes_budgets(const ta_batch* batch, int Hkv, int K_max, const ta_policy* policy,
                                   int n_budget_classes, size_t* out_bytes) {
  if (!out_bytes) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (K_max < 1 || Hkv < 1 || n_budget_classes < 1) return TA_ERR_INVALID_ARG;
  if (n_budget_classes > TA_MAX_BUDGET_CLASSES) return TA_ERR_UNSUPPORTED;
  *out_bytes = make_layout(*batch, Hkv, K_max, *policy, n_budget_classes).end + kAlign;
  return TA_OK;
}

ta_status ta_ctx_poll(ta_ctx* ctx) {
  if (!ctx) return TA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  ta_dev_status st;
  e = cudaMemcpy(&st, ctx->d_status, sizeof st, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  if (st.code != 0) {
    cudaMemset(ctx->d_status, 0, sizeof st);
    ctx->cached_epoch = 0;
    return (ta_status)st.code;
  }
  return TA_OK;
}

int ta_ctx_last_cuda_error(const ta_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }

ta_status ta_ctx_set_wait_limit(ta_ctx* ctx, uint64_t nanoseconds) {
  if (!ctx) return TA_ERR_INVALID_ARG;
  ctx->wait_limit_ns = nanoseconds;
  return TA_OK;
}

ta_status ta_ctx_set_score_cluster(ta_ctx* ctx, int ctas_per_unit) {
  if (!ctx) return TA_ERR_INVALID_ARG;
  if (ctas_per_unit != 0 && ctas_per_unit != 1 && ctas_per_unit != 2 && ctas_per_unit != 4 && ctas_per_unit != 8)
    return TA_ERR_INVALID_ARG;
  ctx->score_force_cluster = ctas_per_unit;
  return TA_OK;
}

ta_status ta_ctx_selftest_wait(ta_ctx* ctx, uint64_t limit_ns, int32_t* outcome, void* stream) {
  if (!ctx || !outcome || limit_ns == 0 || limit_ns > 1000000000ull) return TA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaError_t e = ta_launch_wait_selftest(ctx->d_status, limit_ns, outcome, (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

ta_status ta_ctx_last_launch_info(const ta_ctx* ctx, int32_t out[4]) {
  if (!ctx || !out) return TA_ERR_INVALID_ARG;
  out[0] = ctx->score_cluster;
  out[1] = ctx->score_clusters;
  out[2] = ctx->last_select_gathered;
  out[3] = ctx->last_kernel_launches;
  return TA_OK;
}

ta_status ta_ctx_enable_timing(ta_ctx* ctx, int enable) {
  if (!ctx) return TA_ERR_INVALID_ARG;
  ctx->timing_enabled = enable ? 1 : 0;
  ctx->timing_valid = 0;
  return TA_OK;
}

ta_status ta_ctx_read_timing(ta_ctx* ctx, float out_ms[5]) {
  if (!ctx || !out_ms) return TA_ERR_INVALID_ARG;
  for (int i = 0; i < 5; ++i) out_ms[i] = 0.0f;
  if (!ctx->timing_valid) return TA_ERR_INVALID_ARG;
  DeviceGuard guard(ctx->device);
  cudaError_t e = cudaEventSynchronize(ctx->ev[4]);
  if (e == cudaSuccess && ctx->ev_ran[0]) {  // per-sequence work runs on the side stream, beside the score kernel
    e = cudaEventSynchronize(ctx->ev[6]);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&out_ms[0], ctx->ev[5], ctx->ev[6]);
  }
  for (int i = 1; e == cudaSuccess && i < 4; ++i) e = cudaEventElapsedTime(&out_ms[i], ctx->ev[i], ctx->ev[i + 1]);
  if (e == cudaSuccess) e = cudaEventElapsedTime(&out_ms[4], ctx->ev[0], ctx->ev[4]);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

// ---------------------------------------------------------------------------------------------- patterns
ta_status ta_patterns_create(ta_ctx* ctx, int n_pat, const int32_t* ids_flat, const int32_t* offsets,
                             const float* budget, const int32_t* span, ta_patterns** out) {
  if (!ctx || !out || n_pat < 0 || (n_pat > 0 && (!ids_flat || !offsets))) return TA_ERR_INVALID_ARG;
  *out = nullptr;
  if (n_pat > TA_MAX_PATTERNS) return TA_ERR_UNSUPPORTED;
  const int np = n_pat > 0 ? n_pat : 1;
  int32_t* h_ids = new (std::nothrow) int32_t[np * TA_MAX_PATTERN_LEN];
  int32_t h_len[TA_MAX_PATTERNS], h_span[TA_MAX_PATTERNS];
  float h_bud[TA_MAX_PATTERNS];
  uint32_t h_bloom[32];
  if (!h_ids) return TA_ERR_CUDA;
  memset(h_bloom, 0, sizeof h_bloom);
  for (int i = 0; i < np * TA_MAX_PATTERN_LEN; ++i) h_ids[i] = -1;
  int max_len = 0, max_span = 0;
  ta_status bad = TA_OK;
  for (int p = 0; p < n_pat && bad == TA_OK; ++p) {
    const int len = offsets[p + 1] - offsets[p];
    const int sp = span ? span[p] : 6;
    const float bu = budget ? budget[p] : 15.0f;
    if (len < 1 || sp < 1 || !(bu == bu)) bad = TA_ERR_INVALID_ARG;
    else if (len > TA_MAX_PATTERN_LEN || sp > TA_MAX_SPAN) bad = TA_ERR_UNSUPPORTED;
    else {
      for (int k = 0; k < len; ++k) {
        const int32_t id = ids_flat[offsets[p] + k];
        if (id < 0) bad = TA_ERR_INVALID_ARG;
        h_ids[p * TA_MAX_PATTERN_LEN + k] = id;
      }
      const uint32_t h = ((uint32_t)h_ids[p * TA_MAX_PATTERN_LEN + len - 1] * 2654435761u) >> 22;
      h_bloom[h >> 5] |= 1u << (h & 31);
      h_len[p] = len;
      h_span[p] = sp;
      h_bud[p] = bu;
      if (len > max_len) max_len = len;
      if (sp > max_span) max_span = sp;
    }
  }
  if (bad != TA_OK) {
    delete[] h_ids;
    return bad;
  }
  if (n_pat == 0) {
    h_len[0] = 0;
    h_span[0] = 0;
    h_bud[0] = 0.0f;
  }
  DeviceGuard guard(ctx->device);
  ta_patterns* P = new (std::nothrow) ta_patterns();
  if (!P) {
    delete[] h_ids;
    return TA_ERR_CUDA;
  }
  memset(P, 0, sizeof *P);
  P->device = ctx->device;
  P->n_pat = n_pat;
  P->max_len = max_len;
  P->max_span = max_span;
  cudaError_t e = cudaMalloc(&P->d_ids, sizeof(int32_t) * np * TA_MAX_PATTERN_LEN);
  if (e == cudaSuccess) e = cudaMalloc(&P->d_len, sizeof(int32_t) * np);
  if (e == cudaSuccess) e = cudaMalloc(&P->d_budget, sizeof(float) * np);
  if (e == cudaSuccess) e = cudaMalloc(&P->d_span, sizeof(int32_t) * np);
  if (e == cudaSuccess) e = cudaMalloc(&P->d_bloom, sizeof h_bloom);
  if (e == cudaSuccess) e = cudaMemcpy(P->d_ids, h_ids, sizeof(int32_t) * np * TA_MAX_PATTERN_LEN, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(P->d_len, h_len, sizeof(int32_t) * np, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(P->d_budget, h_bud, sizeof(float) * np, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(P->d_span, h_span, sizeof(int32_t) * np, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMemcpy(P->d_bloom, h_bloom, sizeof h_bloom, cudaMemcpyHostToDevice);
  delete[] h_ids;
  if (e != cudaSuccess) {
    ta_patterns_destroy(P);
    return cuda_fail(ctx, e);
  }
  *out = P;
  return TA_OK;
}

void ta_patterns_destroy(ta_patterns* P) {
  if (!P) return;
  DeviceGuard guard(P->device);
  if (P->d_ids) cudaFree(P->d_ids);
  if (P->d_len) cudaFree(P->d_len);
  if (P->d_budget) cudaFree(P->d_budget);
  if (P->d_span) cudaFree(P->d_span);
  if (P->d_bloom) cudaFree(P->d_bloom);
  delete P;
}

// ---------------------------------------------------------------------------------------------- step 1
ta_status ta_sponsor_mask(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                          const int32_t* token_ids, uint8_t* flags, float* voucher, float* u_static, void* stream) {
  Range range("ta_sponsor_mask");
  if (!ctx || !pats || !token_ids || !flags || !voucher || !u_static) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (pats->device != ctx->device) return TA_ERR_INVALID_ARG;
  const size_t need = align_up((size_t)batch->batch * policy->vocab_size * 4);
  if (need > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  ctx->cached_epoch = 0;
  cudaError_t e = ta_launch_mask(pats, *policy, seq_desc(*batch), token_ids, flags, voucher, u_static,
                                 reinterpret_cast<int32_t*>(ctx->scratch), ctx->d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

ta_status ta_detect_embedding(ta_ctx* ctx, int64_t total_tokens, const void* emb, int64_t stride_tok, int D,
                              const void* concepts, int n_concepts, float* conf, void* stream) {
  Range range("ta_detect_embedding");
  if (!ctx || !emb || !concepts || !conf || total_tokens < 0) return TA_ERR_INVALID_ARG;
  if (D < 32 || n_concepts < 1 || stride_tok < D) return TA_ERR_INVALID_ARG;
  if (D % 32 || D > TA_MAX_EMBED_DIM || n_concepts > TA_MAX_CONCEPTS) return TA_ERR_UNSUPPORTED;
  if ((uintptr_t)emb % 16 || (uintptr_t)concepts % 2 || stride_tok % 8) return TA_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  cudaError_t e = ta_launch_embed_conf(ctx->sm_count, total_tokens, emb, stride_tok, D, concepts, n_concepts, conf,
                                       (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

ta_status ta_sponsor_mask_conf(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, const int32_t* token_ids,
                               const float* conf, float threshold, float budget, int span, int rank_by_confidence,
                               uint8_t* flags, float* voucher, float* u_static, void* stream) {
  Range range("ta_sponsor_mask_conf");
  if (!ctx || !token_ids || !conf || !flags || !voucher || !u_static) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (!(threshold == threshold) || !(budget == budget) || span < 1) return TA_ERR_INVALID_ARG;
  if (span > TA_MAX_SPAN) return TA_ERR_UNSUPPORTED;
  const size_t need = align_up((size_t)batch->batch * policy->vocab_size * 4);
  if (need > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  ctx->cached_epoch = 0;
  cudaError_t e = ta_launch_mask_conf(*policy, seq_desc(*batch), token_ids, conf, threshold, budget, span,
                                      rank_by_confidence ? 1 : 0, flags, voucher, u_static,
                                      reinterpret_cast<int32_t*>(ctx->scratch), ctx->d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

// ---------------------------------------------------------------------------------------------- step 2
static ta_status score_impl(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                            ta_bf16_view q_obs, ta_bf16_view k, const float* lse_obs, float* A, float* P, float* u,
                            void* stream) {
  Range range("ta_score");
  if (!ctx || (!A && !u)) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s == TA_OK) s = check_heads(Hq, Hkv, d, policy, true);
  if (s == TA_OK) s = check_view(q_obs, true);
  if (s == TA_OK) s = check_view(k, batch->cu_seqlens == nullptr);
  if (s != TA_OK) return s;
  DeviceGuard guard(ctx->device);
  ta_score_args a = {};
  a.seq = seq_desc(*batch);
  a.n_layers = batch->n_layers;
  a.Hq = Hq;
  a.Hkv = Hkv;
  a.W = policy->obs_window;
  a.q = q_obs;
  a.k = k;
  a.lse_obs = lse_obs;
  a.A = A;
  a.P = P;
  a.u = u;
  a.alpha = policy->alpha;
  a.delta = policy->delta;
  a.rho = policy->pension_rho;
  a.scale = policy->softmax_scale;
  a.causal = policy->causal;
  // ragged batches: the unit order of the score kernel lives at the start of the context scratch when there is room
  // (whatever ta_compress cached there is dropped)
  if (batch->cu_seqlens && ctx->scratch_bytes >= (size_t)batch->n_layers * batch->batch * Hkv * 4) {
    a.order_scratch = reinterpret_cast<int32_t*>(ctx->scratch);
    ctx->cached_epoch = 0;
  }
  cudaError_t e = ta_launch_score(ctx, a, ctx->d_status, (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

ta_status ta_score(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                   ta_bf16_view q_obs, ta_bf16_view k, const float* lse_obs, float* A, float* P, void* stream) {
  if (!A) return TA_ERR_INVALID_ARG;
  return score_impl(ctx, policy, batch, Hq, Hkv, d, q_obs, k, lse_obs, A, P, nullptr, stream);
}

ta_status ta_score_weighted(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                            ta_bf16_view q_obs, ta_bf16_view k, const float* lse_obs, float* u_att, void* stream) {
  if (!u_att) return TA_ERR_INVALID_ARG;
  return score_impl(ctx, policy, batch, Hq, Hkv, d, q_obs, k, lse_obs, nullptr, nullptr, u_att, stream);
}

// ---------------------------------------------------------------------------------------------- step 3
ta_status ta_select_topk(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hkv, int K,
                         const uint8_t* flags, const float* voucher, const float* u_static, const float* A,
                         const float* P, int32_t* idx, int32_t* count, void* stream) {
  Range range("ta_select_topk");
  if (!ctx || !flags || !voucher || !u_static || !idx || !count) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (Hkv < 1 || K < 1) return TA_ERR_INVALID_ARG;
  if (K > TA_MAX_BUDGET) return TA_ERR_UNSUPPORTED;
  const bool fast = policy->mode == TA_MODE_FAST;
  if (!fast && !A) return TA_ERR_INVALID_ARG;
  Carve carve(ctx->scratch);
  uint8_t* forced = carve.take<uint8_t>((size_t)batch->total_tokens);
  int32_t* r_main = carve.take<int32_t>((size_t)batch->batch);
  int32_t* idx_seq = carve.take<int32_t>(fast ? (size_t)batch->batch * K : 0);
  int32_t* count_seq = carve.take<int32_t>(fast ? (size_t)batch->batch : 0);
  if (carve.off > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  ctx->cached_epoch = 0;
  ta_select_args a = {};
  a.seq = seq_desc(*batch);
  a.n_layers = batch->n_layers;
  a.Hkv = Hkv;
  a.K = K;
  a.n_sink = policy->n_sink;
  a.n_recent = policy->n_recent;
  a.k_protected = policy->k_protected;
  a.fast = fast;
  a.sm_count = ctx->sm_count;
  a.alpha = policy->alpha;
  a.delta = policy->delta;
  a.flags = flags;
  a.voucher = voucher;
  a.u_static = u_static;
  a.A = A;
  a.P = P;
  a.u = nullptr;
  a.forced = forced;
  a.r_main = r_main;
  a.idx = fast ? idx_seq : idx;
  a.count = fast ? count_seq : count;
  cudaError_t e = ta_launch_select(a, ctx->d_status, (cudaStream_t)stream);
  if (e == cudaSuccess && fast)
    e = ta_launch_broadcast_idx(batch->batch, Hkv, K, batch->n_layers, idx_seq, count_seq, idx, count,
                                (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

// ---------------------------------------------------------------------------------------------- step 4
ta_status ta_compact_kv(ta_ctx* ctx, const ta_batch* batch, int Hkv, int d, int K, ta_bf16_view k, ta_bf16_view v,
                        const int32_t* idx, const int32_t* count, void* k_out, void* v_out, void* stream) {
  Range range("ta_compact_kv");
  if (!ctx || !idx || !count || !k_out || !v_out) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s != TA_OK) return s;
  if (Hkv < 1 || K < 1) return TA_ERR_INVALID_ARG;
  if (d != TA_HEAD_DIM || K > TA_MAX_BUDGET) return TA_ERR_UNSUPPORTED;
  const bool uniform = batch->cu_seqlens == nullptr;
  s = check_view(k, uniform);
  if (s == TA_OK) s = check_view(v, uniform);
  if (s != TA_OK) return s;
  if ((uintptr_t)k_out % 16 || (uintptr_t)v_out % 16) return TA_ERR_ALIGNMENT;
  DeviceGuard guard(ctx->device);
  ta_compact_args a = {};
  a.seq = seq_desc(*batch);
  a.n_layers = batch->n_layers;
  a.Hkv = Hkv;
  a.K = K;
  a.k = k;
  a.v = v;
  a.idx = idx;
  a.count = count;
  a.k_out = k_out;
  a.v_out = v_out;
  cudaError_t e = ta_launch_compact(a, ctx->sm_count, (cudaStream_t)stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

// ---------------------------------------------------------------------------------------------- fused
namespace {
// ext_A != nullptr: the attention terms come from the caller (ext_A, ext_P per layer, KV head and token) and the
// score kernel is not run; q_obs is then unused.
ta_status compress_impl(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch, int Hq,
                        int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs, ta_bf16_view k,
                        ta_bf16_view v, uint64_t seq_epoch, void* k_out, void* v_out, int32_t* idx, int32_t* count,
                        void* stream_v, const float* ext_A, const float* ext_P, bool share_heads,
                        const int32_t* budgets = nullptr, const float* ext_u_all = nullptr,
                        const float* lse_obs = nullptr) {
  Range range("ta_compress");
  if (!ctx || !pats || !token_ids || !k_out || !v_out || !idx || !count) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  const bool fast = policy->mode == TA_MODE_FAST;
  // ext_u_all: the head-summed attention part comes from the caller (head-sharded layers); implies share_heads
  const bool external = ext_A != nullptr || ext_u_all != nullptr;
  if ((external || share_heads) && fast) return TA_ERR_INVALID_ARG;
  if (ext_A && share_heads) return TA_ERR_INVALID_ARG;
  if (ext_u_all && (!share_heads || budgets)) return TA_ERR_INVALID_ARG;
  const bool uniform = batch->cu_seqlens == nullptr;
  s = check_heads(Hq, Hkv, d, policy, !fast && !external);
  if (s == TA_OK && !fast && !external) s = check_view(q_obs, true);
  if (s == TA_OK) s = check_view(v, uniform);
  if (s == TA_OK && k.ptr == nullptr) s = TA_ERR_INVALID_ARG;  // K rows are gathered in every mode
  if (s == TA_OK) s = check_view(k, uniform);
  if (s != TA_OK) return s;
  if (K < 1) return TA_ERR_INVALID_ARG;
  if (K > TA_MAX_BUDGET) return TA_ERR_UNSUPPORTED;
  if ((uintptr_t)k_out % 16 || (uintptr_t)v_out % 16) return TA_ERR_ALIGNMENT;
  if (pats->device != ctx->device) return TA_ERR_INVALID_ARG;
  // budgets per (layer, KV head): pairs with equal budgets form a class (HOST work on at most kMaxPairs entries)
  constexpr int kMaxPairs = 4096;
  int n_classes = 0;
  int32_t class_K_h[TA_MAX_BUDGET_CLASSES];
  int32_t class_of_h[kMaxPairs];
  if (budgets) {
    if (fast || share_heads) return TA_ERR_INVALID_ARG;
    const long long pairs = (long long)batch->n_layers * Hkv;
    if (pairs > kMaxPairs) return TA_ERR_UNSUPPORTED;
    for (int i = 0; i < (int)pairs; ++i) {
      if (budgets[i] < 1 || budgets[i] > K) return TA_ERR_INVALID_ARG;
      int c = 0;
      while (c < n_classes && class_K_h[c] != budgets[i]) ++c;
      if (c == n_classes) {
        if (n_classes == TA_MAX_BUDGET_CLASSES) return TA_ERR_UNSUPPORTED;
        class_K_h[n_classes++] = budgets[i];
      }
      class_of_h[i] = c;
    }
  }
  const Layout L = make_layout(*batch, Hkv, K, *policy, n_classes);
  if (L.end > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;

  DeviceGuard guard(ctx->device);
  cudaStream_t stream = (cudaStream_t)stream_v;
  uint8_t* sc = ctx->scratch;
  int32_t* hist = reinterpret_cast<int32_t*>(sc + L.hist);
  uint8_t* flags = sc + L.flags;
  float* voucher = reinterpret_cast<float*>(sc + L.voucher);
  float* u_static = reinterpret_cast<float*>(sc + L.u_static);
  uint8_t* forced = sc + L.forced;
  int32_t* r_main = reinterpret_cast<int32_t*>(sc + L.r_main);
  int32_t* idx_seq = reinterpret_cast<int32_t*>(sc + L.idx_seq);
  int32_t* count_seq = reinterpret_cast<int32_t*>(sc + L.count_seq);
  float* u = reinterpret_cast<float*>(sc + L.u);
  float* u_all = reinterpret_cast<float*>(sc + L.u_all);
  int32_t* idx_lb = reinterpret_cast<int32_t*>(sc + L.idx_lb);
  int32_t* count_lb = reinterpret_cast<int32_t*>(sc + L.count_lb);
  const ta_seq_desc seq = seq_desc(*batch);
  const bool timing = ctx->timing_enabled != 0;
  cudaError_t e = cudaSuccess;
  auto mark = [&](int i) {
    if (timing && e == cudaSuccess) e = cudaEventRecord(ctx->ev[i], stream);
  };

  // (with budget classes the forced sets live elsewhere and depend on the budgets: nothing is reused or cached)
  const uint64_t key = reuse_key(*policy, pats);
  const bool reuse = !budgets && seq_epoch != 0 && seq_epoch == ctx->cached_epoch && key == ctx->cached_key &&
                     ctx->cached_total == batch->total_tokens && ctx->cached_batch == batch->batch && ctx->cached_K == K;
  ta_select_args sel = {};
  sel.seq = seq;
  sel.n_layers = batch->n_layers;
  sel.Hkv = Hkv;
  sel.K = K;
  sel.n_sink = policy->n_sink;
  sel.n_recent = policy->n_recent;
  sel.k_protected = policy->k_protected;
  sel.fast = fast;
  sel.sm_count = ctx->sm_count;
  sel.alpha = policy->alpha;
  sel.delta = policy->delta;
  sel.flags = flags;
  sel.voucher = voucher;
  sel.u_static = u_static;
  // the forced-set kernel writes the static utilities of its sequence (one kernel less on the per-sequence chain)
  sel.static_out = u_static;
  sel.static_ids = token_ids;
  sel.static_hist = hist;
  sel.static_vocab = policy->vocab_size;
  sel.beta = policy->beta;
  sel.gamma = policy->gamma;
  sel.lambda = policy->lambda;
  sel.u = external ? nullptr : u;
  sel.A = ext_A;
  sel.P = ext_P;
  sel.forced = forced;
  sel.r_main = r_main;
  sel.idx = fast ? idx_seq : idx;
  sel.count = fast ? count_seq : count;
  if (share_heads) {  // one selection per (layer, sequence) on the head sums
    sel.Hkv = 1;
    sel.u = ext_u_all ? ext_u_all : u_all;
    sel.idx = idx_lb;
    sel.count = count_lb;
  } else if (!fast) {  // small budgets: the selecting block gathers the unit's rows itself
    sel.gather_k = k;
    sel.gather_v = v;
    sel.gather_k_out = k_out;
    sel.gather_v_out = v_out;
  }
  if (budgets) {
    sel.n_classes = n_classes;
    sel.forced = sc + L.forced_cls;
    sel.r_main = reinterpret_cast<int32_t*>(sc + L.r_main_cls);
    sel.class_K = reinterpret_cast<const int32_t*>(sc + L.class_K);
    sel.class_of = reinterpret_cast<const int32_t*>(sc + L.class_of);
    // the host arrays are pageable: the copies are staged before the calls return
    e = cudaMemcpyAsync(sc + L.class_K, class_K_h, (size_t)n_classes * 4, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(sc + L.class_of, class_of_h, (size_t)batch->n_layers * Hkv * 4, cudaMemcpyHostToDevice, stream);
  }
  const bool select_gathers = ta_select_gathers(sel);
  ctx->last_select_gathered = select_gathers ? 1 : 0;
  int launches = 0;  // kernels of this library enqueued by this call

  // Per-sequence work (anchor mask, vouchers, static utility, forced set) does not depend on Q/K: in scored mode it
  // runs on the context's side stream beside the score kernel and joins before the per-unit selection.
  mark(0);
  ctx->ev_ran[0] = 0;
  cudaStream_t seq_stream = stream;
  // ...but only while the score kernel is short. It is persistent, so kernels beside it need SMs of their own (4 are
  // left free); a long score kernel gains more from those SMs than the step gains from hiding the per-sequence work,
  // which then simply runs first.
  const long long score_jobs = (lse_obs ? 1LL : 2LL) * batch->n_layers * batch->batch * Hkv * ((batch->max_n + 127) / 128) *
                               (((Hq / Hkv) * policy->obs_window + 127) / 128);
  const bool fork = !reuse && !fast && !external && score_jobs <= 400LL * ctx->sm_count;
  // Kernels of the chain that directly follow another kernel of the chain on their stream are launched as its
  // programmatic dependents: their launch overlaps its tail, and they wait for it before they touch memory. The
  // forced-set kernel follows the mask kernel; the selection follows the score kernel, the forced-set kernel or the
  // head sum (not across the join with the side stream); the broadcast and the gather follow the selection.
  sel.pdl_forced = 1;
  sel.pdl_units = fork ? 0 : 1;
  if (fork) {
    seq_stream = ctx->side;
    e = cudaEventRecord(ctx->ev_fork, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0);
  }
  if (!reuse) {
    if (timing && e == cudaSuccess) e = cudaEventRecord(ctx->ev[5], seq_stream);
    if (e == cudaSuccess)
      e = ta_launch_mask(pats, *policy, seq, token_ids, flags, voucher, nullptr, hist, ctx->d_status, seq_stream);
    if (e == cudaSuccess) e = ta_launch_forced(sel, ctx->d_status, seq_stream);
    launches += 2;  // mask, forced set (which also writes the static utilities)
    if (timing && e == cudaSuccess) {
      e = cudaEventRecord(ctx->ev[6], seq_stream);
      ctx->ev_ran[0] = 1;
    }
  }
  if (fork && e == cudaSuccess) e = cudaEventRecord(ctx->ev_join, ctx->side);
  mark(1);
  if (e == cudaSuccess && !fast && !external) {
    ta_score_args a = {};
    a.seq = seq;
    a.n_layers = batch->n_layers;
    a.Hq = Hq;
    a.Hkv = Hkv;
    a.W = policy->obs_window;
    a.q = q_obs;
    a.k = k;
    a.lse_obs = lse_obs;  // the rows' normalisers from the caller's prefill kernel: one pass over the keys
    a.A = nullptr;
    a.P = nullptr;
    a.u = u;
      a.alpha = policy->alpha;
    a.delta = policy->delta;
    a.rho = policy->pension_rho;
    a.scale = policy->softmax_scale;
    a.causal = policy->causal;
    a.reserve_sms = fork ? 4 : 0;
    a.order_scratch = batch->cu_seqlens ? reinterpret_cast<int32_t*>(sc + L.order) : nullptr;
    e = ta_launch_score(ctx, a, ctx->d_status, stream);
    launches += a.order_scratch && batch->batch > 1 ? 2 : 1;  // (unit order of a ragged batch,) score
  }
  mark(2);
  if (fork && e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->ev_join, 0);
  if (e == cudaSuccess && share_heads && !ext_u_all)
    e = ta_launch_headsum(batch->n_layers, Hkv, batch->total_tokens, u, u_all, stream);
  if (e == cudaSuccess && !(fast && reuse)) e = ta_launch_select_units(sel, stream);
  launches += (share_heads ? 2 : 0) + (fast && reuse ? 0 : 1) + (fast ? 1 : 0) + (select_gathers ? 0 : 1);
  if (e == cudaSuccess && share_heads)
    e = ta_launch_broadcast_heads(batch->n_layers, batch->batch, Hkv, K, idx_lb, count_lb, idx, count, stream);
  if (e == cudaSuccess && fast)
    e = ta_launch_broadcast_idx(batch->batch, Hkv, K, batch->n_layers, idx_seq, count_seq, idx, count, stream, true);
  mark(3);
  if (e == cudaSuccess && !select_gathers) {
    ta_compact_args a = {};
    a.seq = seq;
    a.n_layers = batch->n_layers;
    a.Hkv = Hkv;
    a.K = K;
    a.k = k;
    a.v = v;
    a.idx = idx;
    a.count = count;
    a.k_out = k_out;
    a.v_out = v_out;
    a.pdl = 1;
    e = ta_launch_compact(a, ctx->sm_count, stream);
  }
  mark(4);
  if (e != cudaSuccess) {
    ctx->cached_epoch = 0;
    return cuda_fail(ctx, e);
  }
  ctx->timing_valid = timing ? 1 : 0;
  ctx->last_kernel_launches = launches;
  ctx->cached_epoch = budgets ? 0 : seq_epoch;
  ctx->cached_total = batch->total_tokens;
  ctx->cached_batch = batch->batch;
  ctx->cached_K = K;
  ctx->cached_key = key;
  return TA_OK;
}
}  // namespace

ta_status ta_compress(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch, int Hq,
                      int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs, ta_bf16_view k,
                      ta_bf16_view v, uint64_t seq_epoch, void* k_out, void* v_out, int32_t* idx, int32_t* count,
                      void* stream) {
  return compress_impl(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs, k, v, seq_epoch, k_out, v_out, idx,
                       count, stream, nullptr, nullptr, false);
}

ta_status ta_compress_lse(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch, int Hq,
                          int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs, ta_bf16_view k,
                          ta_bf16_view v, const float* lse_obs, uint64_t seq_epoch, void* k_out, void* v_out,
                          int32_t* idx, int32_t* count, void* stream) {
  if (!policy || !lse_obs) return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  return compress_impl(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs, k, v, seq_epoch, k_out, v_out, idx,
                       count, stream, nullptr, nullptr, false, nullptr, nullptr, lse_obs);
}

ta_status ta_compress_allheads(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                               int Hq, int Hkv, int d, int K, const int32_t* token_ids, ta_bf16_view q_obs,
                               ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch, void* k_out, void* v_out,
                               int32_t* idx, int32_t* count, void* stream) {
  if (!policy || policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  return compress_impl(ctx, pats, policy, batch, Hq, Hkv, d, K, token_ids, q_obs, k, v, seq_epoch, k_out, v_out, idx,
                       count, stream, nullptr, nullptr, true);
}

ta_status ta_score_headsum(ta_ctx* ctx, const ta_policy* policy, const ta_batch* batch, int Hq, int Hkv, int d,
                           ta_bf16_view q_obs, ta_bf16_view k, float* u_heads, void* stream_v) {
  Range range("ta_score_headsum");
  if (!ctx || !u_heads) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s == TA_OK && policy->mode != TA_MODE_SCORED) s = TA_ERR_INVALID_ARG;
  if (s == TA_OK) s = check_heads(Hq, Hkv, d, policy, true);
  if (s == TA_OK) s = check_view(q_obs, true);
  if (s == TA_OK) s = check_view(k, batch->cu_seqlens == nullptr);
  if (s != TA_OK) return s;
  const Layout L = make_layout(*batch, Hkv, 1, *policy);
  if (L.end > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = (cudaStream_t)stream_v;
  ctx->cached_epoch = 0;  // the per-unit utilities share the scratch with ta_compress's cache
  float* u = reinterpret_cast<float*>(ctx->scratch + L.u);
  ta_score_args a = {};
  a.seq = seq_desc(*batch);
  a.n_layers = batch->n_layers;
  a.Hq = Hq;
  a.Hkv = Hkv;
  a.W = policy->obs_window;
  a.q = q_obs;
  a.k = k;
  a.u = u;
  a.alpha = policy->alpha;
  a.delta = policy->delta;
  a.rho = policy->pension_rho;
  a.scale = policy->softmax_scale;
  a.causal = policy->causal;
  a.order_scratch = batch->cu_seqlens ? reinterpret_cast<int32_t*>(ctx->scratch + L.order) : nullptr;
  cudaError_t e = ta_launch_score(ctx, a, ctx->d_status, stream);
  if (e == cudaSuccess) e = ta_launch_headsum(batch->n_layers, Hkv, batch->total_tokens, u, u_heads, stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

ta_status ta_compress_from_headsum(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy,
                                   const ta_batch* batch, int Hkv, int d, int K, const int32_t* token_ids,
                                   const float* u_heads, ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch,
                                   void* k_out, void* v_out, int32_t* idx, int32_t* count, void* stream) {
  if (!policy || !u_heads) return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  ta_bf16_view none = {};
  return compress_impl(ctx, pats, policy, batch, Hkv, Hkv, d, K, token_ids, none, k, v, seq_epoch, k_out, v_out, idx,
                       count, stream, nullptr, nullptr, true, nullptr, u_heads);
}

ta_status ta_compress_scores(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                             int Hkv, int d, int K, const int32_t* token_ids, const float* score,
                             const float* score2, ta_bf16_view k, ta_bf16_view v, uint64_t seq_epoch, void* k_out,
                             void* v_out, int32_t* idx, int32_t* count, void* stream) {
  if (!score || !policy) return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  ta_bf16_view none = {};
  return compress_impl(ctx, pats, policy, batch, Hkv, Hkv, d, K, token_ids, none, k, v, seq_epoch, k_out, v_out, idx,
                       count, stream, score, score2, false);
}

ta_status ta_compress_scores_budgets(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy,
                                     const ta_batch* batch, int Hkv, int d, int K_max, const int32_t* budgets,
                                     const int32_t* token_ids, const float* score, const float* score2,
                                     ta_bf16_view k, ta_bf16_view v, void* k_out, void* v_out, int32_t* idx,
                                     int32_t* count, void* stream) {
  if (!score || !policy || !budgets) return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  ta_bf16_view none = {};
  return compress_impl(ctx, pats, policy, batch, Hkv, Hkv, d, K_max, token_ids, none, k, v, 0, k_out, v_out, idx, count,
                       stream, score, score2, false, budgets);
}

ta_status ta_compress_budgets(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                              int Hq, int Hkv, int d, int K_max, const int32_t* budgets, const int32_t* token_ids,
                              ta_bf16_view q_obs, ta_bf16_view k, ta_bf16_view v, void* k_out, void* v_out,
                              int32_t* idx, int32_t* count, void* stream) {
  if (!policy || !budgets) return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED) return TA_ERR_INVALID_ARG;
  return compress_impl(ctx, pats, policy, batch, Hq, Hkv, d, K_max, token_ids, q_obs, k, v, 0, k_out, v_out, idx, count,
                       stream, nullptr, nullptr, false, budgets);
}

// ---------------------------------------------------------------------------------------------- decode loop
namespace {
struct StreamLayout {
  size_t info, end;
};
StreamLayout stream_layout(const ta_stream& st) {
  StreamLayout L;
  L.info = 0;
  L.end = align_up((size_t)st.batch * sizeof(ta_stream_seq_info));
  return L;
}
ta_status check_stream(const ta_stream* st) {
  if (!st) return TA_ERR_INVALID_ARG;
  if (st->n_layers < 1 || st->batch < 1 || st->Hkv < 1 || st->K < 1) return TA_ERR_INVALID_ARG;
  if (st->K > TA_MAX_BUDGET) return TA_ERR_UNSUPPORTED;
  if (st->cache_len < 0 || st->cache_len > st->K) return TA_ERR_INVALID_ARG;
  if ((long long)st->n_layers * st->batch * st->Hkv * ((long long)st->K + 1) > 0x7fffffffLL) return TA_ERR_UNSUPPORTED;
  if (!st->pos || !st->slot || !st->tok || !st->A || !st->P || !st->V || !st->S || !st->next_slot || !st->n_seen ||
      !st->hist || !st->tok_ring || !st->anc_B || !st->anc_L)
    return TA_ERR_INVALID_ARG;
  return TA_OK;
}
}  // namespace

ta_status ta_stream_scratch_bytes(const ta_stream* st, size_t* out_bytes) {
  if (!out_bytes || !st) return TA_ERR_INVALID_ARG;
  if (st->n_layers < 1 || st->batch < 1 || st->Hkv < 1 || st->K < 1) return TA_ERR_INVALID_ARG;
  *out_bytes = stream_layout(*st).end + kAlign;
  return TA_OK;
}

ta_status ta_stream_step(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, ta_stream* st,
                         const int32_t* new_ids, const float* attn, int32_t* evicted_pos, void* stream_v) {
  Range range("ta_stream_step");
  if (!ctx || !pats || !new_ids || !attn || !evicted_pos) return TA_ERR_INVALID_ARG;
  ta_status s = check_policy(policy);
  if (s == TA_OK) s = check_stream(st);
  if (s != TA_OK) return s;
  if (pats->device != ctx->device) return TA_ERR_INVALID_ARG;
  const StreamLayout L = stream_layout(*st);
  if (L.end > ctx->scratch_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  ctx->cached_epoch = 0;  // the scratch is shared with ta_compress's per-sequence cache
  cudaStream_t stream = (cudaStream_t)stream_v;
  uint8_t* sc = ctx->scratch;
  ta_stream_dev d = {};
  d.n_layers = st->n_layers;
  d.B = st->batch;
  d.Hkv = st->Hkv;
  d.K = st->K;
  d.len = st->cache_len;
  d.pos = st->pos;
  d.slot = st->slot;
  d.tok = st->tok;
  d.next_slot = st->next_slot;
  d.A = st->A;
  d.P = st->P;
  d.V = st->V;
  d.S = st->S;
  d.n_seen = st->n_seen;
  d.hist = st->hist;
  d.tok_ring = st->tok_ring;
  d.anc_B = st->anc_B;
  d.anc_L = st->anc_L;
  auto* info = reinterpret_cast<ta_stream_seq_info*>(sc + L.info);
  const bool evict = st->cache_len + 1 > st->K;

  cudaError_t e = ta_launch_stream_seq(d, pats, *policy, new_ids, info, ctx->d_status, stream);
  if (e == cudaSuccess) e = ta_launch_stream_step(d, *policy, info, attn, evicted_pos, ctx->d_status, stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  st->cache_len = evict ? st->K : st->cache_len + 1;
  return TA_OK;
}

// ---------------------------------------------------------------------------------------------- host buffers
namespace {
struct HostLayout {
  size_t ids, cu, q, k, v, k_out, v_out, idx, count, end;
  size_t q_bytes, kv_bytes, out_bytes, idx_bytes, count_bytes;
};
HostLayout host_layout(const ta_batch& b, int Hq, int Hkv, int d, int K, const ta_policy& pol) {
  HostLayout H;
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t o = off;
    off += align_up(bytes);
    return o;
  };
  const size_t L = (size_t)b.n_layers, B = (size_t)b.batch, total = (size_t)b.total_tokens;
  H.q_bytes = pol.mode == TA_MODE_FAST ? 0 : L * B * Hq * (size_t)pol.obs_window * d * 2;
  H.kv_bytes = L * Hkv * total * d * 2;
  H.out_bytes = L * B * Hkv * (size_t)K * d * 2;
  H.idx_bytes = L * B * Hkv * (size_t)K * 4;
  H.count_bytes = L * B * Hkv * 4;
  H.ids = take(total * 4);
  H.cu = take((B + 1) * 4);
  H.q = take(H.q_bytes);
  H.k = take(H.kv_bytes);
  H.v = take(H.kv_bytes);
  H.k_out = take(H.out_bytes);
  H.v_out = take(H.out_bytes);
  H.idx = take(H.idx_bytes);
  H.count = take(H.count_bytes);
  H.end = off;
  return H;
}
}  // namespace

ta_status ta_compress_host_workspace_bytes(const ta_batch* batch, int Hq, int Hkv, int d, int K,
                                           const ta_policy* policy, size_t* out_bytes) {
  if (!out_bytes) return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  if (K < 1 || Hkv < 1 || Hq < 1 || d < 1) return TA_ERR_INVALID_ARG;
  *out_bytes = host_layout(*batch, Hq, Hkv, d, K, *policy).end + kAlign;
  return TA_OK;
}

ta_status ta_compress_host(ta_ctx* ctx, const ta_patterns* pats, const ta_policy* policy, const ta_batch* batch,
                           int Hq, int Hkv, int d, int K, const int32_t* token_ids, const void* q_obs, const void* k,
                           const void* v, void* k_out, void* v_out, int32_t* idx, int32_t* count, void* workspace,
                           size_t workspace_bytes, void* stream_v) {
  Range range("ta_compress_host");
  if (!ctx || !pats || !token_ids || !k || !v || !k_out || !v_out || !idx || !count || !workspace)
    return TA_ERR_INVALID_ARG;
  ta_status s = check_batch(batch);
  if (s == TA_OK) s = check_policy(policy);
  if (s != TA_OK) return s;
  const bool fast = policy->mode == TA_MODE_FAST;
  if (!fast && !q_obs) return TA_ERR_INVALID_ARG;
  if (K < 1 || Hkv < 1 || Hq < Hkv) return TA_ERR_INVALID_ARG;
  if (d != TA_HEAD_DIM) return TA_ERR_UNSUPPORTED;
  if ((uintptr_t)workspace % kAlign) return TA_ERR_ALIGNMENT;
  const HostLayout H = host_layout(*batch, Hq, Hkv, d, K, *policy);
  if (H.end > workspace_bytes) return TA_ERR_SCRATCH_TOO_SMALL;
  DeviceGuard guard(ctx->device);
  cudaStream_t stream = (cudaStream_t)stream_v;
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  const size_t total = (size_t)batch->total_tokens;
  cudaError_t e = cudaMemcpyAsync(ws + H.ids, token_ids, total * 4, cudaMemcpyHostToDevice, stream);
  ta_batch db = *batch;
  if (batch->cu_seqlens) {
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(ws + H.cu, batch->cu_seqlens, ((size_t)batch->batch + 1) * 4, cudaMemcpyHostToDevice, stream);
    db.cu_seqlens = reinterpret_cast<const int32_t*>(ws + H.cu);
  }
  if (e == cudaSuccess && !fast) e = cudaMemcpyAsync(ws + H.q, q_obs, H.q_bytes, cudaMemcpyHostToDevice, stream);
  // Only the retained rows of V are ever read (and, in fast mode, of K): when such a cache sits in pinned or
  // registered host memory the gather kernel reads those rows straight over the bus and the full copy is skipped.
  auto device_visible_host = [&](const void* ptr, const void** dev_alias) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, ptr) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    if (at.type != cudaMemoryTypeHost || !at.devicePointer) return false;
    *dev_alias = at.devicePointer;
    return true;
  };
  const void* k_src = ws + H.k;
  const void* v_src = ws + H.v;
  const void* alias = nullptr;
  if (fast && device_visible_host(k, &alias)) k_src = alias;
  else if (e == cudaSuccess) e = cudaMemcpyAsync(ws + H.k, k, H.kv_bytes, cudaMemcpyHostToDevice, stream);
  if (device_visible_host(v, &alias)) v_src = alias;
  else if (e == cudaSuccess) e = cudaMemcpyAsync(ws + H.v, v, H.kv_bytes, cudaMemcpyHostToDevice, stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e);
  const int64_t n = batch->n_uniform, W = policy->obs_window;
  ta_bf16_view vq = {ws + H.q, (int64_t)batch->batch * Hq * W * d, (int64_t)Hq * W * d, W * d, d};
  ta_bf16_view vk, vv;
  if (batch->cu_seqlens) {
    vk = {k_src, (int64_t)Hkv * (int64_t)total * d, 0, (int64_t)total * d, d};
  } else {
    vk = {k_src, (int64_t)batch->batch * Hkv * n * d, (int64_t)Hkv * n * d, n * d, d};
  }
  vv = vk;
  vv.ptr = v_src;
  s = ta_compress(ctx, pats, policy, &db, Hq, Hkv, d, K, reinterpret_cast<const int32_t*>(ws + H.ids), vq, vk, vv, 0,
                  ws + H.k_out, ws + H.v_out, reinterpret_cast<int32_t*>(ws + H.idx),
                  reinterpret_cast<int32_t*>(ws + H.count), stream);
  if (s != TA_OK) return s;
  e = cudaMemcpyAsync(k_out, ws + H.k_out, H.out_bytes, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(v_out, ws + H.v_out, H.out_bytes, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(idx, ws + H.idx, H.idx_bytes, cudaMemcpyDeviceToHost, stream);
  if (e == cudaSuccess) e = cudaMemcpyAsync(count, ws + H.count, H.count_bytes, cudaMemcpyDeviceToHost, stream);
  return e == cudaSuccess ? TA_OK : cuda_fail(ctx, e);
}

}  // extern "C"
