// Internal declarations shared by the translation units of libta.so (host orchestration <-> kernel launchers).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ta.h"

// Device status block: word 0 = first error code (ta_status), word 1..3 = detail (where, what).
struct ta_dev_status {
  int code;
  int where;
  int detail0;
  int detail1;
};

struct ta_patterns {
  int device;
  int n_pat;
  int max_len;
  int max_span;
  // device tables
  int32_t* d_ids;     // [n_pat][TA_MAX_PATTERN_LEN], right-aligned is NOT used: ids[p][0..len)
  int32_t* d_len;     // [n_pat]
  float* d_budget;    // [n_pat]
  int32_t* d_span;    // [n_pat]
  uint32_t* d_bloom;  // [32] 1024-bit filter over the last id of every pattern
};

struct ta_ctx {
  int device;
  int sm_count;
  int last_cuda_error;
  size_t scratch_bytes;
  uint8_t* scratch;         // device
  ta_dev_status* d_status;  // device
  // cache of per-sequence results inside scratch (ta_compress)
  uint64_t cached_epoch;
  uint64_t cached_key;  // policy fields and pattern set the cached results were computed with
  int64_t cached_total;
  int cached_batch;
  int cached_K;
  // per-kernel timing of ta_compress
  int timing_enabled;
  int timing_valid;
  cudaEvent_t ev[8];
  int ev_ran[4];
  // fork/join of the per-sequence work (mask, vouchers, forced set) beside the score kernel
  cudaStream_t side;
  cudaEvent_t ev_fork, ev_join;
  // launch shape of the most recent score kernel (diagnostics)
  int score_cluster, score_clusters;
  // score kernel launch state per instantiation (2 row-block counts x 3 output forms): attribute set, resident
  // clusters per cluster size (0: not queried yet, -1: does not fit)
  int score_attr_set[6];
  int score_max_clusters[6][9];
  int last_select_gathered;           // the most recent ta_compress let the selection kernel gather the rows
  int last_kernel_launches;           // kernels enqueued by the most recent ta_compress
  int score_force_cluster;            // > 0: CTAs per unit fixed by ta_ctx_set_option (tuning, tests)
  unsigned long long wait_limit_ns;   // 0: default limit of device-side waits
  // driver entry point for tensor-map encoding (resolved at create time)
  void* encode_tiled;
};

// Sizes are validated by the callers in ta_api.cu; launchers return cudaError_t from the launch.

struct ta_seq_desc {  // how a kernel finds sequence b
  const int32_t* cu;  // device, or nullptr
  int n_uniform;
  int batch;
  int max_n;
  long long total;
};

__host__ __device__ inline int ta_seq_begin(const ta_seq_desc& s, int b, const int32_t* cu_cached = nullptr) {
  return s.cu ? s.cu[b] : b * s.n_uniform;
}

// Programmatic dependent launch: a kernel launched with ta_pdl_attribute() may be scheduled while the kernel before it
// on the stream is still draining (its launch latency overlaps that kernel's tail); it must call
// ta_wait_for_prior_grid() before its first access to memory. The call returns at once in a kernel launched normally.
inline void ta_pdl_attribute(cudaLaunchAttribute* attr) {
  attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr->val.programmaticStreamSerializationAllowed = 1;
}
#ifdef __CUDACC__
__device__ __forceinline__ void ta_wait_for_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Static part of a token's utility (Eq. 3): u_static = ((beta*R + gamma*S) - lambda*F) + V with R = (i0+1)/n,
// S = 1 on anchor tokens, F = count(id)/n; one rounding per operation. i0 is the 0-based position in the sequence.
__device__ __forceinline__ float ta_static_utility(int i0, int n, int count, bool anchor_token, float V, float beta,
                                                   float gamma, float lambda) {
  const float R = __fdiv_rn((float)(i0 + 1), (float)n);
  const float S = anchor_token ? 1.0f : 0.0f;
  const float F = __fdiv_rn((float)count, (float)n);
  const float t0 = __fadd_rn(__fmul_rn(beta, R), __fmul_rn(gamma, S));
  const float t1 = __fsub_rn(t0, __fmul_rn(lambda, F));
  return __fadd_rn(t1, V);
}
#endif

// ---- step 1 ------------------------------------------------------------------------------------------------
// u_static may be null: the caller then has ta_launch_forced compute it (ta_select_args::static_out).
cudaError_t ta_launch_mask(const ta_patterns* pats, const ta_policy& pol, const ta_seq_desc& seq, const int32_t* ids,
                           uint8_t* flags, float* voucher, float* u_static, int32_t* hist /*[B][vocab]*/,
                           ta_dev_status* status, cudaStream_t stream);

// the same with anchors from a detector's per-token confidences (single-token anchors, one span for all)
cudaError_t ta_launch_mask_conf(const ta_policy& pol, const ta_seq_desc& seq, const int32_t* ids, const float* conf,
                                float threshold, float budget, int span, int rank, uint8_t* flags, float* voucher,
                                float* u_static, int32_t* hist, ta_dev_status* status, cudaStream_t stream);

// embedding-based detector: conf[i] = max over concepts of the cosine similarity (ta_detect.cu)
cudaError_t ta_launch_embed_conf(int sm_count, long long total, const void* emb, long long stride, int D,
                                 const void* concepts, int C, float* conf, cudaStream_t stream);

// ---- step 2 ------------------------------------------------------------------------------------------------
struct ta_score_args {
  ta_seq_desc seq;
  int n_layers, Hq, Hkv, W;
  ta_bf16_view q, k;
  const float* lse_obs;  // nullable
  float* A;              // nullable
  float* P;              // nullable
  float* u;              // nullable: fused attention part alpha*A + delta*P (u_static is added by the selection)
  float alpha, delta, rho, scale;
  int causal;
  int reserve_sms;       // SMs left free for kernels running beside the (persistent) score kernel
  int32_t* order_scratch; // nullable: n_layers*batch*Hkv ints; ragged batches then run longest sequences first
};
cudaError_t ta_launch_score(ta_ctx* ctx, const ta_score_args& a, ta_dev_status* status, cudaStream_t stream);

// diagnostic: one warp runs into the limit of a bounded wait (TA_ERR_TIMEOUT in `status`); *outcome gets bit 2 set when
// the kernel ran to its end, bits 0/1 when a wait unexpectedly succeeded
cudaError_t ta_launch_wait_selftest(ta_dev_status* status, unsigned long long limit_ns, int* outcome,
                                    cudaStream_t stream);

// ---- step 3 ------------------------------------------------------------------------------------------------
struct ta_static_out {  // what ta_forced_kernel needs to write the static utilities of its sequence (out null: off)
  float* out;
  const int32_t* ids;
  const uint8_t* flags;
  const int32_t* hist;
  int vocab;
  float beta, gamma, lambda;
};

struct ta_select_args {
  ta_seq_desc seq;
  int n_layers, Hkv, K;
  int n_sink, n_recent, k_protected;
  int fast;
  int sm_count;  // of the device the launch goes to (0: ask the runtime about the current device)
  float alpha, delta;
  const uint8_t* flags;
  const float* voucher;
  const float* u_static;
  const float* A;  // scored, unfused
  const float* P;
  const float* u;  // scored, fused: alpha*A + delta*P as written by the score kernel (takes precedence over A/P)
  uint8_t* forced;     // scratch [total]
  int32_t* r_main;     // scratch [B]   main-pool picks per sequence (-1: keep everything)
  int32_t* idx;        // [L][B][Hkv][K]
  int32_t* count;      // [L][B][Hkv]
  // optional: budgets that differ between (layer, KV head) pairs. Pairs with the same budget form a class; the forced
  // set is computed once per (class, sequence): forced [n_classes][total], r_main [n_classes][B]. K is then the
  // largest budget (the stride of idx).
  int n_classes;            // 0: one budget K for all units
  const int32_t* class_K;   // DEVICE [n_classes]
  const int32_t* class_of;  // DEVICE [n_layers][Hkv]
  // optional: the select kernel also gathers the retained rows (small K, one block per unit; see ta_select_gathers)
  ta_bf16_view gather_k, gather_v;
  void* gather_k_out;  // null: no gather
  void* gather_v_out;
  // optional: ta_launch_forced also writes the static utilities (what ta_launch_mask does when it is given the
  // array), saving a kernel on the per-sequence chain. static_out null: not asked for.
  int pdl_forced, pdl_units;  // launch the forced-set / the selection kernel as a programmatic dependent of the kernel before it
  float* static_out;
  const int32_t* static_ids;
  const int32_t* static_hist;  // [B][vocab] token counts per sequence
  int static_vocab;
  float beta, gamma, lambda;
};
bool ta_select_gathers(const ta_select_args& a);  // whether ta_launch_select_units will do the gather itself
cudaError_t ta_launch_select(const ta_select_args& a, ta_dev_status* status, cudaStream_t stream);  // both below
cudaError_t ta_launch_forced(const ta_select_args& a, ta_dev_status* status, cudaStream_t stream);
cudaError_t ta_launch_select_units(const ta_select_args& a, cudaStream_t stream);
cudaError_t ta_launch_broadcast_idx(int B, int Hkv, int K, int n_layers, const int32_t* idx_seq,
                                    const int32_t* count_seq, int32_t* idx, int32_t* count, cudaStream_t stream,
                                    bool pdl = false);

// selection shared by the KV heads of a layer: head sum of the utilities, copy of the result to every head
cudaError_t ta_launch_headsum(int n_layers, int Hkv, long long total, const float* u, float* u_all,
                              cudaStream_t stream);
cudaError_t ta_launch_broadcast_heads(int n_layers, int B, int Hkv, int K, const int32_t* idx_lb,
                                      const int32_t* count_lb, int32_t* idx, int32_t* count, cudaStream_t stream);

// ---- Algorithm 1 per decode step (ta_stream.cu) ---------------------------------------------------------------
struct ta_stream_dev {  // the caller's ta_stream with the cached length of this step
  int n_layers, B, Hkv, K, len;
  int32_t *pos, *slot, *tok, *next_slot;
  float *A, *P, *V;
  uint8_t* S;
  int32_t *n_seen, *hist, *tok_ring;
  float* anc_B;
  int32_t* anc_L;
};
struct ta_stream_seq_info {  // per sequence, written by the sequence kernel of a step
  int t;          // position of the new token
  int match_len;  // tokens t - match_len + 1 .. t belong to a pattern completed by the new token (0: none)
  float v_new;    // voucher of the new token
  int id;         // its token id
};
cudaError_t ta_launch_stream_seq(const ta_stream_dev& st, const ta_patterns* pats, const ta_policy& pol,
                                 const int32_t* new_ids, ta_stream_seq_info* info, ta_dev_status* status,
                                 cudaStream_t stream);
cudaError_t ta_launch_stream_step(const ta_stream_dev& st, const ta_policy& pol, const ta_stream_seq_info* info,
                                  const float* attn, int32_t* evicted_pos, ta_dev_status* status,
                                  cudaStream_t stream);

// ---- step 4 ------------------------------------------------------------------------------------------------
struct ta_compact_args {
  ta_seq_desc seq;
  int n_layers, Hkv, K;
  ta_bf16_view k, v;
  const int32_t* idx;
  const int32_t* count;
  void* k_out;
  void* v_out;
  int pdl;  // launch as a programmatic dependent of the kernel before it on the stream
};
cudaError_t ta_launch_compact(const ta_compact_args& a, int sm_count, cudaStream_t stream);
