// Step 3 of the retention path: budget-K selection with the partition of Section 3.3 (Algorithm 1 step 8).
//
// The retained set is reported in ascending position order, so no sort of the winners is needed: a radix select
// over the order-preserving integer image of the values (8-bit digits, starting below the bits that all keys of the
// unit share) finds the threshold key and how many tokens that tie with it still fit, and one ordered
// stream-compaction pass writes the indices. Order is total and deterministic: larger value first, lower
// position first among equal values.
//
//   ta_forced_kernel   one block per sequence: mandatory sinks/recents and the protected pool (largest vouchers
//                      among sponsored tokens). Independent of layer and head, so it runs once per sequence; on
//                      request it also writes the sequence's static utilities (Eq. 3).
//   ta_select_kernel   one block per unit (layer, sequence, KV head) in scored mode, per sequence in fast mode:
//                      main pool by utility among the tokens not forced, then the ordered write of
//                      forced + chosen positions.
//   ta_broadcast_idx_kernel  fast mode: the per-sequence result is the same for all layers and heads.
//   ta_headsum_kernel, ta_broadcast_heads_kernel  selection shared by the KV heads of a layer: the utilities'
//                      attention parts are summed over the heads, one selection runs per (layer, sequence), and its
//                      result is copied to every head.
#include <cooperative_groups.h>

#include "ta_internal.cuh"

namespace cg = cooperative_groups;

#define TA_SEL_THREADS 512
#define TA_SEL_NS sel512
#include "ta_select_core.cuh"
#undef TA_SEL_THREADS
#undef TA_SEL_NS
#define TA_SEL_THREADS 1024
#define TA_SEL_NS sel1024
#include "ta_select_core.cuh"
#undef TA_SEL_THREADS
#undef TA_SEL_NS

namespace {

using namespace sel512;  // the launchers below name the 512-thread kernels unless they say otherwise

__global__ void ta_broadcast_idx_kernel(int B, int Hkv, int K, int n_layers, const int32_t* __restrict__ idx_seq,
                                        const int32_t* __restrict__ count_seq, int32_t* __restrict__ idx,
                                        int32_t* __restrict__ count) {
  ta_wait_for_prior_grid();
  const long long total = (long long)n_layers * B * Hkv * K;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(t % K);
    const long long unit = t / K;
    const int b = (int)((unit / Hkv) % B);
    idx[t] = idx_seq[(long long)b * K + r];
    if (r == 0) count[unit] = count_seq[b];
  }
}

// u_all[l][tok] = sum over KV heads g (ascending, fp32) of u[l][g][tok]
__global__ void ta_headsum_kernel(int n_layers, int Hkv, long long total, const float* __restrict__ u,
                                  float* __restrict__ u_all) {
  const long long n = (long long)n_layers * total;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < n; t += (long long)gridDim.x * blockDim.x) {
    const long long l = t / total, tok = t - l * total;
    const float* src = u + l * Hkv * total + tok;
    float acc = src[0];
    for (int g = 1; g < Hkv; ++g) acc = __fadd_rn(acc, src[(long long)g * total]);
    u_all[t] = acc;
  }
}

// idx[l][b][g][:] = idx_lb[l][b][:], count[l][b][g] = count_lb[l][b]
__global__ void ta_broadcast_heads_kernel(long long units_lb, int Hkv, int K, const int32_t* __restrict__ idx_lb,
                                          const int32_t* __restrict__ count_lb, int32_t* __restrict__ idx,
                                          int32_t* __restrict__ count) {
  const long long total = units_lb * Hkv * K;
  for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total;
       t += (long long)gridDim.x * blockDim.x) {
    const int r = (int)(t % K);
    const long long unit = t / K, lb = unit / Hkv;
    idx[t] = idx_lb[lb * K + r];
    if (r == 0) count[unit] = count_lb[lb];
  }
}

}  // namespace

// Scratch layout used by the launcher (the caller carves it): forced [total] bytes, r_main [B] ints; fast mode
// additionally idx_seq [B][K] and count_seq [B] (passed through a.idx / a.count by the caller when it wants the
// per-sequence result only).
// Sequences that fit kItems keys per thread run one CTA per unit with the keys in registers; longer ones are split
// over a cluster of kSelectCluster CTAs (keys in registers up to kSelectCluster * 32 * 1024 elements; beyond 65536
// elements the cluster's blocks have 1024 threads).
// Splitting pays only while the clusters of all units fit on the device about at once; with many units one CTA per
// unit (keys re-read in batches when they do not fit in registers) keeps every SM busy without cluster barriers.
bool split_units(int units, int max_n, int sms) {
  if (max_n <= kItems * kThreads) return false;
  return units * kSelectCluster <= 2 * sms;
}

// SM count of the device the launch goes to: the caller's (a context knows its device), else the current device's
int sm_count_of(const ta_select_args& a) {
  if (a.sm_count > 0) return a.sm_count;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    sms = 148;
  return sms;
}

// stream_pdl: the stream, and whether the kernel is launched as a programmatic dependent of the kernel before it
struct StreamPdl {
  cudaStream_t stream;
  bool pdl;
};
template <class Kern, class... Args>
cudaError_t launch_threads(int threads, Kern kern, int units, int cl, StreamPdl sp, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(units * cl), 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = sp.stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cl > 1) {  // no cluster attribute when no cluster is needed
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cl;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (sp.pdl) ta_pdl_attribute(&attr[n++]);
  cfg.attrs = attr;
  cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}
template <class Kern, class... Args>
cudaError_t launch_clustered(Kern kern, int units, int cl, StreamPdl sp, Args... args) {
  return launch_threads(kThreads, kern, units, cl, sp, args...);
}

cudaError_t ta_launch_forced(const ta_select_args& a, ta_dev_status* status, cudaStream_t stream_) {
  if (a.seq.batch == 0 || a.n_layers == 0) return cudaSuccess;
  const StreamPdl stream = {stream_, a.pdl_forced != 0};
  const int B = a.seq.batch * (a.n_classes > 0 ? a.n_classes : 1);  // blocks: (class, sequence)
  const int32_t* ck = a.n_classes > 0 ? a.class_K : nullptr;
  const int sms = sm_count_of(a);
  ta_static_out so = {};
  so.out = a.static_out;
  so.ids = a.static_ids;
  so.flags = a.flags;
  so.hist = a.static_hist;
  so.vocab = a.static_vocab;
  so.beta = a.beta;
  so.gamma = a.gamma;
  so.lambda = a.lambda;
  if (a.seq.max_n <= kItems * kThreads)
    return launch_clustered(ta_forced_kernel<true, 1>, B, 1, stream, a.seq, a.K, a.n_sink, a.n_recent, a.k_protected,
                            a.voucher, a.forced, a.r_main, status, ck, so);
  if (!split_units(B, a.seq.max_n, sms) && a.seq.max_n <= kItemsLong * kThreads)
    return launch_clustered(ta_forced_kernel<true, 1, kItemsLong>, B, 1, stream, a.seq, a.K, a.n_sink, a.n_recent,
                            a.k_protected, a.voucher, a.forced, a.r_main, status, ck, so);
  if (!split_units(B, a.seq.max_n, sms))
    return launch_clustered(ta_forced_kernel<false, 1>, B, 1, stream, a.seq, a.K, a.n_sink, a.n_recent, a.k_protected,
                            a.voucher, a.forced, a.r_main, status, ck, so);
  if (a.seq.max_n <= kSelectCluster * kItems * kThreads)
    return launch_clustered(ta_forced_kernel<true, kSelectCluster>, B, kSelectCluster, stream, a.seq, a.K, a.n_sink,
                            a.n_recent, a.k_protected, a.voucher, a.forced, a.r_main, status, ck, so);
  // few very long sequences: the chain of per-thread sweeps and cluster barriers sets the time, so blocks of 1024
  // threads (half the keys per thread) roughly halve it
  if (a.seq.max_n <= kSelectCluster * sel1024::kItems * sel1024::kThreads)
    return launch_threads(sel1024::kThreads, sel1024::ta_forced_kernel<true, kSelectCluster>, B, kSelectCluster,
                          stream, a.seq, a.K, a.n_sink, a.n_recent, a.k_protected, a.voucher, a.forced, a.r_main,
                          status, ck, so);
  if (a.seq.max_n <= kSelectCluster * sel1024::kItemsLong * sel1024::kThreads)
    return launch_threads(sel1024::kThreads, sel1024::ta_forced_kernel<true, kSelectCluster, sel1024::kItemsLong>, B,
                          kSelectCluster, stream, a.seq, a.K, a.n_sink, a.n_recent, a.k_protected, a.voucher,
                          a.forced, a.r_main, status, ck, so);
  return launch_clustered(ta_forced_kernel<false, kSelectCluster>, B, kSelectCluster, stream, a.seq, a.K, a.n_sink,
                          a.n_recent, a.k_protected, a.voucher, a.forced, a.r_main, status, ck, so);
}

bool ta_select_gathers(const ta_select_args& a) {
  if (!a.gather_k_out || a.fast || a.K > kGatherMaxK) return false;
  // The gather adds one dependent load chain (index -> row -> store, about 2 us) to every block, the separate kernel
  // costs one launch (about 8 us for so few rows): fusing pays only while the blocks run in a few waves. Short units
  // (keys in 16 registers: two blocks per SM) only.
  const int units = a.n_layers * a.seq.batch * a.Hkv;
  return a.seq.max_n <= kItems * kThreads && units <= 4 * sm_count_of(a);
}

cudaError_t ta_launch_select_units(const ta_select_args& a, cudaStream_t stream_) {
  if (a.seq.batch == 0 || a.n_layers == 0) return cudaSuccess;
  const StreamPdl stream = {stream_, a.pdl_units != 0};
  UnitSrc src;
  src.u = a.fast ? nullptr : a.u;
  src.A = a.fast ? nullptr : a.A;
  src.P = a.fast ? nullptr : a.P;
  src.u_static = a.u_static;
  src.alpha = a.alpha;
  src.delta = a.delta;
  const int units = a.fast ? a.seq.batch : a.n_layers * a.seq.batch * a.Hkv;
  const int32_t* co = a.n_classes > 0 ? a.class_of : nullptr;
  const int sms = sm_count_of(a);
  GatherDst gd = {};
  if (ta_select_gathers(a)) {  // implies the first variant below
    gd.k = a.gather_k;
    gd.v = a.gather_v;
    gd.k_out = reinterpret_cast<uint4*>(a.gather_k_out);
    gd.v_out = reinterpret_cast<uint4*>(a.gather_v_out);
    return launch_clustered(ta_select_kernel<true, 1, kItems, true>, units, 1, stream, a.seq, a.n_layers, a.Hkv, a.K,
                            a.fast, src, a.forced, a.r_main, a.idx, a.count, gd, co);
  }
  if (a.seq.max_n <= kItems * kThreads)
    return launch_clustered(ta_select_kernel<true, 1>, units, 1, stream, a.seq, a.n_layers, a.Hkv, a.K, a.fast, src,
                            a.forced, a.r_main, a.idx, a.count, gd, co);
  if (!split_units(units, a.seq.max_n, sms) && a.seq.max_n <= kItemsLong * kThreads)
    return launch_clustered(ta_select_kernel<true, 1, kItemsLong>, units, 1, stream, a.seq, a.n_layers, a.Hkv, a.K, a.fast,
                            src, a.forced, a.r_main, a.idx, a.count, gd, co);
  sel1024::UnitSrc src2;  // the same fields for the kernels built for 1024 threads
  src2.u = src.u;
  src2.A = src.A;
  src2.P = src.P;
  src2.u_static = src.u_static;
  src2.alpha = src.alpha;
  src2.delta = src.delta;
  sel1024::GatherDst gd2 = {};
  if (!split_units(units, a.seq.max_n, sms) && a.seq.max_n <= sel1024::kItemsLong * sel1024::kThreads) {
    // many long units: blocks of 1024 threads hold a unit of up to 32768 keys in registers (read once instead of
    // once per radix pass and once more for the ordered write)
    return launch_threads(sel1024::kThreads, sel1024::ta_select_kernel<true, 1, sel1024::kItemsLong>, units, 1, stream,
                          a.seq, a.n_layers, a.Hkv, a.K, a.fast, src2, a.forced, a.r_main, a.idx, a.count, gd2, co);
  }
  if (!split_units(units, a.seq.max_n, sms))
    return launch_clustered(ta_select_kernel<false, 1>, units, 1, stream, a.seq, a.n_layers, a.Hkv, a.K, a.fast, src,
                            a.forced, a.r_main, a.idx, a.count, gd, co);
  if (a.seq.max_n <= kSelectCluster * kItems * kThreads)
    return launch_clustered(ta_select_kernel<true, kSelectCluster>, units, kSelectCluster, stream, a.seq, a.n_layers,
                            a.Hkv, a.K, a.fast, src, a.forced, a.r_main, a.idx, a.count, gd, co);
  if (a.seq.max_n <= kSelectCluster * sel1024::kItems * sel1024::kThreads)  // as in ta_launch_forced
    return launch_threads(sel1024::kThreads, sel1024::ta_select_kernel<true, kSelectCluster>, units, kSelectCluster,
                          stream, a.seq, a.n_layers, a.Hkv, a.K, a.fast, src2, a.forced, a.r_main, a.idx, a.count, gd2,
                          co);
  if (a.seq.max_n <= kSelectCluster * sel1024::kItemsLong * sel1024::kThreads)
    return launch_threads(sel1024::kThreads, sel1024::ta_select_kernel<true, kSelectCluster, sel1024::kItemsLong>,
                          units, kSelectCluster, stream, a.seq, a.n_layers, a.Hkv, a.K, a.fast, src2, a.forced,
                          a.r_main, a.idx, a.count, gd2, co);
  return launch_clustered(ta_select_kernel<false, kSelectCluster>, units, kSelectCluster, stream, a.seq, a.n_layers,
                          a.Hkv, a.K, a.fast, src, a.forced, a.r_main, a.idx, a.count, gd, co);
}

cudaError_t ta_launch_select(const ta_select_args& a, ta_dev_status* status, cudaStream_t stream) {
  cudaError_t e = ta_launch_forced(a, status, stream);
  if (e != cudaSuccess) return e;
  return ta_launch_select_units(a, stream);
}

cudaError_t ta_launch_broadcast_idx(int B, int Hkv, int K, int n_layers, const int32_t* idx_seq,
                                    const int32_t* count_seq, int32_t* idx, int32_t* count, cudaStream_t stream,
                                    bool pdl) {
  const long long total = (long long)n_layers * B * Hkv * K;
  if (total == 0) return cudaSuccess;
  const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (pdl) ta_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, ta_broadcast_idx_kernel, B, Hkv, K, n_layers, idx_seq, count_seq, idx, count);
}

cudaError_t ta_launch_headsum(int n_layers, int Hkv, long long total, const float* u, float* u_all,
                              cudaStream_t stream) {
  const long long n = (long long)n_layers * total;
  if (n == 0) return cudaSuccess;
  const int blocks = (int)((n + 255) / 256 < 8192 ? (n + 255) / 256 : 8192);
  ta_headsum_kernel<<<blocks, 256, 0, stream>>>(n_layers, Hkv, total, u, u_all);
  return cudaGetLastError();
}

cudaError_t ta_launch_broadcast_heads(int n_layers, int B, int Hkv, int K, const int32_t* idx_lb,
                                      const int32_t* count_lb, int32_t* idx, int32_t* count, cudaStream_t stream) {
  const long long total = (long long)n_layers * B * Hkv * K;
  if (total == 0) return cudaSuccess;
  const int blocks = (int)((total + 255) / 256 < 4096 ? (total + 255) / 256 : 4096);
  ta_broadcast_heads_kernel<<<blocks, 256, 0, stream>>>((long long)n_layers * B, Hkv, K, idx_lb, count_lb, idx, count);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------------------------
// ta_select_topk_static: the selection step for callers that must not allocate device memory.
//
// The regular entry point takes its working memory (one byte per token, a few words per sequence) from a context
// whose creation calls cudaMalloc. This variant keeps that working memory in the array below, which is part of the
// library image: every GPU that loads the library reserves TA_STATIC_SCRATCH_BYTES for it until the process exits.
// The array name is only meaningful to device code; host code must ask the runtime for its device address
// (cudaGetSymbolAddress) once per device, with that device current, and hand that address to the kernels.
#include <mutex>

static __device__ __align__(256) unsigned char g_ta_static_scratch[TA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};  // device address of g_ta_static_scratch, per device ordinal

size_t static_align(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

extern "C" ta_status ta_select_topk_static(const ta_policy* policy, const ta_batch* batch, int Hkv, int K,
                                           const uint8_t* flags, const float* voucher, const float* u_static,
                                           const float* A, const float* P, int32_t* idx, int32_t* count,
                                           void* stream_v) {
  if (!policy || !batch || !flags || !voucher || !u_static || !idx || !count) return TA_ERR_INVALID_ARG;
  if (batch->n_layers < 1 || batch->batch < 1 || batch->max_n < 0 || batch->total_tokens < 0 || Hkv < 1 || K < 1)
    return TA_ERR_INVALID_ARG;
  if (!batch->cu_seqlens && (batch->n_uniform < 0 || batch->n_uniform > batch->max_n ||
                             batch->total_tokens != (int64_t)batch->batch * batch->n_uniform))
    return TA_ERR_INVALID_ARG;
  if (policy->mode != TA_MODE_SCORED && policy->mode != TA_MODE_FAST) return TA_ERR_INVALID_ARG;
  if (policy->n_sink < 0 || policy->n_recent < 0) return TA_ERR_INVALID_ARG;
  if (K > TA_MAX_BUDGET || batch->max_n > TA_MAX_SEQ_LEN) return TA_ERR_UNSUPPORTED;
  const bool fast = policy->mode == TA_MODE_FAST;
  if (!fast && !A) return TA_ERR_INVALID_ARG;

  // carve the fixed array: status block, forced flags, per-sequence counters, fast-mode per-sequence result
  const size_t B = (size_t)batch->batch, total = (size_t)batch->total_tokens;
  size_t off = 0;
  const size_t o_status = off; off += static_align(sizeof(ta_dev_status));
  const size_t o_forced = off; off += static_align(total);
  const size_t o_rmain = off;  off += static_align(B * 4);
  const size_t o_idxseq = off; off += static_align(fast ? B * (size_t)K * 4 : 0);
  const size_t o_cntseq = off; off += static_align(fast ? B * 4 : 0);
  if (off > (size_t)TA_STATIC_SCRATCH_BYTES) return TA_ERR_SCRATCH_TOO_SMALL;  // problem larger than the built-in limit

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TA_ERR_CUDA;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {  // first call on this device: resolve the array's device address (no allocation)
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_ta_static_scratch) != cudaSuccess || !p) return TA_ERR_CUDA;
      g_static_ptr[dev] = static_cast<unsigned char*>(p);
    }
    base = g_static_ptr[dev];
  }
  cudaStream_t stream = (cudaStream_t)stream_v;
  // the array keeps whatever the previous call left: the status block must start at zero; the other pieces are
  // fully rewritten by the kernels before they are read
  if (cudaMemsetAsync(base + o_status, 0, sizeof(ta_dev_status), stream) != cudaSuccess) return TA_ERR_CUDA;

  ta_select_args a = {};
  a.seq.cu = batch->cu_seqlens;
  a.seq.n_uniform = batch->n_uniform;
  a.seq.batch = batch->batch;
  a.seq.max_n = batch->max_n;
  a.seq.total = batch->total_tokens;
  a.n_layers = batch->n_layers;
  a.Hkv = Hkv;
  a.K = K;
  a.n_sink = policy->n_sink;
  a.n_recent = policy->n_recent;
  a.k_protected = policy->k_protected;
  a.fast = fast;
  a.alpha = policy->alpha;
  a.delta = policy->delta;
  a.flags = flags;
  a.voucher = voucher;
  a.u_static = u_static;
  a.A = A;
  a.P = P;
  a.u = nullptr;
  a.forced = base + o_forced;
  a.r_main = reinterpret_cast<int32_t*>(base + o_rmain);
  int32_t* idx_seq = reinterpret_cast<int32_t*>(base + o_idxseq);
  int32_t* cnt_seq = reinterpret_cast<int32_t*>(base + o_cntseq);
  a.idx = fast ? idx_seq : idx;
  a.count = fast ? cnt_seq : count;
  cudaError_t e = ta_launch_select(a, reinterpret_cast<ta_dev_status*>(base + o_status), stream);
  if (e == cudaSuccess && fast)
    e = ta_launch_broadcast_idx(batch->batch, Hkv, K, batch->n_layers, idx_seq, cnt_seq, idx, count, stream);
  return e == cudaSuccess ? TA_OK : TA_ERR_CUDA;
}
