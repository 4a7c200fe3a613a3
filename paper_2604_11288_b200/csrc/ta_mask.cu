// Step 1 of the retention path: anchor detection, voucher allocation and the attention-free utility
// (Section 3.2; Eq. 2; Eq. 3; Algorithm 1 steps 1-7 without the attention terms).
//
// Kernel ta_mask_kernel works on tiles of the packed token stream. A tile needs no data from other tiles beyond a
// halo of (max span + max pattern length) token ids to its left and (max pattern length) to its right, so the grid
// is embarrassingly parallel and HBM traffic is 4 B read + 5 B written per token.
//   phase a  token ids of tile + halo -> shared memory; per-sequence token histogram via global atomics
//   phase b  warp-parallel multi-pattern match: every lane tests one end position; a 1024-bit filter on the last
//            id of all patterns rejects almost every position before the pattern table is walked
//   phase c  span spread: a segmented (by sequence) inclusive max-scan of "anchor position + span" tells each
//            token whether any earlier anchor of its own sequence reaches it; only those tokens add up their
//            vouchers, nearest anchor first, in fp32 with one rounding per operation (bit-exact by construction)
// Kernel ta_ustatic_kernel then combines recency, anchor flag, frequency and voucher into u_static.
// With a detector's per-token confidences instead of a pattern set (Section 5.1) phase b is a threshold test: the
// anchors are single tokens, all with the same span, and their budget is fixed or proportional to the confidence.
#include "ta_internal.cuh"

namespace {

constexpr int kTile = 512;                                   // tokens per block == threads per block
constexpr int kHaloL = TA_MAX_SPAN + TA_MAX_PATTERN_LEN;     // left halo of token ids
constexpr int kHaloR = TA_MAX_PATTERN_LEN;                   // right halo
constexpr int kExt = kHaloL + kTile + kHaloR;                // ids held in shared memory
constexpr int kScan = 2 * kTile;                             // scan slots (2 per thread) >= TA_MAX_SPAN + kTile

__device__ __forceinline__ uint32_t bloom_hash(int32_t x) { return ((uint32_t)x * 2654435761u) >> 22; }

// sequence index of packed token `tok`
__device__ __forceinline__ int seq_of(const ta_seq_desc& s, long long tok) {
  if (!s.cu) return (int)(tok / s.n_uniform);
  int lo = 0, hi = s.batch;  // cu[lo] <= tok < cu[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (s.cu[mid] <= tok) lo = mid; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void report(ta_dev_status* st, int code, int where, int d0, int d1) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where;
    st->detail0 = d0;
    st->detail1 = d1;
  }
}

struct ConfAnchors {   // anchors from a detector's confidences; conf == nullptr: token-id patterns are matched
  const float* conf;   // [total]
  float threshold;     // anchor iff conf > threshold
  float budget;        // sponsor budget B (rank: B_i = budget * conf_i)
  int span;            // L
  int rank;
};

struct SegMax {  // element of the segmented max-scan: flag = a segment starts at or before this element
  int flag;
  int val;
};
__device__ __forceinline__ SegMax seg_combine(SegMax left, SegMax right) {
  SegMax r;
  r.flag = left.flag | right.flag;
  r.val = right.flag ? right.val : max(left.val, right.val);
  return r;
}

__global__ void __launch_bounds__(kTile) ta_mask_kernel(ta_seq_desc seq, const int32_t* __restrict__ ids,
                                                        const int32_t* __restrict__ p_ids,
                                                        const int32_t* __restrict__ p_len,
                                                        const float* __restrict__ p_budget,
                                                        const int32_t* __restrict__ p_span,
                                                        const uint32_t* __restrict__ p_bloom, int n_pat,
                                                        int max_len, int max_span, float voucher_decay,
                                                        float budget_decay, int age_steps, int vocab,
                                                        uint8_t* __restrict__ flags, float* __restrict__ voucher,
                                                        int32_t* __restrict__ hist, ta_dev_status* status,
                                                        ConfAnchors ca) {
  __shared__ int32_t s_id[kExt];
  __shared__ int32_t s_start[kExt];     // packed index of the first token of the position's sequence
  __shared__ int16_t s_apat[kExt];      // winning pattern ending here, -1 none
  __shared__ float s_abud[kExt];        // its decayed budget
  __shared__ int32_t s_pid[TA_MAX_PATTERNS * TA_MAX_PATTERN_LEN];
  __shared__ int32_t s_plen[TA_MAX_PATTERNS];
  __shared__ int32_t s_pspan[TA_MAX_PATTERNS];
  __shared__ float s_pbud[TA_MAX_PATTERNS];
  __shared__ uint32_t s_bloom[32];
  __shared__ float s_w[TA_MAX_SPAN + 1];
  __shared__ SegMax s_warp[kTile / 32];

  const int tid = threadIdx.x;
  const long long T0 = (long long)blockIdx.x * kTile;  // first packed token of the tile
  const long long ext0 = T0 - kHaloL;                  // packed token of s_id[0]

  if (ca.conf) {  // one pseudo-pattern of length 1 stands for "the detector fired here"
    if (tid == 0) {
      s_plen[0] = 1;
      s_pspan[0] = ca.span;
      s_pbud[0] = ca.budget;
    }
  } else {
    // the pattern tables: every load is requested before the first is stored (one memory latency for all of them)
    static_assert(TA_MAX_PATTERNS <= kTile && TA_MAX_PATTERNS * TA_MAX_PATTERN_LEN <= 4 * kTile, "slots per thread");
    int32_t r_pid[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = tid + q * kTile;
      r_pid[q] = i < n_pat * TA_MAX_PATTERN_LEN ? p_ids[i] : 0;
    }
    const int32_t r_len = tid < n_pat ? p_len[tid] : 0, r_span = tid < n_pat ? p_span[tid] : 0;
    const float r_bud = tid < n_pat ? p_budget[tid] : 0.0f;
    const uint32_t r_bloom = (tid < 32 && n_pat) ? p_bloom[tid] : 0u;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int i = tid + q * kTile;
      if (i < n_pat * TA_MAX_PATTERN_LEN) s_pid[i] = r_pid[q];
    }
    if (tid < n_pat) {
      s_plen[tid] = r_len;
      s_pspan[tid] = r_span;
      s_pbud[tid] = r_bud;
    }
    if (tid < 32) s_bloom[tid] = r_bloom;
  }
  if (tid <= TA_MAX_SPAN) {  // s_w[k] = decay^k by repeated multiplication (one rounding per step), thread k on its own
    float w = 1.0f;
    for (int k = 0; k < tid; ++k) w = __fmul_rn(w, voucher_decay);
    s_w[tid] = w;
  }

  // phase a: ids + sequence starts for tile and halo; histogram for the tile proper
  for (int i = tid; i < kExt; i += kTile) {
    const long long tok = ext0 + i;
    int32_t id = -1, start = 0;
    if (tok >= 0 && tok < seq.total) {
      id = ids[tok];
      const int b = seq_of(seq, tok);
      start = ta_seq_begin(seq, b);
      if (i >= kHaloL && i < kHaloL + kTile) {
        if (id >= 0 && id < vocab)
          atomicAdd(&hist[(long long)b * vocab + id], 1);
        else
          report(status, TA_ERR_DEVICE_BOUNDS, 1, (int)tok, id);
      }
    }
    s_id[i] = id;
    s_start[i] = start;
  }
  __syncthreads();

  // phase b: which pattern (longest, then lowest index) ends at each position of [T0 - max_span, T0 + kTile + max_len)
  for (int i = tid; i < kExt; i += kTile) {
    int best = -1, best_len = 0;
    const int32_t x = s_id[i];
    float cf = 0.0f;
    if (ca.conf) {
      const long long tok = ext0 + i;
      if (tok >= 0 && tok < seq.total) {
        cf = ca.conf[tok];
        if (cf > ca.threshold) best = 0;  // false for NaN
      }
    } else if (x >= 0 && i >= TA_MAX_PATTERN_LEN) {
      const uint32_t h = bloom_hash(x);
      if (s_bloom[h >> 5] & (1u << (h & 31))) {
        const long long tok = ext0 + i;
        const int avail = (int)min((long long)TA_MAX_PATTERN_LEN, tok - s_start[i] + 1);  // tokens of this sequence up to here
        for (int p = 0; p < n_pat; ++p) {
          const int len = s_plen[p];
          if (len <= best_len || len > avail) continue;
          const int32_t* pid = &s_pid[p * TA_MAX_PATTERN_LEN];
          if (pid[len - 1] != x) continue;
          bool ok = true;
          for (int k = 0; k < len - 1; ++k) ok = ok && (s_id[i - len + 1 + k] == pid[k]);
          if (ok) {
            best = p;
            best_len = len;
          }
        }
      }
    }
    s_apat[i] = (int16_t)best;
    float B = 0.0f;
    if (best >= 0) {
      B = s_pbud[best];
      if (ca.conf && ca.rank) B = __fmul_rn(B, cf);
      for (int t = 0; t < age_steps; ++t) B = __fmul_rn(B, budget_decay);
    }
    s_abud[i] = B;
  }
  __syncthreads();

  // phase c.1: segmented inclusive max-scan of reach = position + span over scan slots [0, kScan); slot q maps to
  // s_* index q + (kHaloL - TA_MAX_SPAN), i.e. the scan starts TA_MAX_SPAN tokens before the tile.
  constexpr int kScanBase = kHaloL - TA_MAX_SPAN;
  SegMax e0, e1;
  {
    const int q0 = 2 * tid, q1 = 2 * tid + 1;
    auto load = [&](int q) {
      SegMax e;
      e.flag = 0;
      e.val = -1;
      const int i = q + kScanBase;
      if (q < TA_MAX_SPAN + kTile) {
        const long long tok = ext0 + i;
        if (tok >= 0 && tok < seq.total) {
          e.flag = (tok == s_start[i]) ? 1 : 0;
          const int p = s_apat[i];
          if (p >= 0) e.val = i + s_pspan[p];  // reach in s_* coordinates
        }
      }
      return e;
    };
    e0 = load(q0);
    e1 = seg_combine(e0, load(q1));
  }
  SegMax run = e1;  // inclusive over this thread's pair
  const int lane = tid & 31, warp = tid >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    SegMax o;
    o.flag = __shfl_up_sync(0xffffffffu, run.flag, off);
    o.val = __shfl_up_sync(0xffffffffu, run.val, off);
    if (lane >= off) run = seg_combine(o, run);
  }
  if (lane == 31) s_warp[warp] = run;
  __syncthreads();
  if (warp == 0) {
    SegMax w;
    w.flag = 0;
    w.val = -1;
    if (lane < kTile / 32) w = s_warp[lane];
#pragma unroll
    for (int off = 1; off < kTile / 32; off <<= 1) {
      SegMax o;
      o.flag = __shfl_up_sync(0xffffffffu, w.flag, off);
      o.val = __shfl_up_sync(0xffffffffu, w.val, off);
      if (lane >= off) w = seg_combine(o, w);
    }
    if (lane < kTile / 32) s_warp[lane] = w;
  }
  __syncthreads();
  // exclusive prefix for this thread's pair = (carry of previous warps) + (inclusive of previous lane)
  SegMax prev;
  prev.flag = __shfl_up_sync(0xffffffffu, run.flag, 1);
  prev.val = __shfl_up_sync(0xffffffffu, run.val, 1);
  if (lane == 0) {
    prev.flag = 0;
    prev.val = -1;
  }
  if (warp > 0) prev = seg_combine(s_warp[warp - 1], prev);
  // inclusive values at the two slots of this thread -> shared (reuse s_start is not possible: still needed)
  __shared__ int32_t s_reach[kScan];
  {
    const SegMax i0 = seg_combine(prev, e0);
    SegMax second;  // recompute the second element alone
    second.flag = 0;
    second.val = -1;
    {
      const int q = 2 * tid + 1;
      const int i = q + kScanBase;
      if (q < TA_MAX_SPAN + kTile) {
        const long long tok = ext0 + i;
        if (tok >= 0 && tok < seq.total) {
          second.flag = (tok == s_start[i]) ? 1 : 0;
          const int p = s_apat[i];
          if (p >= 0) second.val = i + s_pspan[p];
        }
      }
    }
    const SegMax i1 = seg_combine(i0, second);
    s_reach[2 * tid] = i0.val;
    s_reach[2 * tid + 1] = i1.val;
  }
  __syncthreads();

  // phase c.2: flags and vouchers for the tile's own tokens
  {
    const int i = kHaloL + tid;  // s_* index
    const long long tok = T0 + tid;
    if (tok < seq.total) {
      const int32_t start = s_start[i];
      // S flag: a match ending at e in [tok, tok + max_len) that starts at or before tok
      int anchor_tok = 0;
      for (int k = 0; k < max_len; ++k) {
        const int p = s_apat[i + k];
        if (p >= 0 && s_plen[p] > k) anchor_tok = 1;
      }
      const int anchor_end = s_apat[i] >= 0;
      // is any earlier anchor of this sequence reaching this token? inclusive scan value of the previous slot,
      // unless this token starts its sequence
      float V = 0.0f;
      const int q = i - kScanBase;
      const bool head = (tok == start);
      const int reach = (head || q == 0) ? -1 : s_reach[q - 1];
      if (reach >= i) {
        // which of the kmax positions before this token hold an anchor whose span reaches it: independent loads,
        // collected in a bit mask; the sum then runs over the few set bits, nearest anchor first
        const int kmax = (int)min((long long)max_span, tok - start);
        static_assert(TA_MAX_SPAN <= 64, "one bit per distance");
        unsigned long long reaching = 0;
#pragma unroll 8
        for (int k = 1; k <= kmax; ++k) {
          const int p = s_apat[i - k];
          const int span = p >= 0 ? s_pspan[p] : 0;
          if (k <= span) reaching |= 1ull << (k - 1);
        }
        while (reaching) {
          const int k = __ffsll((long long)reaching);
          reaching &= reaching - 1ull;
          V = __fadd_rn(V, __fmul_rn(s_abud[i - k], s_w[k]));
        }
      }
      flags[tok] = (uint8_t)((anchor_tok ? TA_FLAG_ANCHOR_TOKEN : 0) | (anchor_end ? TA_FLAG_ANCHOR_END : 0) |
                             (V > 0.0f ? TA_FLAG_SPONSORED : 0));
      voucher[tok] = V;
    }
  }
}

// u_static = ((beta*R + gamma*S) - lambda*F) + V, R = (i0+1)/n, F = count(id)/n  (Eq. 3), one rounding per operation.
__global__ void __launch_bounds__(256) ta_ustatic_kernel(ta_seq_desc seq, const int32_t* __restrict__ ids,
                                                         const uint8_t* __restrict__ flags,
                                                         const float* __restrict__ voucher,
                                                         const int32_t* __restrict__ hist, int vocab, float beta,
                                                         float gamma, float lambda, float* __restrict__ u_static) {
  ta_wait_for_prior_grid();  // launched as a programmatic dependent of the mask kernel
  const long long tok = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (tok >= seq.total) return;
  const int b = seq_of(seq, tok);
  const int start = ta_seq_begin(seq, b);
  const int n = (seq.cu ? seq.cu[b + 1] : start + seq.n_uniform) - start;
  const int id = ids[tok];
  const int c = (id >= 0 && id < vocab) ? hist[(long long)b * vocab + id] : 0;
  u_static[tok] = ta_static_utility((int)(tok - start), n, c, (flags[tok] & TA_FLAG_ANCHOR_TOKEN) != 0, voucher[tok],
                                    beta, gamma, lambda);
}

}  // namespace

namespace {
cudaError_t finish_static_utility(const ta_policy& pol, const ta_seq_desc& seq, const int32_t* ids, const uint8_t* flags,
                                  const float* voucher, const int32_t* hist, float* u_static, cudaStream_t stream) {
  if (!u_static) return cudaSuccess;  // left to the forced-set kernel
  const int blocks = (int)((seq.total + 255) / 256);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks, 1, 1);
  cfg.blockDim = dim3(256, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  ta_pdl_attribute(&attr[0]);  // always directly behind the mask kernel
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, ta_ustatic_kernel, seq, ids, flags, voucher, hist, pol.vocab_size, pol.beta,
                            pol.gamma, pol.lambda, u_static);
}
}  // namespace

cudaError_t ta_launch_mask_conf(const ta_policy& pol, const ta_seq_desc& seq, const int32_t* ids, const float* conf,
                                float threshold, float budget, int span, int rank, uint8_t* flags, float* voucher,
                                float* u_static, int32_t* hist, ta_dev_status* status, cudaStream_t stream) {
  if (seq.total == 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(hist, 0, (size_t)seq.batch * pol.vocab_size * sizeof(int32_t), stream);
  if (e != cudaSuccess) return e;
  const int tiles = (int)((seq.total + kTile - 1) / kTile);
  ConfAnchors ca = {conf, threshold, budget, span, rank};
  ta_mask_kernel<<<tiles, kTile, 0, stream>>>(seq, ids, nullptr, nullptr, nullptr, nullptr, nullptr, 1, 1, span,
                                              pol.voucher_decay, pol.budget_decay, pol.age_steps, pol.vocab_size, flags,
                                              voucher, hist, status, ca);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return finish_static_utility(pol, seq, ids, flags, voucher, hist, u_static, stream);
}

cudaError_t ta_launch_mask(const ta_patterns* pats, const ta_policy& pol, const ta_seq_desc& seq, const int32_t* ids,
                           uint8_t* flags, float* voucher, float* u_static, int32_t* hist, ta_dev_status* status,
                           cudaStream_t stream) {
  if (seq.total == 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(hist, 0, (size_t)seq.batch * pol.vocab_size * sizeof(int32_t), stream);
  if (e != cudaSuccess) return e;
  const int tiles = (int)((seq.total + kTile - 1) / kTile);
  ta_mask_kernel<<<tiles, kTile, 0, stream>>>(seq, ids, pats->d_ids, pats->d_len, pats->d_budget, pats->d_span,
                                              pats->d_bloom, pats->n_pat, pats->max_len, pats->max_span,
                                              pol.voucher_decay, pol.budget_decay, pol.age_steps, pol.vocab_size, flags,
                                              voucher, hist, status, ConfAnchors{nullptr, 0.0f, 0.0f, 0, 0});
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return finish_static_utility(pol, seq, ids, flags, voucher, hist, u_static, stream);
}
