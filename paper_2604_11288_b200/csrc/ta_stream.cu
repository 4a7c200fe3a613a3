// Algorithm 1 in the decode loop: one new token per sequence and step, at most K cached tokens per unit afterwards.
// (Section 3.1: a retention policy selects S, |S| <= K, "after each generation step"; Algorithm 1 steps 1-10.)
//
// Per step two kernels run:
//   ta_stream_seq_kernel    one warp per sequence: token histogram, pattern match ending at the new token (longest
//                           pattern wins, then the lowest index), the new token's voucher from the anchors of the last
//                           TA_MAX_SPAN positions (Eq. 2 with budgets that decayed once per step since detection)
//   ta_stream_step_kernel   one block per unit with the unit's K+1 entries in shared memory: appends the new token to
//                           the position-ordered state, adds this step's attention mass to A, updates the pension
//                           average P, forms the utility of Eq. 1, applies the budget partition of Section 3.3 to the
//                           K+1 cached tokens (exactly one token loses), removes it from the ordered state (4-byte
//                           entries move; key/value rows never do: the freed cache row is handed to the next token) and
//                           decays every voucher by budget_decay (Algorithm 1 step 10)
// All arithmetic that decides the selection is fp32 with one rounding per operation, in the order the CPU oracle uses.
#include <atomic>

#include "ta_internal.cuh"

namespace {

__device__ __forceinline__ void report(ta_dev_status* st, int code, int where, int d0, int d1) {
  if (atomicCAS(&st->code, 0, code) == 0) {
    st->where = where;
    st->detail0 = d0;
    st->detail1 = d1;
  }
}

__global__ void __launch_bounds__(32) ta_stream_seq_kernel(ta_stream_dev st, const int32_t* __restrict__ new_ids,
                                                           const int32_t* __restrict__ p_ids,
                                                           const int32_t* __restrict__ p_len,
                                                           const float* __restrict__ p_budget,
                                                           const int32_t* __restrict__ p_span, int n_pat,
                                                           float voucher_decay, float budget_decay, int vocab,
                                                           ta_stream_seq_info* __restrict__ info,
                                                           ta_dev_status* status) {
  const int b = blockIdx.x, lane = threadIdx.x;
  const int x = new_ids[b];
  const int t = st.n_seen[b];
  int32_t* ring = st.tok_ring + (size_t)b * TA_MAX_PATTERN_LEN;
  float* aB = st.anc_B + (size_t)b * TA_MAX_SPAN;
  int32_t* aL = st.anc_L + (size_t)b * TA_MAX_SPAN;
  if (lane == 0) {
    ring[t % TA_MAX_PATTERN_LEN] = x;
    if (x >= 0 && x < vocab) atomicAdd(&st.hist[(size_t)b * vocab + x], 1);
    else report(status, TA_ERR_DEVICE_BOUNDS, 5, b, x);
  }
  __syncwarp();
  // patterns ending at t
  int best = -1, best_len = 0;
  for (int p = lane; p < n_pat; p += 32) {
    const int len = p_len[p];
    if (len > t + 1 || len <= best_len) continue;  // within a lane p ascends: a later pattern wins only if longer
    bool ok = true;
    for (int k = 0; k < len; ++k)
      ok = ok && (((volatile int32_t*)ring)[(t - len + 1 + k) % TA_MAX_PATTERN_LEN] == p_ids[p * TA_MAX_PATTERN_LEN + k]);
    if (ok) {
      best = p;
      best_len = len;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const int ol = __shfl_xor_sync(0xffffffffu, best_len, o), ob = __shfl_xor_sync(0xffffffffu, best, o);
    if (ol > best_len || (ol == best_len && ob >= 0 && (best < 0 || ob < best))) {
      best_len = ol;
      best = ob;
    }
  }
  if (lane == 0) {
    // voucher of the new token from the anchors at t-1, t-2, ..: nearest first
    float v = 0.0f, w = 1.0f;
    const int kmax = t < TA_MAX_SPAN ? t : TA_MAX_SPAN;
    for (int k = 1; k <= kmax; ++k) {
      w = __fmul_rn(w, voucher_decay);
      const int i = (t - k) % TA_MAX_SPAN;
      const int L = aL[i];
      if (L > 0 && k <= L) {
        float Bk = aB[i];
        for (int s = 0; s < k; ++s) Bk = __fmul_rn(Bk, budget_decay);
        v = __fadd_rn(v, __fmul_rn(Bk, w));
      }
    }
    aB[t % TA_MAX_SPAN] = best >= 0 ? p_budget[best] : 0.0f;
    aL[t % TA_MAX_SPAN] = best >= 0 ? p_span[best] : 0;
    st.n_seen[b] = t + 1;
    ta_stream_seq_info si;
    si.t = t;
    si.match_len = best_len;  // the longest matching pattern covers the tokens of every pattern that ends here
    si.v_new = v;
    si.id = x;
    info[b] = si;
  }
}

__device__ __forceinline__ uint32_t sortable_key(float f) {
  uint32_t b = __float_as_uint(f);
  if ((b << 1) == 0u) b = 0u;  // -0 == +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// One block per unit; the unit's K+1 entries live in shared memory for the whole step. Thread t owns the contiguous
// entries [t*per, (t+1)*per), so everything that depends on position order is a block-wide scan of per-thread counts.
// Selection (Section 3.3 on the K+1 cached tokens): mandatory sinks and recents; the protected pool = the sponsored,
// non-mandatory tokens with the largest vouchers (lower position first among equals), found with a 4-pass radix
// select on the voucher keys when there are more candidates than protected slots; exactly one token is then not
// forced and loses: the one with the smallest utility, the latest position among equals.
__global__ void ta_stream_step_kernel(ta_stream_dev st, const ta_stream_seq_info* __restrict__ info,
                                      const float* __restrict__ attn, int vocab, float alpha, float beta, float gamma,
                                      float delta, float lambda, float rho, float budget_decay, int n_sink,
                                      int n_recent, int k_protected, int32_t* __restrict__ evicted_pos,
                                      ta_dev_status* status) {
  extern __shared__ __align__(16) unsigned char smem[];
  ta_wait_for_prior_grid();  // launched as a programmatic dependent of the per-sequence kernel
  const int u = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
  const int b = (u / st.Hkv) % st.B;
  const int K = st.K, C = K + 1, len = st.len, n = len + 1;
  const size_t base = (size_t)u * C;
  int32_t* s_pos = reinterpret_cast<int32_t*>(smem);
  int32_t* s_slot = s_pos + C;
  int32_t* s_tok = s_slot + C;
  float* s_A = reinterpret_cast<float*>(s_tok + C);
  float* s_P = s_A + C;
  float* s_V = s_P + C;
  uint32_t* s_ku = reinterpret_cast<uint32_t*>(s_V + C);  // sortable key of the utility
  uint8_t* s_S = reinterpret_cast<uint8_t*>(s_ku + C);
  uint8_t* s_forced = s_S + C;
  __shared__ uint32_t hist[256];
  __shared__ uint32_t scan[512];
  __shared__ unsigned long long best;
  __shared__ uint32_t sel_prefix, sel_mask;
  __shared__ int sel_remaining, cand_total;

  const ta_stream_seq_info si = info[b];
  const int t = si.t;
  const float nf = (float)(t + 1);
  const float omr = __fsub_rn(1.0f, rho);
  // ---- append, attention update, utility
  for (int r = tid; r < n; r += nt) {
    int p, row, id, S;
    float A, P, V;
    if (r < len) {
      p = st.pos[base + r];
      row = st.slot[base + r];
      id = st.tok[base + r];
      A = st.A[base + r];
      P = st.P[base + r];
      V = st.V[base + r];
      S = st.S[base + r];
    } else {
      p = t;
      row = st.next_slot[u];
      id = si.id;
      A = 0.0f;
      P = 0.0f;
      V = si.v_new;
      S = 0;
    }
    float a = 0.0f;
    if (row >= 0 && row < C) a = attn[base + row];
    else report(status, TA_ERR_DEVICE_BOUNDS, 6, u, row);
    A = __fadd_rn(A, a);
    P = __fadd_rn(__fmul_rn(rho, P), __fmul_rn(omr, a));
    if (p >= t - si.match_len + 1) S = 1;
    const int c = (id >= 0 && id < vocab) ? st.hist[(size_t)b * vocab + id] : 0;
    const float R = __fdiv_rn((float)(p + 1), nf);
    const float F = __fdiv_rn((float)c, nf);
    const float t0 = __fadd_rn(__fmul_rn(beta, R), __fmul_rn(gamma, S ? 1.0f : 0.0f));
    const float t1 = __fsub_rn(t0, __fmul_rn(lambda, F));
    const float us = __fadd_rn(t1, V);
    const float ua = __fadd_rn(__fmul_rn(alpha, A), __fmul_rn(delta, P));
    s_pos[r] = p;
    s_slot[r] = row;
    s_tok[r] = id;
    s_A[r] = A;
    s_P[r] = P;
    s_V[r] = V;
    s_S[r] = (uint8_t)S;
    s_ku[r] = sortable_key(__fadd_rn(ua, us));
  }
  __syncthreads();
  int e = -1;  // entry to evict
  if (n > K) {
    // ---- budget partition on n = K + 1 tokens
    int p = k_protected < 0 ? K - n_sink - n_recent : k_protected;
    p = max(0, min(p, K));
    const int K_main = K - p;
    const int sinks = min(n_sink, n);
    const int recents = max(0, min(n_recent, n - sinks));
    const int s_take = min(sinks, K_main);
    const int r_take = min(recents, K_main - s_take);
    auto mandatory = [&](int i) { return i < s_take || i >= n - r_take; };
    const int per = (n + nt - 1) / nt;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    // candidates of the protected pool
    int my_c = 0;
    for (int i = lo; i < hi; ++i) my_c += (s_V[i] > 0.0f && !mandatory(i));
    if (tid == 0) cand_total = 0;
    __syncthreads();
    if (my_c) atomicAdd(&cand_total, my_c);
    __syncthreads();
    const int cs = cand_total;
    uint32_t thresh = 0;
    int ties = 0;
    const bool all_protected = cs <= p;
    if (!all_protected && p > 0) {
      if (tid == 0) {
        sel_prefix = 0;
        sel_mask = 0;
        sel_remaining = p;
      }
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        for (int k = tid; k < 256; k += nt) hist[k] = 0;
        __syncthreads();
        const uint32_t prefix = sel_prefix, mask = sel_mask;
        for (int i = lo; i < hi; ++i) {
          const float v = s_V[i];
          if (v > 0.0f && !mandatory(i)) {
            const uint32_t key = sortable_key(v);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
          }
        }
        __syncthreads();
        if (tid == 0) {
          int remaining = sel_remaining;
          uint32_t cum = 0;
          int bin = 255;
          for (; bin > 0; --bin) {
            if (cum + hist[bin] >= (uint32_t)remaining) break;
            cum += hist[bin];
          }
          sel_remaining = remaining - (int)cum;
          sel_prefix = prefix | ((uint32_t)bin << shift);
          sel_mask = mask | (255u << shift);
        }
        __syncthreads();
      }
      thresh = sel_prefix;
      ties = sel_remaining;
    }
    // ---- forced set: mandatory, vouchers above the threshold, and the first `ties` of the vouchers equal to it
    int my_ties = 0;
    for (int i = lo; i < hi; ++i) {
      const float v = s_V[i];
      const bool cand = v > 0.0f && !mandatory(i);
      bool f = mandatory(i);
      if (cand && p > 0) {
        if (all_protected) f = true;
        else {
          const uint32_t key = sortable_key(v);
          if (key > thresh) f = true;
          else if (key == thresh) ++my_ties;
        }
      }
      s_forced[i] = f ? 1 : 0;
    }
    if (!all_protected && p > 0) {
      // exclusive scan of the per-thread tie counts (thread order = position order)
      scan[tid] = (uint32_t)my_ties;
      __syncthreads();
      for (int off = 1; off < nt; off <<= 1) {
        const uint32_t add = tid >= off ? scan[tid - off] : 0u;
        __syncthreads();
        scan[tid] += add;
        __syncthreads();
      }
      int seen = (int)scan[tid] - my_ties;
      for (int i = lo; i < hi; ++i) {
        const float v = s_V[i];
        if (v > 0.0f && !mandatory(i) && sortable_key(v) == thresh) {
          if (seen < ties) s_forced[i] = 1;
          ++seen;
        }
      }
    }
    if (tid == 0) best = ~0ull;
    __syncthreads();
    // ---- the loser: smallest utility among the tokens that are not forced, latest position among equals
    unsigned long long mine = ~0ull;
    for (int i = lo; i < hi; ++i)
      if (!s_forced[i]) {
        const unsigned long long cnd = ((unsigned long long)s_ku[i] << 32) | (uint32_t)(~(uint32_t)i);
        mine = cnd < mine ? cnd : mine;
      }
    if (mine != ~0ull) atomicMin(&best, mine);
    __syncthreads();
    e = (int)(~(uint32_t)(best & 0xffffffffull));
    if (best == ~0ull) e = K;  // cannot happen: K + 1 tokens and at most K forced
  }
  // ---- write the state back without the evicted entry; vouchers decay (Algorithm 1 step 10)
  const int kept = e >= 0 ? K : n;
  for (int r = tid; r < kept; r += nt) {
    const int src = (e >= 0 && r >= e) ? r + 1 : r;
    st.pos[base + r] = s_pos[src];
    st.slot[base + r] = s_slot[src];
    st.tok[base + r] = s_tok[src];
    st.A[base + r] = s_A[src];
    st.P[base + r] = s_P[src];
    st.V[base + r] = __fmul_rn(s_V[src], budget_decay);
    st.S[base + r] = s_S[src];
  }
  if (tid == 0) {
    st.next_slot[u] = e >= 0 ? s_slot[e] : n;  // rows fill up in order until the cache is full
    evicted_pos[u] = e >= 0 ? s_pos[e] : -1;
  }
}

}  // namespace

cudaError_t ta_launch_stream_seq(const ta_stream_dev& st, const ta_patterns* pats, const ta_policy& pol,
                                 const int32_t* new_ids, ta_stream_seq_info* info, ta_dev_status* status,
                                 cudaStream_t stream) {
  ta_stream_seq_kernel<<<st.B, 32, 0, stream>>>(st, new_ids, pats->d_ids, pats->d_len, pats->d_budget, pats->d_span,
                                                 pats->n_pat, pol.voucher_decay, pol.budget_decay, pol.vocab_size, info,
                                                 status);
  return cudaGetLastError();
}

cudaError_t ta_launch_stream_step(const ta_stream_dev& st, const ta_policy& pol, const ta_stream_seq_info* info,
                                  const float* attn, int32_t* evicted_pos, ta_dev_status* status,
                                  cudaStream_t stream) {
  const int U = st.n_layers * st.B * st.Hkv, C = st.K + 1;
  const int threads = C <= 512 ? 128 : 512;
  const size_t smem = (size_t)C * (7 * 4 + 2) + 16;
  // per device; setting the (sticky) attribute twice from two threads is harmless, the flag only saves the call
  static std::atomic<bool> attr_set[64];
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!attr_set[dev & 63].load(std::memory_order_acquire)) {
    e = cudaFuncSetAttribute(ta_stream_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63].store(true, std::memory_order_release);
  }
  // the launch overlaps the tail of the kernel before it on the stream (ta_stream_seq_kernel in ta_stream_step)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)U, 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  ta_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, ta_stream_step_kernel, st, info, attn, pol.vocab_size, pol.alpha, pol.beta, pol.gamma,
                            pol.delta, pol.lambda, pol.pension_rho, pol.budget_decay, pol.n_sink, pol.n_recent,
                            pol.k_protected, evicted_pos, status);
}
