// Algorithm 1 in the decode loop: one new token per sequence and step, at most K cached tokens per unit afterwards.
// (Section 3.1: a retention policy selects S, |S| <= K, "after each generation step"; Algorithm 1 steps 1-10.)
//
// Per step three small kernels run around the selection kernels of ta_select.cu:
//   ta_stream_seq_kernel    one warp per sequence: token histogram, pattern match ending at the new token (longest
//                           pattern wins, then the lowest index), the new token's voucher from the anchors of the last
//                           TA_MAX_SPAN positions (Eq. 2 with budgets that decayed once per step since detection)
//   ta_stream_unit_kernel   one block per unit: appends the new token to the position-ordered state, adds this step's
//                           attention mass to A, updates the pension average P, and writes the two parts of the utility
//                           of Eq. 1 for the K+1 cached tokens
//   (selection of K of the K+1 tokens: ta_forced_kernel + ta_select_kernel, each unit taken as a sequence of K+1 tokens)
//   ta_stream_evict_kernel  one block per unit: removes the evicted token from the ordered state (4-byte entries move;
//                           key/value rows never do: the freed cache row is handed to the next token), then decays
//                           every voucher by budget_decay (Algorithm 1 step 10)
// All arithmetic that decides the selection is fp32 with one rounding per operation, in the order the CPU oracle uses.
#include "ta_internal.cuh"

namespace {

constexpr int kUnitThreads = 256;

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

__global__ void __launch_bounds__(kUnitThreads)
ta_stream_unit_kernel(ta_stream_dev st, const ta_stream_seq_info* __restrict__ info, const float* __restrict__ attn,
                      int vocab, float alpha, float beta, float gamma, float delta, float lambda, float rho,
                      float* __restrict__ u_att, float* __restrict__ u_static, float* __restrict__ vbuf,
                      uint8_t* __restrict__ flagbuf, ta_dev_status* status) {
  const int u = blockIdx.x;
  const int b = (u / st.Hkv) % st.B;
  const int C = st.K + 1, len = st.len;
  const size_t base = (size_t)u * C;
  const ta_stream_seq_info si = info[b];
  const int t = si.t;
  const float nf = (float)(t + 1);
  const float omr = __fsub_rn(1.0f, rho);
  for (int r = threadIdx.x; r < C; r += kUnitThreads) {
    float vu = 0.0f, us = 0.0f, vv = 0.0f;
    uint8_t fl = 0;
    if (r <= len) {
      int p, row, id;
      float A, P, V;
      int S;
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
        st.pos[base + r] = p;
        st.slot[base + r] = row;
        st.tok[base + r] = id;
        st.V[base + r] = V;
      }
      float a = 0.0f;
      if (row >= 0 && row < C) a = attn[base + row];
      else report(status, TA_ERR_DEVICE_BOUNDS, 6, u, row);
      A = __fadd_rn(A, a);
      P = __fadd_rn(__fmul_rn(rho, P), __fmul_rn(omr, a));
      if (p >= t - si.match_len + 1) S = 1;
      st.A[base + r] = A;
      st.P[base + r] = P;
      st.S[base + r] = (uint8_t)S;
      const int c = (id >= 0 && id < vocab) ? st.hist[(size_t)b * vocab + id] : 0;
      const float R = __fdiv_rn((float)(p + 1), nf);
      const float F = __fdiv_rn((float)c, nf);
      const float t0 = __fadd_rn(__fmul_rn(beta, R), __fmul_rn(gamma, S ? 1.0f : 0.0f));
      const float t1 = __fsub_rn(t0, __fmul_rn(lambda, F));
      us = __fadd_rn(t1, V);
      vu = __fadd_rn(__fmul_rn(alpha, A), __fmul_rn(delta, P));
      vv = V;
      fl = (uint8_t)((S ? TA_FLAG_ANCHOR_TOKEN : 0) | (V > 0.0f ? TA_FLAG_SPONSORED : 0));
    }
    u_att[base + r] = vu;
    u_static[base + r] = us;
    vbuf[base + r] = vv;
    flagbuf[base + r] = fl;
  }
}

// Moves entries (from, to] of one per-unit array down by one, 256 at a time in ascending order: a chunk is read by
// all threads before any of them writes it one place lower.
template <class T>
__device__ __forceinline__ void shift_down(T* a, int from, int to) {
  for (int r0 = from + 1; r0 <= to; r0 += kUnitThreads) {
    const int r = r0 + threadIdx.x;
    T v = T();
    if (r <= to) v = a[r];
    __syncthreads();
    if (r <= to) a[r - 1] = v;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kUnitThreads)
ta_stream_evict_kernel(ta_stream_dev st, int evict, const int32_t* __restrict__ idx, float budget_decay,
                       int32_t* __restrict__ evicted_pos) {
  __shared__ int e_sh;
  const int u = blockIdx.x;
  const int C = st.K + 1, K = st.K, len = st.len;  // len + 1 tokens are cached when this kernel starts
  const size_t base = (size_t)u * C;
  int kept = len + 1;
  if (evict) {
    if (threadIdx.x == 0) e_sh = K;  // all of idx[0..K) in place: the last entry goes
    __syncthreads();
    for (int r = threadIdx.x; r < K; r += kUnitThreads)
      if (idx[(size_t)u * K + r] != r) atomicMin(&e_sh, r);
    __syncthreads();
    const int e = e_sh;
    const int freed = st.slot[base + e];
    const int gone = st.pos[base + e];
    __syncthreads();
    shift_down(st.pos + base, e, K);
    shift_down(st.slot + base, e, K);
    shift_down(st.tok + base, e, K);
    shift_down(st.A + base, e, K);
    shift_down(st.P + base, e, K);
    shift_down(st.V + base, e, K);
    shift_down(st.S + base, e, K);
    if (threadIdx.x == 0) {
      st.next_slot[u] = freed;
      evicted_pos[u] = gone;
    }
    kept = K;
  } else if (threadIdx.x == 0) {
    st.next_slot[u] = len + 1;  // rows fill up in order until the cache is full
    evicted_pos[u] = -1;
  }
  __syncthreads();
  for (int r = threadIdx.x; r < kept; r += kUnitThreads) st.V[base + r] = __fmul_rn(st.V[base + r], budget_decay);
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

cudaError_t ta_launch_stream_unit(const ta_stream_dev& st, const ta_policy& pol, const ta_stream_seq_info* info,
                                  const float* attn, float* u_att, float* u_static, float* vbuf, uint8_t* flagbuf,
                                  ta_dev_status* status, cudaStream_t stream) {
  const int U = st.n_layers * st.B * st.Hkv;
  ta_stream_unit_kernel<<<U, kUnitThreads, 0, stream>>>(st, info, attn, pol.vocab_size, pol.alpha, pol.beta, pol.gamma,
                                                       pol.delta, pol.lambda, pol.pension_rho, u_att, u_static, vbuf,
                                                       flagbuf, status);
  return cudaGetLastError();
}

cudaError_t ta_launch_stream_evict(const ta_stream_dev& st, int evict, const int32_t* idx, float budget_decay,
                                   int32_t* evicted_pos, cudaStream_t stream) {
  const int U = st.n_layers * st.B * st.Hkv;
  ta_stream_evict_kernel<<<U, kUnitThreads, 0, stream>>>(st, evict, idx, budget_decay, evicted_pos);
  return cudaGetLastError();
}
