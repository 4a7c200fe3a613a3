// TEST INFRASTRUCTURE — not part of the product.
//
// Plain, slow, obviously-correct CPU statement of the Transactional Attention retention step, written from the
// paper's definitions (Algorithm 1; Eq. 1, 2, 3; Section 3.3). It exists so that tests can compare the CUDA
// library against it; it shares no code with that library and is never on a product path.
//
// Precision: the paper runs in fp16/fp32 and fixes no rounding. Where a float decides an integer (which tokens
// are retained) the decision is taken in fp32 with one rounding per operation, in the order written here
// (compile with -ffp-contract=off so no fused multiply-add is formed). The attention sums, which have a plain
// mathematical definition, are evaluated in double and rounded to fp32 once at the end.
//
// What pins each function is listed beside it; see tests/test_oracle_pins.py. End-task accuracy (does the model
// answer correctly after compaction) is "parity unpinned": it needs model weights that are not available.
//
// Build: g++ -O2 -std=c++17 -fopenmp -ffp-contract=off -shared -fPIC ta_oracle.cpp -o libta_oracle.so

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// bf16 -> double, exact (bf16 is the upper half of an IEEE fp32).
inline double bf16_to_double(uint16_t h) {
  uint32_t bits = (uint32_t)h << 16;
  float f;
  std::memcpy(&f, &bits, sizeof f);
  return (double)f;
}

}  // namespace

extern "C" {

int ora_num_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// ---------------------------------------------------------------------------------------------------------
// Anchor detection (Section 3.2 "Anchor detection", Algorithm 1 step 1), for ONE sequence of n token ids.
// The paper matches text patterns; here a pattern is a short sequence of token ids. Readings (the paper does
// not say): the anchor position of a multi-token match is its LAST token (the value follows it); every token of
// a match has S = 1; when several patterns end at the same position the longest wins, then the lowest index;
// a match may not start before the sequence does. The per-anchor budget is B_p decayed age_steps times by
// budget_decay (Section 3.2 "Sponsor budgets decay over time", Algorithm 1 step 10), each product rounded to fp32.
// Outputs: anchor_tok[i] (S_i), anchor_end[i], B_e[i] and L_e[i] at anchor ends (0 elsewhere).
// Pinned by: brute-force substring search on tiny alphabets; prefix-only decoys; sequence-boundary case.
void ora_anchors(int n, const int32_t* ids, int n_pat, const int32_t* pat_ids, const int32_t* pat_off,
                 const float* pat_budget, const int32_t* pat_span, float budget_decay, int age_steps,
                 uint8_t* anchor_tok, uint8_t* anchor_end, float* B_e, int32_t* L_e) {
  for (int i = 0; i < n; ++i) {
    anchor_tok[i] = 0;
    anchor_end[i] = 0;
    B_e[i] = 0.0f;
    L_e[i] = 0;
  }
  for (int e = 0; e < n; ++e) {
    int best = -1, best_len = 0;
    for (int p = 0; p < n_pat; ++p) {
      const int len = pat_off[p + 1] - pat_off[p];
      const int start = e - len + 1;
      if (start < 0) continue;
      bool match = true;
      for (int k = 0; k < len; ++k)
        if (ids[start + k] != pat_ids[pat_off[p] + k]) {
          match = false;
          break;
        }
      if (!match) continue;
      for (int k = 0; k < len; ++k) anchor_tok[start + k] = 1;  // every token of every match
      if (len > best_len) {                                     // longest wins; first (lowest p) among equals
        best = p;
        best_len = len;
      }
    }
    if (best >= 0) {
      float B = pat_budget[best];
      for (int t = 0; t < age_steps; ++t) B = B * budget_decay;
      anchor_end[e] = 1;
      B_e[e] = B;
      L_e[e] = pat_span[best];
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Anchor detection by a learned detector (Section 5.1 "Learned Anchor Detection"), for ONE sequence. The detector
// itself (an MLP on hidden states) is outside this path: its per-token confidence f(h_i) in [0, 1] is an input.
// Token i is an anchor iff f(h_i) > threshold (strictly, as the paper writes it); anchors are single tokens, so
// S_i = 1 exactly on them. Two variants, both feeding the voucher sum of Eq. 2 unchanged:
//   TA-Learned   (rank = 0): threshold 0.5, every anchor sponsors with the fixed budget B.
//   TA-LearnRank (rank = 1): threshold 0.3, the confidence takes the place of the budget: B_i = budget * f(h_i)
//                (budget = 1 gives the paper's equation V_j = sum_i f(h_i) 0.8^(j-i) 1[f(h_i) > 0.3, i < j <= i+L]).
// The budget is aged like a pattern's (age_steps products with budget_decay, fp32). A NaN confidence is no anchor.
// Pinned by: closed forms f*0.8^k; threshold edge (equal is not above); rank = 0 on the indicator of a token id
// equals the pattern detector with that one-token pattern.
void ora_anchors_conf(int n, const float* conf, float threshold, float budget, int span, int rank,
                      float budget_decay, int age_steps, uint8_t* anchor_tok, uint8_t* anchor_end, float* B_e,
                      int32_t* L_e) {
  for (int i = 0; i < n; ++i) {
    const bool is_anchor = conf[i] > threshold;
    anchor_tok[i] = is_anchor ? 1 : 0;
    anchor_end[i] = is_anchor ? 1 : 0;
    B_e[i] = 0.0f;
    L_e[i] = 0;
    if (is_anchor) {
      float B = rank ? budget * conf[i] : budget;
      for (int t = 0; t < age_steps; ++t) B = B * budget_decay;
      B_e[i] = B;
      L_e[i] = span;
    }
  }
}

// ---------------------------------------------------------------------------------------------------------
// Voucher allocation (Eq. 2; Algorithm 1 steps 2-6) for one sequence:
//   V_j = sum over anchors i with i < j <= i + L_i of B_i * decay^(j-i).
// decay^k is built by repeated fp32 multiplication (w[1] = decay, w[k] = w[k-1]*decay); the sum over anchors is
// taken nearest anchor first (k = j-i ascending), one fp32 rounding per product and per addition. Spans stop at
// the end of the sequence.
// Pinned by: the closed form B*0.8^k (12, 9.6, 7.68, 6.144, 4.9152, 3.93216 for B=15) and the paper's printed
// "approx 3.9" for k = 6; two anchors three apart add on the overlap; a span clipped at the sequence end.
void ora_vouchers(int n, const uint8_t* anchor_end, const float* B_e, const int32_t* L_e, float voucher_decay,
                  float* V) {
  int Lmax = 0;
  for (int i = 0; i < n; ++i)
    if (anchor_end[i] && L_e[i] > Lmax) Lmax = L_e[i];
  std::vector<float> w(Lmax + 2, 0.0f);
  if (Lmax >= 1) w[1] = voucher_decay;
  for (int k = 2; k <= Lmax; ++k) w[k] = w[k - 1] * voucher_decay;
  for (int j = 0; j < n; ++j) {
    float v = 0.0f;
    for (int k = 1; k <= Lmax; ++k) {
      const int i = j - k;
      if (i < 0) break;
      if (anchor_end[i] && k <= L_e[i]) {
        const float term = B_e[i] * w[k];
        v = v + term;
      }
    }
    V[j] = v;
  }
}

// ---------------------------------------------------------------------------------------------------------
// Attention-free part of the utility (Eq. 1 without alpha*A and delta*P; this is exactly Eq. 3, TA-Fast):
//   u0_i = beta*R_i + gamma*S_i - lambda*F_i + V_i,   R_i = i/n with the paper's 1-based i.
// Reading for F_i (the paper gives no formula): the relative frequency of the token's id within its sequence.
// fp32, evaluated as ((beta*R + gamma*S) - lambda*F) + V.
// Pinned by: a hand-computed 6-token example (tests/golden/utility_example.txt).
void ora_static_utility(int n, const int32_t* ids, const uint8_t* anchor_tok, const float* V, float beta,
                        float gamma, float lambda, float* u0) {
  for (int i = 0; i < n; ++i) {
    int c = 0;
    for (int j = 0; j < n; ++j) c += (ids[j] == ids[i]);
    const float R = (float)(i + 1) / (float)n;
    const float S = anchor_tok[i] ? 1.0f : 0.0f;
    const float F = (float)c / (float)n;
    const float bR = beta * R;
    const float gS = gamma * S;
    const float lF = lambda * F;
    const float t0 = bR + gS;
    const float t1 = t0 - lF;
    u0[i] = t1 + V[i];
  }
}

// Same result as ora_static_utility with the occurrence count taken from a histogram, so that full-size
// workloads finish. Integer counting is exact, so the two agree bit for bit (checked in the pin tests).
void ora_static_utility_hist(int n, const int32_t* ids, int vocab, const uint8_t* anchor_tok, const float* V,
                             float beta, float gamma, float lambda, float* u0) {
  std::vector<int32_t> cnt(vocab, 0);
  for (int i = 0; i < n; ++i) cnt[ids[i]]++;
  for (int i = 0; i < n; ++i) {
    const float R = (float)(i + 1) / (float)n;
    const float S = anchor_tok[i] ? 1.0f : 0.0f;
    const float F = (float)cnt[ids[i]] / (float)n;
    const float bR = beta * R;
    const float gS = gamma * S;
    const float lF = lambda * F;
    const float t0 = bR + gS;
    const float t1 = t0 - lF;
    u0[i] = t1 + V[i];
  }
}

// ---------------------------------------------------------------------------------------------------------
// Attention terms of Eq. 1 for one (sequence, KV head): A_i ("cumulative attention across heads and steps",
// Appendix A Definition 1: A_i = sum over steps and heads of a_{h,i}) and the pension P_i ("exponential moving
// average of past attention"). Reading: the steps are the last W' = min(W, n) query positions, the heads are the
// G query heads that share this KV head, attention is softmax(scale * q.k) over the keys a row may see
// (causal: key i <= query position), and the EMA runs over the W' rows in position order with coefficient rho
// and zero initial state, i.e. weight (1-rho)*rho^(W'-1-t) on row t.
//   Q: bf16 bits, [G][W][d] with strides (q_stride_h, q_stride_t) in elements; row t is position n - W + t;
//      rows with negative position are ignored.
//   K: bf16 bits, n rows with stride k_stride_n.
// Everything in double; rounded to fp32 on output.
// Pinned by: every softmax row sums to one => sum_i A_i = G*W', sum_i P_i = G*(1 - rho^W'); W=1,G=1 equals a
// library softmax; equal keys => a_{t,i} = 1/(q_t + 1); rho = 0 => P = last row; causal zeros.
void ora_attention(int n, int G, int W, int d, const uint16_t* Q, int64_t q_stride_h, int64_t q_stride_t,
                   const uint16_t* K, int64_t k_stride_n, double scale, int causal, double rho, float* A_out,
                   float* P_out) {
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int Wp = W < n ? W : n;
  std::vector<double> A(n, 0.0), P(n, 0.0), s(n), q(d);
  for (int h = 0; h < G; ++h) {
    for (int tp = 0; tp < Wp; ++tp) {
      const int t = W - Wp + tp;     // row inside the W-row window buffer
      const int pos = n - Wp + tp;   // absolute position of this query
      const int last = causal ? pos : n - 1;
      for (int c = 0; c < d; ++c) q[c] = bf16_to_double(Q[h * q_stride_h + t * q_stride_t + c]);
      double mx = -INFINITY;
      for (int i = 0; i <= last; ++i) {
        const uint16_t* kr = K + (int64_t)i * k_stride_n;
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += q[c] * bf16_to_double(kr[c]);
        s[i] = scale * acc;
        if (s[i] > mx) mx = s[i];
      }
      double Z = 0.0;
      for (int i = 0; i <= last; ++i) {
        s[i] = std::exp(s[i] - mx);
        Z += s[i];
      }
      const double wt = (1.0 - rho) * std::pow(rho, (double)(Wp - 1 - tp));
      for (int i = 0; i <= last; ++i) {
        const double a = s[i] / Z;
        A[i] += a;
        P[i] += wt * a;
      }
    }
  }
  for (int i = 0; i < n; ++i) {
    A_out[i] = (float)A[i];
    if (P_out) P_out[i] = (float)P[i];
  }
}

// ---------------------------------------------------------------------------------------------------------
// The same sums taken over ALL query heads of a layer (the literal "cumulative attention across heads" of Eq. 1 and
// Appendix A Definition 1): query head h attends to the keys of its KV head h / G. One A and one P per token, shared
// by every KV head of the layer.
//   Q: [Hq][W][d] as above; K: Hkv blocks of n rows, block g at K + g*k_stride_h.
// Pinned by: sum_i A_i = Hq*W'; equals the sum over KV heads of ora_attention (a different summation order in
// double, so equal to rounding); with Hkv = 1 it is ora_attention.
void ora_attention_allheads(int n, int Hq, int Hkv, int W, int d, const uint16_t* Q, int64_t q_stride_h,
                            int64_t q_stride_t, const uint16_t* K, int64_t k_stride_h, int64_t k_stride_n,
                            double scale, int causal, double rho, float* A_out, float* P_out) {
  if (scale <= 0.0) scale = 1.0 / std::sqrt((double)d);
  const int G = Hq / Hkv;
  const int Wp = W < n ? W : n;
  std::vector<double> A(n, 0.0), P(n, 0.0), s(n), q(d);
  for (int h = 0; h < Hq; ++h) {
    const uint16_t* Kg = K + (int64_t)(h / G) * k_stride_h;
    for (int tp = 0; tp < Wp; ++tp) {
      const int t = W - Wp + tp;
      const int pos = n - Wp + tp;
      const int last = causal ? pos : n - 1;
      for (int c = 0; c < d; ++c) q[c] = bf16_to_double(Q[h * q_stride_h + t * q_stride_t + c]);
      double mx = -INFINITY;
      for (int i = 0; i <= last; ++i) {
        const uint16_t* kr = Kg + (int64_t)i * k_stride_n;
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += q[c] * bf16_to_double(kr[c]);
        s[i] = scale * acc;
        if (s[i] > mx) mx = s[i];
      }
      double Z = 0.0;
      for (int i = 0; i <= last; ++i) {
        s[i] = std::exp(s[i] - mx);
        Z += s[i];
      }
      const double wt = (1.0 - rho) * std::pow(rho, (double)(Wp - 1 - tp));
      for (int i = 0; i <= last; ++i) {
        const double a = s[i] / Z;
        A[i] += a;
        P[i] += wt * a;
      }
    }
  }
  for (int i = 0; i < n; ++i) {
    A_out[i] = (float)A[i];
    if (P_out) P_out[i] = (float)P[i];
  }
}

// ---------------------------------------------------------------------------------------------------------
// Full utility of Eq. 1 from its parts: u = (alpha*A + delta*P) + u0, fp32, one rounding per operation.
void ora_utility(int n, float alpha, float delta, const float* A, const float* P, const float* u0, float* u) {
  for (int i = 0; i < n; ++i) {
    const float aA = alpha * A[i];
    const float dP = delta * (P ? P[i] : 0.0f);
    const float t = aA + dP;
    u[i] = t + u0[i];
  }
}

// ---------------------------------------------------------------------------------------------------------
// Token selection (Algorithm 1 step 8 with the budget partition of Section 3.3) for one unit.
//   K_eff = min(K, n); K_eff == n keeps everything. Otherwise K = K_main + K_protected with
//   p = K_protected (k_protected < 0: K_eff - n_sink - n_recent, the K_p = K - 1 - W of Theorems 2-4; clipped to
//   [0, K_eff]). Mandatory tokens "are drawn from the main pool": the list first-token sinks 0,1,.. then recents
//   n-1, n-2, .. is taken in that order while main slots last. The protected pool holds the sponsored tokens
//   (V > 0) not already mandatory, largest voucher first, lower position first among equals. All remaining slots
//   (unused protected slots included: "a partition within K", exactly K tokens are retained) go to the other
//   tokens by utility, largest first, lower position first among equals. The result is reported in ascending
//   position order, as index_select with a sorted index keeps causal order.
// Pinned by: exhaustive search over subsets on n <= 12; no anchors and no mandatory tokens => library top-K;
// K >= n identity; |S| = K_eff; Theorem 2, the minimum-budget corollary, Theorem 4; the worked 4096-token example.
void ora_select(int n, int K, int n_sink, int n_recent, int k_protected, const float* V, const float* u,
                int32_t* idx_out /*K*/, int32_t* count_out) {
  const int K_eff = K < n ? K : n;
  std::vector<char> keep(n, 0);
  if (K_eff == n) {
    for (int i = 0; i < n; ++i) keep[i] = 1;
  } else {
    int p = k_protected < 0 ? K_eff - n_sink - n_recent : k_protected;
    if (p < 0) p = 0;
    if (p > K_eff) p = K_eff;
    const int K_main = K_eff - p;
    int used = 0;
    // mandatory, in priority order, while main slots last
    int taken_m = 0;
    for (int i = 0; i < n_sink && i < n && taken_m < K_main; ++i)
      if (!keep[i]) {
        keep[i] = 1;
        ++taken_m;
      }
    for (int r = 0; r < n_recent && r < n && taken_m < K_main; ++r) {
      const int i = n - 1 - r;
      if (!keep[i]) {
        keep[i] = 1;
        ++taken_m;
      }
    }
    used = taken_m;
    // protected pool
    std::vector<int> cand;
    for (int i = 0; i < n; ++i)
      if (!keep[i] && V[i] > 0.0f) cand.push_back(i);
    std::stable_sort(cand.begin(), cand.end(), [&](int a, int b) { return V[a] > V[b]; });
    for (int r = 0; r < (int)cand.size() && r < p; ++r) {
      keep[cand[r]] = 1;
      ++used;
    }
    // main pool by utility
    std::vector<int> rest;
    for (int i = 0; i < n; ++i)
      if (!keep[i]) rest.push_back(i);
    std::stable_sort(rest.begin(), rest.end(), [&](int a, int b) { return u[a] > u[b]; });
    for (int r = 0; r < (int)rest.size() && used < K_eff; ++r) {
      keep[rest[r]] = 1;
      ++used;
    }
  }
  int c = 0;
  for (int i = 0; i < n; ++i)
    if (keep[i]) idx_out[c++] = i;
  *count_out = c;
  for (int r = c; r < K; ++r) idx_out[r] = -1;
}

// ---------------------------------------------------------------------------------------------------------
// Eviction (Algorithm 1 step 9; "index_select on KV tensors along the sequence dimension"): copy the retained
// rows in index order, bit for bit; rows beyond count are zero.
// Pinned by: byte equality with library fancy indexing.
void ora_compact(int d, int K, const uint16_t* src, int64_t stride_n, const int32_t* idx, int count,
                 uint16_t* dst /*[K][d]*/) {
  for (int r = 0; r < K; ++r) {
    if (r < count)
      std::memcpy(dst + (int64_t)r * d, src + (int64_t)idx[r] * stride_n, sizeof(uint16_t) * d);
    else
      std::memset(dst + (int64_t)r * d, 0, sizeof(uint16_t) * d);
  }
}

// ---------------------------------------------------------------------------------------------------------
// Algorithm 1 for one layer of a batch: the functions above chained, units (sequence, KV head) in an OpenMP
// parallel-for. Tensors are dense: Q [B][Hq][W][d], K and V [B][Hkv][n][d] (uniform) or [Hkv][total][d] (ragged,
// cu given). Per-sequence steps are done once per sequence (they do not depend on the head); in fast mode the
// selection is also per sequence. Outputs: idx [B][Hkv][K], count [B][Hkv], k_out / v_out [B][Hkv][K][d].
// seconds_out[0] = per-sequence steps, seconds_out[1] = per-unit steps (wall clock).
void ora_compress_layer(int B, const int32_t* cu /*B+1*/, int uniform, int Hq, int Hkv, int d, int W, int K,
                        const int32_t* ids, int vocab, int n_pat, const int32_t* pat_ids, const int32_t* pat_off,
                        const float* pat_budget, const int32_t* pat_span, float alpha, float beta, float gamma,
                        float delta, float lambda, float voucher_decay, float budget_decay, int age_steps,
                        int n_sink, int n_recent, int k_protected, double rho, double scale, int causal, int fast,
                        const uint16_t* Q, const uint16_t* Kc, const uint16_t* Vc, int32_t* idx_out,
                        int32_t* count_out, uint16_t* k_out, uint16_t* v_out, double* seconds_out) {
  const int64_t total = cu[B];
  const int G = Hq / Hkv;
  std::vector<float> V(total), u0(total);
  std::vector<uint8_t> atok(total), aend(total);
  double t0 = 0, t1 = 0, t2 = 0;
#ifdef _OPENMP
  t0 = omp_get_wtime();
#endif
#pragma omp parallel for schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    const int n = cu[b + 1] - cu[b];
    const int64_t o = cu[b];
    std::vector<float> Be(n);
    std::vector<int32_t> Le(n);
    ora_anchors(n, ids + o, n_pat, pat_ids, pat_off, pat_budget, pat_span, budget_decay, age_steps, atok.data() + o,
                aend.data() + o, Be.data(), Le.data());
    ora_vouchers(n, aend.data() + o, Be.data(), Le.data(), voucher_decay, V.data() + o);
    ora_static_utility_hist(n, ids + o, vocab, atok.data() + o, V.data() + o, beta, gamma, lambda, u0.data() + o);
  }
#ifdef _OPENMP
  t1 = omp_get_wtime();
#endif
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b) {
    for (int g = 0; g < Hkv; ++g) {
      const int n = cu[b + 1] - cu[b];
      const int64_t o = cu[b];
      const uint16_t* kbase = uniform ? Kc + ((int64_t)(b * Hkv + g) * n) * d : Kc + ((int64_t)g * total + o) * d;
      const uint16_t* vbase = uniform ? Vc + ((int64_t)(b * Hkv + g) * n) * d : Vc + ((int64_t)g * total + o) * d;
      std::vector<float> u(n);
      if (fast) {
        for (int i = 0; i < n; ++i) u[i] = u0[o + i];
      } else {
        std::vector<float> A(n), P(n);
        const uint16_t* qbase = Q + ((int64_t)(b * Hq + g * G) * W) * d;
        ora_attention(n, G, W, d, qbase, (int64_t)W * d, d, kbase, d, scale, causal, rho, A.data(), P.data());
        ora_utility(n, alpha, delta, A.data(), P.data(), u0.data() + o, u.data());
      }
      int32_t* idx = idx_out + (int64_t)(b * Hkv + g) * K;
      int32_t cnt = 0;
      ora_select(n, K, n_sink, n_recent, k_protected, V.data() + o, u.data(), idx, &cnt);
      count_out[b * Hkv + g] = cnt;
      ora_compact(d, K, kbase, d, idx, cnt, k_out + (int64_t)(b * Hkv + g) * K * d);
      ora_compact(d, K, vbase, d, idx, cnt, v_out + (int64_t)(b * Hkv + g) * K * d);
    }
  }
#ifdef _OPENMP
  t2 = omp_get_wtime();
#endif
  if (seconds_out) {
    seconds_out[0] = t1 - t0;
    seconds_out[1] = t2 - t1;
  }
}

}  // extern "C"
