// Step 2 of the retention path: the attention terms of Eq. 1 (A_i, the pension P_i) over the observation window,
// optionally fused with the rest of the utility. sm_100a only: TMA tile loads, tcgen05 tensor-core MMAs with the
// accumulators in tensor memory, and a thread-block cluster per unit for the softmax statistics.
//
// For unit (l, b, g) the score matrix is S = Q_obs[heads of g] * K^T, M = G*W rows (<= 256) by n keys. Each row is
// softmax-normalised over the keys it may see and the result is summed over rows per key. The normaliser of a row
// needs every key before any column sum can be finished, so the keys are swept twice:
//   pass 1  S = Q * Ktile^T   (TMEM lane = query row)  -> running max and sum of exponentials per row
//   pass 2  S^T = Ktile * Q^T (TMEM lane = key)        -> A_i = sum_rows exp2(s*c - lse_row), P_i likewise
// Both passes use the same shared-memory operand tiles (both K-major, 128-byte swizzle); only the roles in the
// instruction descriptor swap, which puts the reduction axis of each pass along a thread's own registers.
// The keys of a unit are split over the CTAs of a cluster (each CTA owns a contiguous range of 128-key tiles);
// between the passes the CTAs exchange their per-row statistics through distributed shared memory. Pass 2
// re-reads the CTA's own tiles, which are still in L2, so HBM sees every key once.
// When the caller supplies the rows' log-sum-exp (lse_obs), pass 1 is skipped.
//
// Warp roles (320 threads): warp 0 TMA producer, warp 1 MMA issuer + TMEM owner, warps 2-9 two softmax groups that
// alternate over the two accumulator stages. Every wait on an mbarrier is bounded by wall time; when one runs out
// the CTA records TA_ERR_TIMEOUT, stops waiting anywhere, drains its copies, frees its tensor memory and returns.
#include <cuda.h>

#include "ta_internal.cuh"

namespace {

constexpr int kTileN = 128;                       // keys per tile
constexpr int kD = TA_HEAD_DIM;                   // 128
constexpr int kHalfBytes = kTileN * 128;          // one 64-column half of a 128-row operand tile: 16 KB
constexpr int kKTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr int kStages = 4;                        // shared-memory ring of key tiles
constexpr int kMaxCluster = 8;
constexpr int kThreads = 320;
constexpr int kSoftmaxThreads = 256;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s

struct ScoreParams {
  ta_seq_desc seq;
  int n_layers, Hq, Hkv, G, W;
  int rows;           // G*W
  int cluster;        // CTAs per unit
  int two_pass;       // 0 when lse_obs is given
  int causal;
  float c;            // softmax scale * log2(e)
  float alpha, delta;
  const float* lse_obs;
  const float* u_static;
  float* A;
  float* P;
  float* u;
  ta_dev_status* status;
  float wrow[TA_MAX_WINDOW];  // pension weight of window row t (for W' = W; shorter sequences are handled in-kernel)
  float rho;
};

// ---------------------------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait. Returns false (and raises the CTA's abort flag) when the limit is reached or another thread of the
// CTA already gave up.
__device__ __noinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                       ta_dev_status* status, int where) {
  if (*abort_flag) return false;
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it)
      if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (globaltimer_ns() - t0 > kWaitLimitNs) {
      *abort_flag = 1;
      if (atomicCAS(&status->code, 0, (int)TA_ERR_TIMEOUT) == 0) {
        status->where = where;
        status->detail0 = (int)blockIdx.x;
        status->detail1 = (int)parity;
      }
      return false;
    }
  }
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], "
      "[%2];" ::"r"(dst),
      "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(tmem_d),
      "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (quadrant base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int j = 0; j < 32; ++j) v[j] = __uint_as_float(r[j]);
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t local_addr, uint32_t rank, float v) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}
__device__ __forceinline__ void softmax_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Shared-memory matrix descriptor for a K-major operand tile stored as rows of 128 bytes with the 128-byte swizzle
// (what a TMA box of 64 bf16 x rows with CU_TENSOR_MAP_SWIZZLE_128B writes): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address
  d |= (uint64_t)0 << 16;                         // leading byte offset: unused for swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of sm_100
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}

// Instruction descriptor for kind::f16: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t idesc_bf16(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ---------------------------------------------------------------------------------------------- shared memory
template <int MB>
struct alignas(1024) ScoreSmem {
  uint8_t q[MB * 2 * kHalfBytes];         // [half][MB*128 rows][128 B]
  uint8_t k[kStages][kKTileBytes];        // [stage][half][128 rows][128 B]
  float xchg_m[kMaxCluster][MB * 128];    // per-CTA row statistics of every CTA of the cluster
  float xchg_z[kMaxCluster][MB * 128];
  float part_m[2][MB * 128];              // per softmax group
  float part_z[2][MB * 128];
  float lse2[MB * 128];                   // log2-domain log-sum-exp per row (+inf: row contributes nothing)
  float wrow[MB * 128];                   // pension weight per row
  int lim[MB * 128];                      // last key a row may see (-1: none)
  unsigned long long full[kStages], empty[kStages], acc_full[2], acc_empty[2], q_full, drain;
  uint32_t tmem_base;
  int abort_flag;
};

// ---------------------------------------------------------------------------------------------- the kernel
template <int MB, bool kNeedP>
__global__ void __launch_bounds__(kThreads, 1)
ta_score_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ ScoreParams p) {
  extern __shared__ uint8_t smem_raw[];
  ScoreSmem<MB>& sm = *reinterpret_cast<ScoreSmem<MB>*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int unit = blockIdx.x / p.cluster;
  const int g = unit % p.Hkv;
  const int b = (unit / p.Hkv) % p.seq.batch;
  const int l = unit / (p.Hkv * p.seq.batch);
  const int tok0 = ta_seq_begin(p.seq, b);
  int n = (p.seq.cu ? p.seq.cu[b + 1] : tok0 + p.seq.n_uniform) - tok0;
  if (n > p.seq.max_n || n < 0) {  // reported by the selection step as well; here: just do nothing harmful
    if (tid == 0 && atomicCAS(&p.status->code, 0, (int)TA_ERR_DEVICE_BOUNDS) == 0) {
      p.status->where = 2;
      p.status->detail0 = b;
      p.status->detail1 = n;
    }
    n = 0;
  }
  const int Wp = min(p.W, n);
  const int tiles_total = (n + kTileN - 1) / kTileN;
  const int t_begin = (int)((long long)tiles_total * rank / p.cluster);
  const int t_end = (int)((long long)tiles_total * (rank + 1) / p.cluster);
  const int T = t_end - t_begin;
  const int n_jobs = p.two_pass ? 2 * T : T;
  volatile int* abort_flag = &sm.abort_flag;
  constexpr uint32_t kTmemCols = MB * 256;
  constexpr int kRowsPad = MB * 128;

  // ---- set-up
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sm.full[s]), 1);
      mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sm.acc_full[a]), 1);
      mbar_init(smem_u32(&sm.acc_empty[a]), 4);
    }
    mbar_init(smem_u32(&sm.q_full), 1);
    mbar_init(smem_u32(&sm.drain), 1);
    // a wait that ran out in an earlier CTA or call (not yet polled) makes the remaining CTAs skip their waits
    sm.abort_flag = (*reinterpret_cast<volatile int*>(&p.status->code) == (int)TA_ERR_TIMEOUT) ? 1 : 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sm.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  // per-row tables: last visible key and pension weight. Row r = h*W + t; its query sits at position n - W + t.
  for (int r = tid; r < kRowsPad; r += kThreads) {
    int lim = -1;
    float w = 0.0f;
    if (r < p.rows) {
      const int t = r % p.W;
      const int pos = n - p.W + t;
      if (pos >= 0) {
        lim = p.causal ? pos : n - 1;
        // weight (1-rho) rho^(W'-1-t') with t' = t - (W - W'): the exponent is W-1-t for every valid row
        w = p.wrow[t];
      }
    }
    sm.lim[r] = lim;
    sm.wrow[r] = w;
    if (!p.two_pass) {
      float lse2 = INFINITY;
      if (lim >= 0) {
        const int h = r / p.W, t = r % p.W;
        const float lse = p.lse_obs[(((long long)l * p.seq.batch + b) * p.Hq + (g * p.G + h)) * p.W + t];
        lse2 = lse * 1.4426950408889634f;
      }
      sm.lse2[r] = lse2;
    }
  }
  // Rows of the query tile that the TMA box does not cover are multiplied like any other row: make them zeros so
  // that the padded score columns are finite.
  if (p.rows < kRowsPad) {
    const int pad_rows = kRowsPad - p.rows;
    for (int i = tid; i < 2 * pad_rows * 8; i += kThreads) {
      const int half = i / (pad_rows * 8), rem = i % (pad_rows * 8);
      const int row = p.rows + rem / 8, chunk = rem % 8;
      *reinterpret_cast<uint4*>(&sm.q[half * (MB * kHalfBytes) + row * 128 + chunk * 16]) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sm.tmem_base;
  // every CTA of the cluster must be running before any of them writes into a peer's shared memory
  cluster_arrive();
  cluster_wait();

  const uint32_t q_smem = smem_u32(sm.q);
  const uint32_t k_smem = smem_u32(sm.k);
  const int row_coord_base = p.seq.cu ? tok0 : 0;  // ragged: tokens are packed along the row axis
  const int b_coord = p.seq.cu ? 0 : b;

  if (warp == 0) {
    // =========================================================================== TMA producer
    int issued[kStages];
#pragma unroll
    for (int s = 0; s < kStages; ++s) issued[s] = 0;
    auto issue = [&](int j) {
      const int s = j % kStages;
      const uint32_t ph = (uint32_t)(j / kStages) & 1u;
      mbar_wait(smem_u32(&sm.empty[s]), ph ^ 1u, abort_flag, p.status, 10);
      const int tile = t_begin + (p.two_pass ? j % T : j);
      const uint32_t bar = smem_u32(&sm.full[s]);
      mbar_expect_tx(bar, kKTileBytes);
      const uint32_t dst = k_smem + s * kKTileBytes;
      tma_load_5d(dst, &map_k, bar, 0, row_coord_base + tile * kTileN, g, b_coord, l);
      tma_load_5d(dst + kHalfBytes, &map_k, bar, 64, row_coord_base + tile * kTileN, g, b_coord, l);
      issued[s] = j + 1;
    };
    if (lane == 0 && T > 0) {
      const uint32_t bar = smem_u32(&sm.q_full);
      mbar_expect_tx(bar, (uint32_t)(2 * p.rows * 128));
      tma_load_5d(q_smem, &map_q, bar, 0, 0, g * p.G, b, l);
      tma_load_5d(q_smem + MB * kHalfBytes, &map_q, bar, 64, 0, g * p.G, b, l);
      if (p.two_pass)
        for (int j = 0; j < T; ++j) issue(j);
    }
    __syncwarp();
    cluster_arrive();
    if (lane == 0 && T > 0) {
      for (int j = p.two_pass ? T : 0; j < n_jobs; ++j) issue(j);
      if (*abort_flag) {  // drain: every armed stage must have landed before the CTA may leave
        for (int s = 0; s < kStages; ++s) {
          if (!issued[s]) continue;
          const uint32_t ph = (uint32_t)((issued[s] - 1) / kStages) & 1u;
          const unsigned long long t0 = globaltimer_ns();
          while (!mbar_try_wait(smem_u32(&sm.full[s]), ph) && globaltimer_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
    __syncwarp();
    cluster_wait();
  } else if (warp == 1) {
    // =========================================================================== MMA issuer
    auto issue = [&](int j) {
      const int s = j % kStages;
      const uint32_t ph = (uint32_t)(j / kStages) & 1u;
      const int a = j & 1;
      const uint32_t aph = (uint32_t)(j >> 1) & 1u;
      const bool stats = p.two_pass && j < T;
      mbar_wait(smem_u32(&sm.full[s]), ph, abort_flag, p.status, 20);
      mbar_wait(smem_u32(&sm.acc_empty[a]), aph ^ 1u, abort_flag, p.status, 21);
      tc_fence_after();
      const uint32_t kt = k_smem + s * kKTileBytes;
      const uint32_t acc = tmem_base + (uint32_t)(a * kRowsPad);
      if (stats) {
        const uint32_t idesc = idesc_bf16(128, kTileN);
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint32_t off = (uint32_t)(k & 3) * 32u;
            const uint64_t da = smem_desc_sw128(q_smem + (k >> 2) * (MB * kHalfBytes) + mb * kHalfBytes + off);
            const uint64_t db = smem_desc_sw128(kt + (k >> 2) * kHalfBytes + off);
            umma_bf16(acc + mb * 128, da, db, idesc, k > 0);
          }
        }
      } else {
        const uint32_t idesc = idesc_bf16(128, kRowsPad);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const uint32_t off = (uint32_t)(k & 3) * 32u;
          const uint64_t da = smem_desc_sw128(kt + (k >> 2) * kHalfBytes + off);
          const uint64_t db = smem_desc_sw128(q_smem + (k >> 2) * (MB * kHalfBytes) + off);
          umma_bf16(acc, da, db, idesc, k > 0);
        }
      }
      umma_commit(smem_u32(&sm.empty[s]));
      umma_commit(smem_u32(&sm.acc_full[a]));
    };
    if (lane == 0 && T > 0) {
      mbar_wait(smem_u32(&sm.q_full), 0, abort_flag, p.status, 22);
      if (p.two_pass)
        for (int j = 0; j < T; ++j) issue(j);
    }
    __syncwarp();
    cluster_arrive();
    if (lane == 0 && T > 0) {
      for (int j = p.two_pass ? T : 0; j < n_jobs; ++j) issue(j);
      if (*abort_flag) {  // make sure no MMA is still writing tensor memory before it is freed
        umma_commit(smem_u32(&sm.drain));
        const unsigned long long t0 = globaltimer_ns();
        while (!mbar_try_wait(smem_u32(&sm.drain), 0) && globaltimer_ns() - t0 < kWaitLimitNs) {
        }
      }
    }
    __syncwarp();
    cluster_wait();
  } else {
    // =========================================================================== softmax warps
    const int st = tid - 64;              // 0..255
    const int grp = st >> 7;              // accumulator stage this group serves
    const int quad = warp & 3;            // TMEM lane quadrant this warp may read
    const int row_in_tile = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const float c = p.c;

    // ---- pass 1: running max / sum of exponentials for rows row_in_tile (+128 when MB == 2)
    float m_run[MB], z_run[MB];
    int lim_row[MB];
#pragma unroll
    for (int mb = 0; mb < MB; ++mb) {
      m_run[mb] = -INFINITY;
      z_run[mb] = 0.0f;
      lim_row[mb] = sm.lim[mb * 128 + row_in_tile];
    }
    if (p.two_pass) {
      for (int j = grp; j < T; j += 2) {
        const uint32_t aph = (uint32_t)(j >> 1) & 1u;
        mbar_wait(smem_u32(&sm.acc_full[grp]), aph, abort_flag, p.status, 30);
        tc_fence_after();
        const int key0 = (t_begin + j) * kTileN;
#pragma unroll
        for (int mb = 0; mb < MB; ++mb) {
          const int lim = lim_row[mb];
          const bool skip = __all_sync(0xffffffffu, lim < 0);
          const bool full = __all_sync(0xffffffffu, key0 + kTileN - 1 <= lim);
#pragma unroll 1
          for (int ch = 0; ch < 4; ++ch) {
            float v[32];
            tmem_ld32(tmem_base + lane_addr + (uint32_t)(grp * kRowsPad + mb * 128 + ch * 32), v);
            if (mb == MB - 1 && ch == 3) {  // all of this job's accumulator is in registers: hand the stage back
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&sm.acc_empty[grp]));
            }
            if (skip) continue;
            if (!full) {
              const int kbase = key0 + ch * 32;
#pragma unroll
              for (int q = 0; q < 32; ++q)
                if (kbase + q > lim) v[q] = -INFINITY;
            }
            float cmax = v[0];
#pragma unroll
            for (int q = 1; q < 32; ++q) cmax = fmaxf(cmax, v[q]);
            const float m_new = fmaxf(m_run[mb], cmax);
            if (m_new > -INFINITY) {
              const float mc = m_new * c;
              float acc = z_run[mb] * ex2(m_run[mb] * c - mc);
#pragma unroll
              for (int q = 0; q < 32; ++q) acc += ex2(fmaf(v[q], c, -mc));
              z_run[mb] = acc;
              m_run[mb] = m_new;
            }
          }
        }
      }
      // ---- exchange: group partials -> CTA partial -> every CTA of the cluster
#pragma unroll
      for (int mb = 0; mb < MB; ++mb) {
        sm.part_m[grp][mb * 128 + row_in_tile] = m_run[mb];
        sm.part_z[grp][mb * 128 + row_in_tile] = z_run[mb];
      }
      softmax_bar();
      if (st < kRowsPad) {
        const float m0 = sm.part_m[0][st], m1 = sm.part_m[1][st];
        const float m = fmaxf(m0, m1);
        float z = 0.0f;
        if (m > -INFINITY) z = sm.part_z[0][st] * ex2((m0 - m) * c) + sm.part_z[1][st] * ex2((m1 - m) * c);
        for (int r = 0; r < p.cluster; ++r) {
          st_cluster_f32(smem_u32(&sm.xchg_m[rank][st]), (uint32_t)r, m);
          st_cluster_f32(smem_u32(&sm.xchg_z[rank][st]), (uint32_t)r, z);
        }
      }
    }
    cluster_arrive();
    cluster_wait();
    if (p.two_pass) {
      if (st < kRowsPad) {
        float m = -INFINITY;
        for (int r = 0; r < p.cluster; ++r) m = fmaxf(m, sm.xchg_m[r][st]);
        float z = 0.0f;
        if (m > -INFINITY)
          for (int r = 0; r < p.cluster; ++r) z += sm.xchg_z[r][st] * ex2((sm.xchg_m[r][st] - m) * c);
        sm.lse2[st] = (z > 0.0f) ? m * c + log2f(z) : INFINITY;
      }
      softmax_bar();
    }

    // ---- pass 2: column sums for key row_in_tile of each tile
    const int min_lim = p.causal ? n - Wp : n - 1;  // every valid row sees keys up to here
    const int j0 = p.two_pass ? T : 0;
    const int first = j0 + (((j0 & 1) == grp) ? 0 : 1);
    const long long unit_off = ((long long)l * p.Hkv + g) * p.seq.total;
    for (int j = first; j < n_jobs; j += 2) {
      const uint32_t aph = (uint32_t)(j >> 1) & 1u;
      mbar_wait(smem_u32(&sm.acc_full[grp]), aph, abort_flag, p.status, 31);
      tc_fence_after();
      const int key = (t_begin + (j - j0)) * kTileN + row_in_tile;
      const bool fast_path = __all_sync(0xffffffffu, key <= min_lim || key >= n);
      float sumA = 0.0f, sumP = 0.0f;
      const int n_chunks = (p.rows + 31) >> 5;
#pragma unroll 1
      for (int ch = 0; ch < n_chunks; ++ch) {
        float v[32];
        tmem_ld32(tmem_base + lane_addr + (uint32_t)(grp * kRowsPad + ch * 32), v);
        if (ch == n_chunks - 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&sm.acc_empty[grp]));
        }
        const float4* l4 = reinterpret_cast<const float4*>(&sm.lse2[ch * 32]);
        const float4* w4 = reinterpret_cast<const float4*>(&sm.wrow[ch * 32]);
        if (fast_path) {
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const float4 ls = l4[q];
            const float a0 = ex2(fmaf(v[4 * q + 0], c, -ls.x));
            const float a1 = ex2(fmaf(v[4 * q + 1], c, -ls.y));
            const float a2 = ex2(fmaf(v[4 * q + 2], c, -ls.z));
            const float a3 = ex2(fmaf(v[4 * q + 3], c, -ls.w));
            sumA += (a0 + a1) + (a2 + a3);
            if (kNeedP) {
              const float4 ws = w4[q];
              sumP = fmaf(ws.x, a0, sumP);
              sumP = fmaf(ws.y, a1, sumP);
              sumP = fmaf(ws.z, a2, sumP);
              sumP = fmaf(ws.w, a3, sumP);
            }
          }
        } else {
#pragma unroll
          for (int q = 0; q < 32; ++q) {
            const int r = ch * 32 + q;
            float a = 0.0f;
            if (key <= sm.lim[r]) a = ex2(fmaf(v[q], c, -sm.lse2[r]));
            sumA += a;
            if (kNeedP) sumP = fmaf(sm.wrow[r], a, sumP);
          }
        }
      }
      if (key < n) {
        const long long o = unit_off + tok0 + key;
        if (p.A) p.A[o] = sumA;
        if (p.P) p.P[o] = sumP;
        if (p.u) {
          const float t = __fadd_rn(__fmul_rn(p.alpha, sumA), __fmul_rn(p.delta, sumP));
          p.u[o] = __fadd_rn(t, p.u_static[tok0 + key]);
        }
      }
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int MB>
size_t score_smem_bytes() {
  return sizeof(ScoreSmem<MB>) + 1024;
}

CUresult encode_5d(void* fn, CUtensorMap* map, const void* base, const uint64_t dims[5], const uint64_t strides_el[4],
                   const uint32_t box[5]) {
  auto enc = reinterpret_cast<CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                           const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                           CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                           CUtensorMapFloatOOBfill)>(fn);
  cuuint64_t gdim[5], gstr[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < 5; ++i) {
    gdim[i] = dims[i];
    bx[i] = box[i];
    es[i] = 1;
  }
  for (int i = 0; i < 4; ++i) gstr[i] = strides_el[i] * 2;  // bytes
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), gdim, gstr, bx, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

template <int MB, bool NP>
cudaError_t launch_variant(const CUtensorMap& mq, const CUtensorMap& mk, const ScoreParams& sp, int units,
                           cudaStream_t stream) {
  auto kern = ta_score_kernel<MB, NP>;
  const size_t smem = score_smem_bytes<MB>();
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(units * sp.cluster), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)sp.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, mq, mk, sp);
}

}  // namespace

// A stride that multiplies a coordinate which is always 0 still has to be a valid tensor-map stride.
static uint64_t safe_stride(int64_t s, uint64_t dim) { return (dim <= 1 || s <= 0) ? 128 : (uint64_t)s; }

cudaError_t ta_launch_score(ta_ctx* ctx, const ta_score_args& a, ta_dev_status* status, cudaStream_t stream) {
  const int B = a.seq.batch, L = a.n_layers;
  const int units = L * B * a.Hkv;
  if (units == 0 || a.seq.total == 0) return cudaSuccess;
  const int G = a.Hq / a.Hkv;
  const int rows = G * a.W;
  const int MB = rows <= 128 ? 1 : 2;

  ScoreParams sp = {};
  sp.seq = a.seq;
  sp.n_layers = L;
  sp.Hq = a.Hq;
  sp.Hkv = a.Hkv;
  sp.G = G;
  sp.W = a.W;
  sp.rows = rows;
  sp.two_pass = a.lse_obs ? 0 : 1;
  sp.causal = a.causal;
  const float scale = a.scale > 0.0f ? a.scale : 1.0f / sqrtf((float)kD);
  sp.c = scale * 1.4426950408889634f;
  sp.alpha = a.alpha;
  sp.delta = a.delta;
  sp.lse_obs = a.lse_obs;
  sp.u_static = a.u_static;
  sp.A = a.A;
  sp.P = a.P;
  sp.u = a.u;
  sp.status = status;
  sp.rho = a.rho;
  for (int t = 0; t < a.W; ++t) sp.wrow[t] = (float)((1.0 - (double)a.rho) * pow((double)a.rho, (double)(a.W - 1 - t)));
  const int tiles_max = (a.seq.max_n + kTileN - 1) / kTileN;
  sp.cluster = tiles_max >= 32 ? 8 : tiles_max >= 16 ? 4 : tiles_max >= 8 ? 2 : 1;

  // tensor maps: dims (d, position, head, batch, layer)
  CUtensorMap mq, mk;
  {
    const uint64_t dims[5] = {(uint64_t)kD, (uint64_t)a.W, (uint64_t)a.Hq, (uint64_t)B, (uint64_t)L};
    const uint64_t str[4] = {safe_stride(a.q.stride_n, dims[1]), safe_stride(a.q.stride_h, dims[2]),
                             safe_stride(a.q.stride_b, dims[3]), safe_stride(a.q.stride_l, dims[4])};
    const uint32_t box[5] = {64, (uint32_t)a.W, (uint32_t)G, 1, 1};
    if (encode_5d(ctx->encode_tiled, &mq, a.q.ptr, dims, str, box) != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  {
    const bool ragged = a.seq.cu != nullptr;
    const uint64_t dims[5] = {(uint64_t)kD, ragged ? (uint64_t)a.seq.total : (uint64_t)a.seq.n_uniform,
                              (uint64_t)a.Hkv, ragged ? 1ull : (uint64_t)B, (uint64_t)L};
    const uint64_t str[4] = {safe_stride(a.k.stride_n, dims[1]), safe_stride(a.k.stride_h, dims[2]),
                             safe_stride(a.k.stride_b, dims[3]), safe_stride(a.k.stride_l, dims[4])};
    const uint32_t box[5] = {64, (uint32_t)kTileN, 1, 1, 1};
    if (encode_5d(ctx->encode_tiled, &mk, a.k.ptr, dims, str, box) != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  const bool need_p = a.P != nullptr || (a.u != nullptr && a.delta != 0.0f);
  if (MB == 1) return need_p ? launch_variant<1, true>(mq, mk, sp, units, stream)
                             : launch_variant<1, false>(mq, mk, sp, units, stream);
  return need_p ? launch_variant<2, true>(mq, mk, sp, units, stream)
                : launch_variant<2, false>(mq, mk, sp, units, stream);
}
