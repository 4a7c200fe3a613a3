// Step 2 of the retention path: the attention terms of Eq. 1 (A_i, the pension P_i) over the observation window,
// optionally fused with their weights alpha and delta. sm_100a only: TMA tile loads, tcgen05 tensor-core MMAs with the
// accumulators in tensor memory, and a thread-block cluster per unit for the softmax statistics.
//
// For unit (l, b, g) the score matrix is S = Q_obs[heads of g] * K^T, M = G*W rows (<= 256) by n keys. Each row is
// softmax-normalised over the keys it may see and the result is summed over rows per key. The normaliser of a row
// needs every key before any column sum can be finished, so the keys are swept twice:
//   pass 1  S = Q * Ktile^T   (TMEM lane = query row)  -> reference and sum of exponentials per row
//   pass 2  S^T = Ktile * Q^T (TMEM lane = key)        -> sum over rows of exp2(s*c - beta_row) per key
// Both passes use the same shared-memory operand tiles (both K-major, 128-byte swizzle); only the roles in the
// instruction descriptor swap, which puts the reduction axis of each pass along a thread's own registers.
// A unit is handled by a cluster of 1, 2, 4 or 8 CTAs (chosen per launch: one CTA when there are many units, more when
// there are few); each CTA owns a contiguous range of 128-key tiles. Between the passes every CTA publishes its
// per-row (reference, sum) pairs in its own shared memory, signals its peers with a remote mbarrier arrive, and reads
// the peers' pairs with distributed-shared-memory loads. Pass 2 walks the CTA's tiles backwards so that the tiles read
// last are re-read first from L2. When the caller supplies the rows' log-sum-exp (lse_obs), pass 1 is skipped.
//
// The grid is persistent: as many clusters as the device can hold at once, each walking over units
// cluster, cluster + n_clusters, ...; the TMA and MMA warps run ahead across pass and unit boundaries (double-buffered
// query tile, ring of key tiles, one accumulator stage per softmax group or pair of groups), so barrier set-up, TMEM
// allocation and pipeline fill are paid once per CTA and not once per unit.
//
// Warp roles: four softmax warpgroups plus one warpgroup with the TMA producer warp, the MMA issuer warp (TMEM owner)
// and two idle warps. A "job" is one block of up to 128 score rows of one key tile in one pass. With up to 128 score rows (MB 1) the four groups take the
// jobs round-robin, one accumulator stage of 128 columns each. With 129..256 rows (MB 2) every tile is two jobs, one
// per block of 128 rows, again one group and one stage each: in pass 1 a group owns the rows of its block, in pass 2
// it sums its block's rows for the tile's keys and the two partial sums meet in a small shared-memory ring.
// After set-up the last warpgroup gives registers back (setmaxnreg) and the softmax warpgroups take them.
//
// The softmax warps are bound by instruction issue and by the special-function unit (one ex2 per score element and
// pass), so a fixed share of the exponentials (2 of every 16 with 256 score rows) is evaluated on the FMA pipe instead: the argument is
// clamped to [-126, 126] with a saturating multiply-add, split into integer and fraction with the 1.5*2^23 rounding
// trick, 2^fraction comes from a cubic polynomial (relative error 7.5e-5) and the integer part goes into the exponent
// field with an integer add. The other exponentials take their scale-and-shift and their running sums two at a time
// (fma.rn.f32x2, add.rn.f32x2: the same roundings as the scalar forms, a third fewer issue slots per element).
//
// Every wait on an mbarrier is bounded by wall time; when one runs out the CTA records TA_ERR_TIMEOUT, its producer
// and MMA warps stop issuing work, the copies and MMAs in flight are drained, and the softmax warps finish their loops
// without waiting or storing. The only unbounded waits are hardware barriers that every thread reaches on every path.
#include <cuda.h>

#include <type_traits>

#include "ta_internal.cuh"
#include "ta_sm100.cuh"

namespace {

using namespace ta_sm100;

constexpr int kTileN = 128;                       // keys per tile
constexpr int kD = TA_HEAD_DIM;                   // 128
constexpr int kHalfBytes = kTileN * 128;          // one 64-column half of a 128-row operand tile: 16 KB
constexpr int kKTileBytes = 2 * kHalfBytes;       // 32 KB
constexpr int kMaxCluster = 8;
constexpr int kGroups = 4;                        // softmax warpgroups
constexpr int kThreads = (kGroups + 1) * 128;     // 640
// Register split after set-up (setmaxnreg); the shares must fit in threads x registers at launch:
// 640 threads x 96 = 61440 = 16*32*112 + 4*32*32
constexpr int kRegsSoftmax = 112;
constexpr int kRegsOther = 32;
constexpr int kRegsNeeded = (kGroups * 4 * kRegsSoftmax + 4 * kRegsOther) * 32;

// Of every 16 exponentials, this many run on the FMA pipe. Measured on B200: with up to 128 score rows the softmax
// warps are not what limits the kernel (replacing every ex2 by a multiply changes its duration by 3 %) and any
// polynomial share costs issue slots (0: 119 us, 4: 129 us on 32 layers x 4096 tokens); with 256 rows the
// special-function unit is the longest pole and 2 of 16 is the best share (1.69 -> 1.62 ms on 2 layers of 16 x 32768).
#ifndef TA_SCORE_POLY_MB1
#define TA_SCORE_POLY_MB1 0
#endif
#ifndef TA_SCORE_POLY_MB2
#define TA_SCORE_POLY_MB2 2
#endif

// how pass 2 turns the exponentials of a key into outputs
constexpr int kOutA = 0;      // A only
constexpr int kOutAP = 3;     // A and P (per-row pension weights), or their weighted sum
constexpr int kOutFused = 4;  // alpha*A + delta*P with the positive row weights folded into the exponent

struct ScoreParams {
  ta_seq_desc seq;
  int n_layers, Hq, Hkv, G, W;
  int rows;           // G*W
  int cluster;        // CTAs per unit
  int units;          // L * B * Hkv
  int two_pass;       // 0 when lse_obs is given
  int causal;
  float c;            // softmax scale * log2(e)
  float alpha, delta;
  const float* lse_obs;
  const int32_t* order;  // nullable: the clusters walk units order[0], order[1], .. (longest sequences first)
  float* A;
  float* P;
  float* u;
  ta_dev_status* status;
  unsigned long long wait_limit_ns;
  float wrow[TA_MAX_WINDOW];  // pension weight of window row t (for W' = W; shorter sequences are handled in-kernel)
};

// ---------------------------------------------------------------------------------------------- shared memory
template <int MB>
struct ScoreCfg {
  static constexpr int kQBufs = MB == 1 ? 2 : 1;   // query tiles in flight (next unit's tile loads early)
  static constexpr int kStages = MB == 1 ? 4 : 3;  // ring of key tiles
  static constexpr int kRowsPad = MB * 128;
  static constexpr int kAcc = 4;                   // accumulator stages of 128 columns (512 columns in all)
  static constexpr int kWarpsPerJob = 4;           // softmax warps that read one accumulator stage
  static constexpr int kRing = 4;                  // MB 2: partial sums in flight between the two groups of a pair
};

template <int MB>
struct alignas(1024) ScoreSmem {
  using Cfg = ScoreCfg<MB>;
  uint8_t q[Cfg::kQBufs][MB * 2 * kHalfBytes];    // [buffer][half][MB*128 rows][128 B]
  uint8_t k[Cfg::kStages][kKTileBytes];           // [stage][half][128 rows][128 B]
  float mine_m[2][MB * 128];                      // [unit parity][row]: this CTA's row statistics, read by its peers
  float mine_z[2][MB * 128];
  float part_m[kGroups][128];                     // per softmax group: MB 1 rows 0..127; MB 2 rows of block (group & 1)
  float part_z[kGroups][128];
  float tab[2][MB * 128];                         // [unit parity][row] pass-2 constant of the row (see row constants)
  float nbeta[2][MB * 128];                       // [unit parity][row] -beta (masked tiles use ex2 for every row)
  float wrow[MB * 128];                           // pension weight per row
  float lv[MB * 128];                             // log2 of the row's output weight (kOutFused), else 0
  float psum[2][Cfg::kRing][2][128];              // MB 2: [pair][ring slot][A|P][key] partial sums of row block 0
  int row_t[MB * 128];                            // window index t of the row, -1 for padding rows
  unsigned long long full[Cfg::kStages], empty[Cfg::kStages], acc_full[Cfg::kAcc], acc_empty[Cfg::kAcc];
  unsigned long long q_full[Cfg::kQBufs], q_empty[Cfg::kQBufs], xchg_full[2], drain;
  unsigned long long pfull[2][Cfg::kRing], pfree[2][Cfg::kRing];
  uint32_t tmem_base;
  int abort_flag;
};

struct UnitInfo {
  int l, b, g, tok0, n, t_begin, T;
};

// ---------------------------------------------------------------------------------------------- exponentials
// Position q of a 16-element group runs on the FMA pipe when this is true (the positions are spread evenly).
template <int MB>
__host__ __device__ constexpr bool poly_slot(int q) {
  constexpr int kPoly = MB == 1 ? TA_SCORE_POLY_MB1 : TA_SCORE_POLY_MB2;
  return ((q * kPoly) / 16) != (((q + 1) * kPoly) / 16);
}

constexpr float kPolyRange = 252.0f;                // width of the clamped argument range [-126, 126]
constexpr float kPolyMagic = 12582912.0f - 126.0f;  // 1.5 * 2^23 - 126: adding it leaves the integer part in the low bits
// minimax cubic for 2^f on [0, 1) in relative error (7.5e-5)
constexpr float kC0 = 0.9999251961708069f, kC1 = 0.6958335638046265f, kC2 = 0.22606715559959412f,
                kC3 = 0.07802452147006989f;

__device__ __forceinline__ float fma_sat(float a, float b, float c) {
  float d;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// exp2(x) for x = s*c - beta clamped to [-126, 126], given c252 = c/252 and bias = (126 - beta)/252
__device__ __forceinline__ float exp2_poly(float s, float c252, float bias) {
  const float t = fma_sat(s, c252, bias);                 // (x + 126) / 252 in [0, 1]
  const float y = __fmaf_rd(t, kPolyRange, kPolyMagic);   // 1.5*2^23 + floor(x)
  const float w = kPolyMagic - y;                         // -126 - floor(x), exact
  const float f = fmaf(t, kPolyRange, w);                 // x - floor(x)
  float p = fmaf(kC3, f, kC2);
  p = fmaf(p, f, kC1);
  p = fmaf(p, f, kC0);
  return __int_as_float((__float_as_int(y) << 23) + __float_as_int(p));
}
// two multiply-adds / two adds in one instruction (same roundings as the scalar forms)
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b, float c0, float c1) {
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %6};\n\t"
      "fma.rn.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1)
      : "f"(a0), "f"(a1), "f"(b), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {
  asm("{\n\t.reg .b64 ra, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\tadd.rn.f32x2 rd, rd, ra;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "+f"(d0), "+f"(d1)
      : "f"(a0), "f"(a1));
}
__device__ __forceinline__ float poly_bias(float beta) { return (126.0f - beta) * (1.0f / kPolyRange); }

// ---------------------------------------------------------------------------------------------- the kernel
template <int MB, int PM>
__global__ void __launch_bounds__(kThreads, 1)
ta_score_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ ScoreParams p) {
  using Cfg = ScoreCfg<MB>;
  constexpr int kWarpTma = kGroups * 4, kWarpMma = kGroups * 4 + 1;
  constexpr int kStages = Cfg::kStages, kQBufs = Cfg::kQBufs, kRowsPad = Cfg::kRowsPad;
  constexpr int kAcc = Cfg::kAcc;
  constexpr uint32_t kTmemCols = 512;  // kAcc accumulator stages of 128 columns
  extern __shared__ uint8_t smem_raw[];
  ScoreSmem<MB>& sm = *reinterpret_cast<ScoreSmem<MB>*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const int cluster_id = blockIdx.x / p.cluster;
  const int n_clusters = gridDim.x / p.cluster;
  volatile int* abort_flag = &sm.abort_flag;
  const unsigned long long limit = p.wait_limit_ns;

  // `walk` = cluster_id + round * n_clusters. With a length-sorted order the rounds are taken in alternating
  // direction (the cluster that got the longest unit of one round gets the shortest of the next), which evens out the
  // clusters' totals; a position past the end of the list is an empty unit.
  auto get_unit = [&](int walk) {
    // every cluster makes the same number of rounds; walk positions at and beyond the number of units are empty
    int u = walk;
    bool empty = walk >= p.units;
    if (p.order) {
      const int round = walk / n_clusters;
      const int w = (round & 1) ? round * n_clusters + (n_clusters - 1 - cluster_id) : walk;
      empty = w >= p.units;
      u = empty ? 0 : p.order[w];
    } else if (empty) {
      u = 0;
    }
    UnitInfo ui;
    ui.g = u % p.Hkv;
    ui.b = (u / p.Hkv) % p.seq.batch;
    ui.l = u / (p.Hkv * p.seq.batch);
    ui.tok0 = ta_seq_begin(p.seq, ui.b);
    int n = (p.seq.cu ? p.seq.cu[ui.b + 1] : ui.tok0 + p.seq.n_uniform) - ui.tok0;
    // a sequence that does not lie inside the token arrays is skipped here and rejected by the selection step
    if (n > p.seq.max_n || n < 0 || ui.tok0 < 0 || (long long)ui.tok0 + n > p.seq.total) {
      if (tid == 0 && atomicCAS(&p.status->code, 0, (int)TA_ERR_DEVICE_BOUNDS) == 0) {
        p.status->where = 2;
        p.status->detail0 = ui.b;
        p.status->detail1 = n;
      }
      n = 0;
    }
    if (empty) n = 0;
    ui.n = n;
    const int tiles_total = (n + kTileN - 1) / kTileN;
    ui.t_begin = (int)((long long)tiles_total * rank / p.cluster);
    ui.T = (int)((long long)tiles_total * (rank + 1) / p.cluster) - ui.t_begin;
    return ui;
  };

  // ---- set-up (once per CTA)
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sm.full[s]), 1);
      mbar_init(smem_u32(&sm.empty[s]), 1);
    }
    for (int a = 0; a < kAcc; ++a) {
      mbar_init(smem_u32(&sm.acc_full[a]), 1);
      mbar_init(smem_u32(&sm.acc_empty[a]), Cfg::kWarpsPerJob);
    }
    for (int a = 0; a < 2; ++a) mbar_init(smem_u32(&sm.xchg_full[a]), (uint32_t)p.cluster);
    for (int qb = 0; qb < kQBufs; ++qb) {
      mbar_init(smem_u32(&sm.q_full[qb]), 1);
      mbar_init(smem_u32(&sm.q_empty[qb]), 1);
    }
    mbar_init(smem_u32(&sm.drain), 1);
    for (int pr = 0; pr < 2; ++pr)
      for (int r = 0; r < Cfg::kRing; ++r) {
        mbar_init(smem_u32(&sm.pfull[pr][r]), 4);
        mbar_init(smem_u32(&sm.pfree[pr][r]), 4);
      }
    // a wait that ran out in an earlier CTA or call (not yet polled) makes the remaining CTAs skip their waits
    sm.abort_flag = (*reinterpret_cast<volatile int*>(&p.status->code) == (int)TA_ERR_TIMEOUT) ? 1 : 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) {
    tmem_alloc(smem_u32(&sm.tmem_base), kTmemCols);
    tmem_relinquish();
  }
  // per-row tables: row r = h*W + t
  for (int r = tid; r < kRowsPad; r += kThreads) {
    const int t = r < p.rows ? r % p.W : -1;
    sm.row_t[r] = t;
    const float w = t >= 0 ? p.wrow[t] : 0.0f;  // (1-rho) rho^(W-1-t); also right for W' < W (same exponent)
    sm.wrow[r] = w;
    // kOutFused: the row's contribution alpha + delta*w (positive, checked by the host) goes into the exponent
    sm.lv[r] = (PM == kOutFused && t >= 0) ? log2f(fmaf(p.delta, w, p.alpha)) : 0.0f;
  }
  // Rows of the query tile that the TMA box does not cover are multiplied like any other row: make them zeros so
  // that the padded score columns are finite.
  if (p.rows < kRowsPad) {
    const int pad_rows = kRowsPad - p.rows;
    for (int i = tid; i < kQBufs * 2 * pad_rows * 8; i += kThreads) {
      const int qb = i / (2 * pad_rows * 8), i2 = i % (2 * pad_rows * 8);
      const int half = i2 / (pad_rows * 8), rem = i2 % (pad_rows * 8);
      const int row = p.rows + rem / 8, chunk = rem % 8;
      *reinterpret_cast<uint4*>(&sm.q[qb][half * (MB * kHalfBytes) + row * 128 + chunk * 16]) = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sm.tmem_base;
  // every CTA of the cluster must be running (barriers initialised) before any peer writes into its shared memory
  cluster_arrive();
  cluster_wait();

  const uint32_t k_smem = smem_u32(sm.k);

  if (warp >= kWarpTma) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
    if (warp == kWarpTma) {
      // =========================================================================== TMA producer
      if (lane == 0) {
        int issued[kStages], q_issued[kQBufs];
#pragma unroll
        for (int s = 0; s < kStages; ++s) issued[s] = 0;
#pragma unroll
        for (int s = 0; s < kQBufs; ++s) q_issued[s] = 0;
        int jg = 0, qn = 0;
        bool ok = true;
        for (int u = cluster_id; ok && u - cluster_id < p.units; u += n_clusters) {
          const UnitInfo ui = get_unit(u);
          if (ui.T == 0) continue;
          const int qb = qn % kQBufs;
          ok = mbar_wait(smem_u32(&sm.q_empty[qb]), ((uint32_t)(qn / kQBufs) & 1u) ^ 1u, abort_flag, p.status, 11, limit);
          if (!ok) break;  // nothing may be copied into a buffer that was not handed back
          {
            const uint32_t bar = smem_u32(&sm.q_full[qb]);
            const uint32_t dst = smem_u32(sm.q[qb]);
            mbar_expect_tx(bar, (uint32_t)(2 * p.rows * 128));
            tma_load_5d(dst, &map_q, bar, 0, 0, ui.g * p.G, ui.b, ui.l);
            tma_load_5d(dst + MB * kHalfBytes, &map_q, bar, 64, 0, ui.g * p.G, ui.b, ui.l);
            q_issued[qb] = qn + 1;
          }
          ++qn;
          const int row0 = p.seq.cu ? ui.tok0 : 0;  // ragged: tokens are packed along the row axis
          const int bc = p.seq.cu ? 0 : ui.b;
          const int n_jobs = p.two_pass ? 2 * ui.T : ui.T;
          for (int j = 0; j < n_jobs; ++j, ++jg) {
            const int s = jg % kStages;
            ok = mbar_wait(smem_u32(&sm.empty[s]), ((uint32_t)(jg / kStages) & 1u) ^ 1u, abort_flag, p.status, 10, limit);
            if (!ok) break;
            // the second sweep walks the CTA's tiles backwards: the tiles read last are the ones still in L2
            const int tile = ui.t_begin + (j >= ui.T ? 2 * ui.T - 1 - j : j);
            const uint32_t bar = smem_u32(&sm.full[s]);
            mbar_expect_tx(bar, kKTileBytes);
            const uint32_t dst = k_smem + s * kKTileBytes;
            tma_load_5d(dst, &map_k, bar, 0, row0 + tile * kTileN, ui.g, bc, ui.l);
            tma_load_5d(dst + kHalfBytes, &map_k, bar, 64, row0 + tile * kTileN, ui.g, bc, ui.l);
            issued[s] = jg + 1;
          }
        }
        if (!ok || *abort_flag) {
          // drain: every copy that was started must have landed before the CTA may leave. A stage is only ever armed
          // after its previous contents were handed back, so at most the last copy per stage can still be in flight.
          for (int s = 0; s < kStages; ++s)
            if (issued[s]) mbar_wait_drain(smem_u32(&sm.full[s]), (uint32_t)((issued[s] - 1) / kStages) & 1u, limit);
          for (int s = 0; s < kQBufs; ++s)
            if (q_issued[s]) mbar_wait_drain(smem_u32(&sm.q_full[s]), (uint32_t)((q_issued[s] - 1) / kQBufs) & 1u, limit);
        }
      }
    } else if (warp == kWarpMma) {
      // =========================================================================== MMA issuer
      if (lane == 0) {
        int jg = 0, tg = 0, qn = 0;
        bool ok = true;
        // operand descriptors: the upper word is the same for every tile; the lower word is the address >> 4
        const uint32_t desc_hi = (uint32_t)(smem_desc_sw128(0) >> 32);
        const uint32_t k_lo = (k_smem & 0x3FFFFu) >> 4;
        const uint32_t idesc = idesc_bf16(128, 128);
        for (int u = cluster_id; ok && u - cluster_id < p.units; u += n_clusters) {
          const UnitInfo ui = get_unit(u);
          if (ui.T == 0) continue;
          const int qb = qn % kQBufs;
          ok = mbar_wait(smem_u32(&sm.q_full[qb]), (uint32_t)(qn / kQBufs) & 1u, abort_flag, p.status, 22, limit);
          if (!ok) break;
          const uint32_t q_lo = (smem_u32(sm.q[qb]) & 0x3FFFFu) >> 4;
          // A tile's product is issued as MB jobs, one per block of 128 score rows, each into its own accumulator
          // stage of 128 columns: S = Q_block * Ktile^T in pass 1, S^T = Ktile * Q_block^T in pass 2.
          const int n_tiles = p.two_pass ? 2 * ui.T : ui.T;
          for (int jt = 0; ok && jt < n_tiles; ++jt, ++tg) {
            const int s = tg % kStages;
            const bool stats = p.two_pass && jt < ui.T;
            ok = mbar_wait(smem_u32(&sm.full[s]), (uint32_t)(tg / kStages) & 1u, abort_flag, p.status, 20, limit);
            if (!ok) break;  // no product is issued on operands that are not ready
            const uint32_t dk_lo = k_lo + (uint32_t)((s * kKTileBytes) >> 4);
#pragma unroll
            for (int rb = 0; rb < MB; ++rb, ++jg) {
              const int a = jg % kAcc;
              ok = ok && mbar_wait(smem_u32(&sm.acc_empty[a]), ((uint32_t)(jg / kAcc) & 1u) ^ 1u, abort_flag, p.status,
                                   21, limit);
              if (ok) {  // (nor into an accumulator that was not handed back)
                tc_fence_after();
                const uint32_t acc = tmem_base + (uint32_t)(a * 128);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                  const uint32_t dq = q_lo + (uint32_t)(((k >> 2) * (MB * kHalfBytes) + rb * kHalfBytes + (k & 3) * 32) >> 4);
                  const uint32_t dk = dk_lo + (uint32_t)(((k >> 2) * kHalfBytes + (k & 3) * 32) >> 4);
                  umma_bf16_lo(acc, stats ? dq : dk, stats ? dk : dq, desc_hi, idesc, k > 0);
                }
                if (rb == MB - 1) umma_commit(smem_u32(&sm.empty[s]));
                umma_commit(smem_u32(&sm.acc_full[a]));
              }
            }
          }
          if (!ok) break;
          umma_commit(smem_u32(&sm.q_empty[qb]));  // the query tile may be overwritten once these MMAs are done
          ++qn;
        }
        if (!ok || *abort_flag) {  // make sure no MMA is still writing tensor memory before it is freed
          umma_commit(smem_u32(&sm.drain));
          mbar_wait_drain(smem_u32(&sm.drain), 0, limit);
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
    // =========================================================================== softmax warps
    // A job is one block of 128 score rows of one key tile in one pass; jobs are dealt round-robin to the four
    // groups. With two row blocks (MB 2) a tile is two consecutive jobs, every unit has an even number of jobs, and
    // group g therefore always gets row block g & 1.
    constexpr int kShare = kAcc;
    const int st = tid;                     // 0..511
    const int grp = st >> 7;
    const int slot = grp;                   // serves jobs with (global job index % kShare) == slot
    const int blk = MB == 1 ? 0 : grp & 1;  // the row block of every job this group gets
    const int coff = blk * 128;              // first score row of that block
    const int quad = warp & 3;              // TMEM lane quadrant this warp may read
    const int row_in_tile = quad * 32 + lane;
    const uint32_t tlane = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = p.c;
    const float c252 = c * (1.0f / kPolyRange);
    const int my_t = sm.row_t[coff + row_in_tile];  // pass 1: this thread's row is coff + row_in_tile
    const int rows_mine = min(128, p.rows - coff);
    const int n_chunks2 = (rows_mine + 31) >> 5;

    auto acc_addr = [&](int jj) { return tlane + (uint32_t)((jj % kAcc) * 128); };
    auto wait_full = [&](int jj, int where) {
      mbar_wait(smem_u32(&sm.acc_full[jj % kAcc]), (uint32_t)(jj / kAcc) & 1u, abort_flag, p.status, where, limit);
      tc_fence_after();
    };
    auto release = [&](int jj) {  // the whole accumulator of the job is in registers: hand the stage back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sm.acc_empty[jj % kAcc]));
    };

    int jg = 0, it = 0;
    int pc = 0;  // MB 2: tiles of pass 2 this group has handled (same count in both groups of a pair)
    for (int u = cluster_id; u - cluster_id < p.units; u += n_clusters, ++it) {
      const UnitInfo ui = get_unit(u);
      const int n = ui.n, T = ui.T;
      const int up = it & 1;
      const int Wp = min(p.W, n);

      if (p.two_pass) {
        // ---- pass 1: per row, sum of exp2(s*c - ref) against a reference `ref` that only has to keep the sum inside
        // the fp32 range (the result does not depend on it): the largest of the first 16 keys the row sees. After that
        // a key costs one multiply-add, one exponential and one add, and no maximum is tracked. A tile whose sum
        // leaves the safe range (a score more than 2^60 above ref) is redone against its own maximum. That check must
        // not wait for the tile's last exponentials (the accumulator stage is released right after it, and the next
        // product into the stage waits for the release): it uses the sum without the last 16 keys and, for those,
        // their largest score. The polynomial exponentials saturate at 2^126, which the same check catches.
        float ref_c, z_run = 0.0f, pb;
        const int pos = n - p.W + my_t;
        const int lim = (my_t >= 0 && pos >= 0) ? (p.causal ? pos : n - 1) : -1;
        // rows that see no key (padding) get a reference that turns every exponential into 0
        ref_c = lim >= 0 ? -1e30f : 1e30f;
        pb = poly_bias(ref_c);
        constexpr float kSumLimit = 1.0e18f;  // about 2^60
        // 16 keys of one row: adds exp2(s*c - rc) to the four sums; `mix`: kPoly of them on the FMA pipe;
        // `track`: also the largest s in `mx`. Masked tiles (cold) drop keys beyond `lim`.
        auto half1 = [&](auto masked_tag, auto mix_tag, auto track_tag, const float(&cur)[16], float rc, float pbias,
                         float(&s4)[4], float& mx, int kbase) {
          constexpr bool masked = decltype(masked_tag)::value;
          constexpr bool mix = decltype(mix_tag)::value && !masked;
          constexpr bool track = decltype(track_tag)::value;
          float v[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) v[q] = cur[q];
          if (masked) {
#pragma unroll
            for (int q = 0; q < 16; ++q)
              if (kbase + q > lim) v[q] = -INFINITY;
          }
#pragma unroll
          for (int q = 0; q < 16; q += 2) {
            if (mix && (poly_slot<MB>(q) || poly_slot<MB>(q + 1))) {
#pragma unroll
              for (int e2 = 0; e2 < 2; ++e2) {
                const float e = poly_slot<MB>(q + e2) ? exp2_poly(v[q + e2], c252, pbias) : ex2(fmaf(v[q + e2], c, -rc));
                s4[(q + e2) & 3] += e;
              }
            } else {
              float a0, a1;
              fma2(a0, a1, v[q], v[q + 1], c, -rc, -rc);
              add2(s4[q & 3], s4[(q & 3) + 1], ex2(a0), ex2(a1));
            }
          }
          if (track) {
            float t4[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) t4[q] = fmaxf(fmaxf(v[4 * q], v[4 * q + 1]), fmaxf(v[4 * q + 2], v[4 * q + 3]));
            mx = fmaxf(mx, fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3])));
          }
        };
        // largest of 16 keys of one row
        auto max16 = [&](auto masked_tag, const float(&cur)[16], float& mx, int kbase) {
          constexpr bool masked = decltype(masked_tag)::value;
          float t4[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            float w[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) w[e] = (masked && kbase + 4 * q + e > lim) ? -INFINITY : cur[4 * q + e];
            t4[q] = fmaxf(fmaxf(w[0], w[1]), fmaxf(w[2], w[3]));
          }
          mx = fmaxf(mx, fmaxf(fmaxf(t4[0], t4[1]), fmaxf(t4[2], t4[3])));
        };
        float ra[16], rb[16];
        int j = (slot - jg % kShare + kShare) % kShare;  // first job of this pass that belongs to the group
        if (j < MB * T) {
          wait_full(jg + j, 30);
          tmem_ld16_issue(acc_addr(jg + j), ra);
        }
        // One job: the 128 accumulator columns in 32-column chunks, each fetched as two 16-column loads (ra, rb) so
        // that one load is always in flight. On entry the load of the first 16 columns is in flight in `ra`.
        auto job1 = [&](auto masked_tag, int j) {
          const int jj = jg + j;
          const int key0 = (ui.t_begin + j / MB) * kTileN;
          const uint32_t abase = acc_addr(jj);
          float rc = ref_c;
          const bool first = rc < -1e29f;
          if (__any_sync(0xffffffffu, first)) {  // the row has no reference yet: take it from the 16 keys in flight
            float mx = -INFINITY;
            tmem_ld_wait(ra);
            max16(masked_tag, ra, mx, key0);
            if (first && mx > -INFINITY) {
              rc = mx * c;
              ref_c = rc;
              pb = poly_bias(rc);
            }
          }
          float s4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
          float sum_head = 0.0f, mx_tail = -INFINITY, unused = 0.0f;
#pragma unroll 1
          for (int c4 = 0; c4 < 4; ++c4) {
            const uint32_t col = (uint32_t)(c4 * 32);
            tmem_ld_wait(ra);
            tmem_ld16_issue(abase + col + 16, rb);
            half1(masked_tag, std::true_type{}, std::false_type{}, ra, rc, pb, s4, unused, key0 + c4 * 32);
            tmem_ld_wait(rb);
            if (c4 < 3) {
              tmem_ld16_issue(abase + col + 32, ra);
              half1(masked_tag, std::true_type{}, std::false_type{}, rb, rc, pb, s4, unused, key0 + c4 * 32 + 16);
            } else {
              sum_head = (s4[0] + s4[1]) + (s4[2] + s4[3]);
              half1(masked_tag, std::true_type{}, std::true_type{}, rb, rc, pb, s4, mx_tail, key0 + c4 * 32 + 16);
            }
          }
          float sum = (s4[0] + s4[1]) + (s4[2] + s4[3]);
          // also true for inf and NaN sums
          const bool over = !(sum_head < kSumLimit) || fmaf(mx_tail, c, -rc) > 60.0f;
          if (__any_sync(0xffffffffu, over)) {   // rare: a score far above the reference
            float mx = -INFINITY;
#pragma unroll 1
            for (int h = 0; h < 8; ++h) {
              tmem_ld16_issue(abase + (uint32_t)(h * 16), rb);
              tmem_ld_wait(rb);
              max16(masked_tag, rb, mx, key0 + h * 16);
            }
            const float mx_c = mx * c;
            float r4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll 1
            for (int h = 0; h < 8; ++h) {
              tmem_ld16_issue(abase + (uint32_t)(h * 16), rb);
              tmem_ld_wait(rb);
              half1(masked_tag, std::false_type{}, std::false_type{}, rb, over ? mx_c : rc, 0.0f, r4, unused,
                    key0 + h * 16);
            }
            if (over) {
              z_run *= ex2(rc - mx_c);
              ref_c = mx_c;
              pb = poly_bias(mx_c);
              sum = (r4[0] + r4[1]) + (r4[2] + r4[3]);
            }
          }
          z_run += sum;
          release(jj);
          if (j + kShare < MB * T) {  // the next job of the group reuses this stage: fetch it once it is full again
            wait_full(jj + kShare, 30);
            tmem_ld16_issue(acc_addr(jj + kShare), ra);
          }
        };
        for (; j < MB * T; j += kShare) {
          // tiles that every row of the warp sees completely take the unmasked path (rows that see nothing at all,
          // i.e. padding, still run: their sums are never used)
          const bool masked = lim >= 0 && (ui.t_begin + j / MB) * kTileN + kTileN - 1 > lim;
          if (__any_sync(0xffffffffu, masked)) job1(std::true_type{}, j);
          else job1(std::false_type{}, j);
        }
        // ---- exchange: group partials -> CTA partial -> every CTA of the cluster reads every other's
        // rows that see no key at all (padding, window positions before the sequence start) stay mute
        sm.part_m[grp][row_in_tile] = lim >= 0 ? ref_c : -1e30f;
        sm.part_z[grp][row_in_tile] = lim >= 0 ? z_run : 0.0f;
        softmax_bar<kGroups>();
        float lse2_row = INFINITY;  // log2-domain log-sum-exp of row `st` (+inf: the row is mute)
        if (st < kRowsPad) {
          float m, z = 0.0f;
          if (MB == 1) {
            m = sm.part_m[0][st];
#pragma unroll
            for (int gq = 1; gq < kGroups; ++gq) m = fmaxf(m, sm.part_m[gq][st]);
#pragma unroll
            for (int gq = 0; gq < kGroups; ++gq) z += sm.part_z[gq][st] * ex2(sm.part_m[gq][st] - m);
          } else {  // rows of block h were summed by groups h and h + 2
            const int h = st >> 7, i = st & 127;
            m = fmaxf(sm.part_m[h][i], sm.part_m[h + 2][i]);
            z = sm.part_z[h][i] * ex2(sm.part_m[h][i] - m) + sm.part_z[h + 2][i] * ex2(sm.part_m[h + 2][i] - m);
          }
          if (p.cluster == 1) {  // nothing to exchange: the CTA's statistics are the unit's
            lse2_row = (z > 0.0f) ? m + log2f(z) : INFINITY;
          } else {
            sm.mine_m[up][st] = m;
            sm.mine_z[up][st] = z;
          }
        }
        if (p.cluster > 1) {
          softmax_bar<kGroups>();
          // one thread per peer tells that peer that this CTA's statistics of the unit are in place
          if (st < p.cluster) {
            fence_cluster();
            mbar_arrive_remote(smem_u32(&sm.xchg_full[up]), (uint32_t)st);
          }
          if (st < kRowsPad) {
            mbar_wait_cluster(smem_u32(&sm.xchg_full[up]), (uint32_t)(it >> 1) & 1u, abort_flag, p.status, 32, limit);
            float pm[kMaxCluster], pz[kMaxCluster];
#pragma unroll
            for (int r = 0; r < kMaxCluster; ++r) {
              pm[r] = -1e30f;
              pz[r] = 0.0f;
              if (r < p.cluster) {
                pm[r] = ld_cluster_f32(smem_u32(&sm.mine_m[up][st]), (uint32_t)r);
                pz[r] = ld_cluster_f32(smem_u32(&sm.mine_z[up][st]), (uint32_t)r);
              }
            }
            float m = pm[0];
#pragma unroll
            for (int r = 1; r < kMaxCluster; ++r) m = fmaxf(m, pm[r]);
            float z = 0.0f;
#pragma unroll
            for (int r = 0; r < kMaxCluster; ++r) z += pz[r] * ex2(pm[r] - m);
            lse2_row = (z > 0.0f) ? m + log2f(z) : INFINITY;
          }
        }
        if (st < kRowsPad) {
          const float beta = lse2_row - sm.lv[st];
          sm.nbeta[up][st] = -beta;
          sm.tab[up][st] = poly_slot<MB>(st & 15) ? poly_bias(beta) : -beta;
        }
        softmax_bar<kGroups>();
      } else {
        if (st < kRowsPad) {
          float lse2 = INFINITY;
          const int t = sm.row_t[st];
          if (t >= 0 && n - p.W + t >= 0) {
            const int h = st / p.W;
            const float lse = p.lse_obs[(((long long)ui.l * p.seq.batch + ui.b) * p.Hq + (ui.g * p.G + h)) * p.W + t];
            lse2 = lse * 1.4426950408889634f;
          }
          const float beta = lse2 - sm.lv[st];
          sm.nbeta[up][st] = -beta;
          sm.tab[up][st] = poly_slot<MB>(st & 15) ? poly_bias(beta) : -beta;
        }
        softmax_bar<kGroups>();
      }

      // ---- pass 2: for key row_in_tile of each tile, the sum over this group's rows of exp2(s*c - beta_row)
      const int min_lim = p.causal ? n - Wp : n - 1;  // every valid row sees keys up to here
      const int j0 = p.two_pass ? MB * T : 0;
      const int n_jobs = j0 + MB * T;
      const long long unit_off = ((long long)ui.l * p.Hkv + ui.g) * p.seq.total;
      const float4* tab4 = reinterpret_cast<const float4*>(sm.tab[up] + coff);
      const float4* nb4 = reinterpret_cast<const float4*>(sm.nbeta[up] + coff);
      const float4* w4 = reinterpret_cast<const float4*>(sm.wrow + coff);
      {
        float sA4[4], sP = 0.0f;
        // 16 rows (half `hi` of the 32-row chunk cc) of this thread's key. Hot form: kPoly of the 16 exponentials on
        // the FMA pipe, row constants from `tab`. Masked form (keys inside the observation window, cold tiles only):
        // every exponential on the special-function unit against -beta, rows that do not see the key dropped.
        auto chunk2 = [&](auto masked_tag, auto hi_tag, const float(&cur)[16], int cc, int key) {
          constexpr bool masked = decltype(masked_tag)::value;
          constexpr int hi = decltype(hi_tag)::value;  // 0: rows 32cc..32cc+15, 1: rows 32cc+16..32cc+31
#pragma unroll
          for (int q4 = 0; q4 < 4; ++q4) {
            const float4 tb = masked ? nb4[cc * 8 + hi * 4 + q4] : tab4[cc * 8 + hi * 4 + q4];
            const float tbv[4] = {tb.x, tb.y, tb.z, tb.w};
            float a[4];
#pragma unroll
            for (int e = 0; e < 4; e += 2) {
              if (!masked && (poly_slot<MB>(4 * q4 + e) || poly_slot<MB>(4 * q4 + e + 1))) {
#pragma unroll
                for (int e2 = e; e2 < e + 2; ++e2)
                  a[e2] = poly_slot<MB>(4 * q4 + e2) ? exp2_poly(cur[4 * q4 + e2], c252, tbv[e2])
                                                     : ex2(fmaf(cur[4 * q4 + e2], c, tbv[e2]));
              } else {
                float x0, x1;
                fma2(x0, x1, cur[4 * q4 + e], cur[4 * q4 + e + 1], c, tbv[e], tbv[e + 1]);
                a[e] = ex2(x0);
                a[e + 1] = ex2(x1);
              }
            }
            if (masked) {  // row r sees key i only if i <= the row's own position
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const int t = sm.row_t[coff + cc * 32 + hi * 16 + 4 * q4 + e];
                const int pos = n - p.W + t;
                const int lim = (t >= 0 && pos >= 0) ? (p.causal ? pos : n - 1) : -1;
                if (key > lim) a[e] = 0.0f;
              }
            }
            add2(sA4[0], sA4[1], a[0], a[1]);
            add2(sA4[2], sA4[3], a[2], a[3]);
            if (PM == kOutAP) {
              const float4 ws = w4[cc * 8 + hi * 4 + q4];
              sP = fmaf(ws.x, a[0], sP);
              sP = fmaf(ws.y, a[1], sP);
              sP = fmaf(ws.z, a[2], sP);
              sP = fmaf(ws.w, a[3], sP);
            }
          }
        };
        float ra[16], rb[16];
        int j = j0 + (slot - (jg + j0) % kShare + kShare) % kShare;
        if (j < n_jobs) {
          wait_full(jg + j, 31);
          tmem_ld16_issue(acc_addr(jg + j), ra);
        }
        // one job: 32-row chunks, each as two 16-column loads (ra low half, rb high half)
        auto job2 = [&](auto masked_tag, int j, int key) {
          const int jj = jg + j;
          const uint32_t abase = acc_addr(jj);
#pragma unroll 1
          for (int ci = 0; ci < n_chunks2; ++ci) {
            const uint32_t col = (uint32_t)(ci * 32);
            tmem_ld_wait(ra);
            tmem_ld16_issue(abase + col + 16, rb);
            chunk2(masked_tag, std::integral_constant<int, 0>{}, ra, ci, key);
            tmem_ld_wait(rb);
            if (ci == n_chunks2 - 1) {
              release(jj);
              if (j + kShare < n_jobs) {
                wait_full(jj + kShare, 31);
                tmem_ld16_issue(acc_addr(jj + kShare), ra);
              }
            } else {
              tmem_ld16_issue(abase + col + 32, ra);
            }
            chunk2(masked_tag, std::integral_constant<int, 1>{}, rb, ci, key);
          }
        };
        for (; j < n_jobs; j += kShare) {
          const int tl = (j - j0) / MB;  // the pass walks the CTA's tiles backwards after a first pass
          const int key = (ui.t_begin + (p.two_pass ? T - 1 - tl : tl)) * kTileN + row_in_tile;
          sA4[0] = sA4[1] = sA4[2] = sA4[3] = 0.0f;
          sP = 0.0f;
          // only the last W-1 keys of a sequence are hidden from some rows: those tiles take the masked path
          if (__all_sync(0xffffffffu, key <= min_lim || key >= n)) job2(std::false_type{}, j, key);
          else job2(std::true_type{}, j, key);
          float sA = (sA4[0] + sA4[1]) + (sA4[2] + sA4[3]);
          if (MB == 2) {
            // The two row blocks of a tile are consecutive jobs of two different groups. The group of block 0 leaves
            // its sums in a ring slot and goes on; the group of block 1, which gets its job later, picks them up, adds
            // its own and stores. Neither waits for the other unless the ring is full (block 0 four tiles ahead).
            const int pr = grp >> 1, r = pc % Cfg::kRing;
            const uint32_t ph = (uint32_t)(pc / Cfg::kRing) & 1u;
            ++pc;
            if (blk == 0) {
              mbar_wait(smem_u32(&sm.pfree[pr][r]), ph ^ 1u, abort_flag, p.status, 33, limit);
              sm.psum[pr][r][0][row_in_tile] = sA;
              if (PM == kOutAP) sm.psum[pr][r][1][row_in_tile] = sP;
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&sm.pfull[pr][r]));
            } else {
              mbar_wait(smem_u32(&sm.pfull[pr][r]), ph, abort_flag, p.status, 34, limit);
              sA += sm.psum[pr][r][0][row_in_tile];
              if (PM == kOutAP) sP += sm.psum[pr][r][1][row_in_tile];
              __syncwarp();
              if (lane == 0) mbar_arrive(smem_u32(&sm.pfree[pr][r]));
            }
          }
          if (blk == MB - 1 && key < n && !*abort_flag) {
            const long long o = unit_off + ui.tok0 + key;
            if (PM == kOutFused) {
              p.u[o] = sA;
            } else {
              if (p.A) p.A[o] = sA;
              if (p.P) p.P[o] = sP;
              if (p.u) p.u[o] = __fadd_rn(__fmul_rn(p.alpha, sA), __fmul_rn(p.delta, sP));
            }
          }
        }
      }
      if (T > 0) jg += n_jobs;
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
  // no CTA may leave while a peer can still store into its shared memory or arrive on its barriers
  cluster_arrive();
  cluster_wait();
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

template <int MB, int PM>
cudaError_t launch_variant(ta_ctx* ctx, const CUtensorMap& mq, const CUtensorMap& mk, ScoreParams& sp,
                           int tiles_max, int reserve_sms, cudaStream_t stream) {
  auto kern = ta_score_kernel<MB, PM>;
  const size_t smem = score_smem_bytes<MB>();
  // per context (and so per device) and instantiation: the attribute is sticky, the occupancy does not change
  constexpr int vi = (MB - 1) * 3 + (PM == kOutA ? 0 : PM == kOutAP ? 1 : 2);
  int* max_clusters = ctx->score_max_clusters[vi];
  if (!ctx->score_attr_set[vi]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    // the in-kernel register split must fit in what the launch provides, or the warps asking for more wait forever
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, kern);
    if (e != cudaSuccess) return e;
    if (fa.numRegs * kThreads < kRegsNeeded) return cudaErrorLaunchOutOfResources;
    for (int cl = 0; cl <= kMaxCluster; ++cl) max_clusters[cl] = 0;
    ctx->score_attr_set[vi] = 1;
  }
  cudaLaunchConfig_t cfg = {};
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
  // Persistent grid: as many clusters as can be resident at once (queried once per cluster size). CTAs per unit:
  // the size with the fewest tile-times on the busiest CTA, counting ~1 tile-time of overhead per unit and ~2 more
  // for the statistics exchange when a unit spans several CTAs. (Choosing more CTAs per unit so that the keys of
  // all units in flight fit in L2 was measured and lost: 16 x 32768 tokens, 8 CTAs per unit 2.02 ms against 1.63 ms.)
  int best_cl = ctx->score_force_cluster;
  long long best_cost = best_cl > 0 ? 0 : -1;
  for (int cl = 1; cl <= kMaxCluster; cl *= 2) {
    if (ctx->score_force_cluster > 0 && cl != ctx->score_force_cluster) continue;
    if (cl > 1 && tiles_max < 2 * cl && ctx->score_force_cluster <= 0) break;
    if (max_clusters[cl] == 0) {
      attr[0].val.clusterDim.x = (unsigned)cl;
      cfg.gridDim = dim3((unsigned)(ctx->sm_count / cl * cl), 1, 1);
      int n = 0;
      cudaError_t e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
      if (e != cudaSuccess) return e;
      max_clusters[cl] = n < 1 ? -1 : n;
    }
    if (max_clusters[cl] < 1) {
      if (ctx->score_force_cluster > 0) return cudaErrorLaunchOutOfResources;
      continue;
    }
    if (ctx->score_force_cluster > 0) break;
    const int avail = max_clusters[cl] - (reserve_sms + cl - 1) / cl > 0 ? max_clusters[cl] - (reserve_sms + cl - 1) / cl : 1;
    const long long rounds = (sp.units + avail - 1) / avail;
    const long long per_cta = (tiles_max + cl - 1) / cl;
    const long long cost = rounds * (per_cta + (cl > 1 ? 3 : 1));
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost;
      best_cl = cl;
    }
  }
  if (best_cost < 0) return cudaErrorLaunchOutOfResources;
  sp.cluster = best_cl;
  attr[0].val.clusterDim.x = (unsigned)best_cl;
  int n_clusters = max_clusters[best_cl] - (reserve_sms + best_cl - 1) / best_cl;
  if (n_clusters < 1) n_clusters = 1;
  if (n_clusters > sp.units) n_clusters = sp.units;
  ctx->score_cluster = sp.cluster;
  ctx->score_clusters = n_clusters;
  cfg.gridDim = dim3((unsigned)(n_clusters * sp.cluster), 1, 1);
  return cudaLaunchKernelEx(&cfg, kern, mq, mk, sp);
}

// Ragged batches: units in descending order of sequence length (ties: lower sequence first). Walking this list
// round-robin gives every cluster a similar number of key tiles; in unit order the lengths a cluster meets are
// random and the busiest cluster of a batch with lengths spread 8x carries about 30 % more than the average.
__global__ void ta_unit_order_kernel(ta_seq_desc seq, int n_layers, int Hkv, int32_t* __restrict__ order) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= seq.batch) return;
  const int nb = seq.cu[b + 1] - seq.cu[b];
  int rank = 0;
  for (int o = 0; o < seq.batch; ++o) {
    const int no = seq.cu[o + 1] - seq.cu[o];
    rank += (no > nb) || (no == nb && o < b);
  }
  const int per = n_layers * Hkv;
  for (int j = 0; j < per; ++j) {
    const int l = j / Hkv, g = j - l * Hkv;
    order[(long long)rank * per + j] = (l * seq.batch + b) * Hkv + g;
  }
}

// One warp that waits, with the bounded waits of the score kernel, on a barrier nothing ever completes: first the CTA-scope
// form, then (with the abort flag lowered again) the cluster-scope form. Nothing else is in flight.
__global__ void ta_wait_selftest_kernel(ta_dev_status* status, unsigned long long limit_ns, int* outcome) {
  __shared__ unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncwarp();
  volatile int* af = &abort_flag;
  const bool a = mbar_wait(smem_u32(&bar), 0, af, status, 90, limit_ns);
  __syncwarp();
  if (threadIdx.x == 0) abort_flag = 0;
  __syncwarp();
  const bool b = mbar_wait_cluster(smem_u32(&bar), 0, af, status, 91, limit_ns);
  if (threadIdx.x == 0 && outcome) *outcome = (a ? 1 : 0) | (b ? 2 : 0) | 4;  // 4: the kernel ran to its end
}

}  // namespace

cudaError_t ta_launch_wait_selftest(ta_dev_status* status, unsigned long long limit_ns, int* outcome,
                                    cudaStream_t stream) {
  ta_wait_selftest_kernel<<<1, 32, 0, stream>>>(status, limit_ns, outcome);
  return cudaGetLastError();
}

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
  sp.A = a.A;
  sp.P = a.P;
  sp.u = a.u;
  sp.status = status;
  sp.wait_limit_ns = ctx->wait_limit_ns ? ctx->wait_limit_ns : kWaitLimitNs;
  for (int t = 0; t < a.W; ++t) sp.wrow[t] = (float)((1.0 - (double)a.rho) * pow((double)a.rho, (double)(a.W - 1 - t)));
  sp.units = units;
  sp.order = nullptr;
  if (a.seq.cu && a.order_scratch && B > 1) {
    ta_unit_order_kernel<<<(B + 127) / 128, 128, 0, stream>>>(a.seq, L, a.Hkv, a.order_scratch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    sp.order = a.order_scratch;
  }
  const int tiles_max = (a.seq.max_n + kTileN - 1) / kTileN;
  sp.cluster = 1;  // chosen at launch

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
  // Output form of pass 2. With only the weighted sum alpha*A + delta*P wanted and every row weight
  // alpha + delta*w_t positive, the weights go into the exponents and a key costs one sum (kOutFused); otherwise A
  // alone (kOutA) or A and P with per-row weights (kOutAP).
  bool fused = a.u != nullptr && a.A == nullptr && a.P == nullptr;
  for (int t = 0; fused && t < a.W; ++t) fused = a.alpha + a.delta * sp.wrow[t] > 0.0f;
  const bool need_p = a.P != nullptr || (a.u != nullptr && a.delta != 0.0f);
  if (MB == 1) {
    if (fused) return launch_variant<1, kOutFused>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
    if (need_p) return launch_variant<1, kOutAP>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
    return launch_variant<1, kOutA>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
  }
  if (fused) return launch_variant<2, kOutFused>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
  if (need_p) return launch_variant<2, kOutAP>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
  return launch_variant<2, kOutA>(ctx, mq, mk, sp, tiles_max, a.reserve_sms, stream);
}
