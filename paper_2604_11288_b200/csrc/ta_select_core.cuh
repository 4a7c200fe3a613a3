// Core of the budget-K selection (radix select, ordered emit, the two kernels), written against a block size that the
// including file fixes with TA_SEL_THREADS before each inclusion; everything lives in namespace TA_SEL_NS. The
// selection kernels are built for 512 threads (two blocks per SM for short units) and for 1024 threads (twice the keys
// in registers for long units).
namespace TA_SEL_NS {

constexpr int kThreads = TA_SEL_THREADS;
constexpr int kWarps = kThreads / 32;

__device__ __forceinline__ uint32_t sortable_key(float f) {
  uint32_t b = __float_as_uint(f);
  if ((b << 1) == 0u) b = 0u;  // -0 == +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

constexpr int kItemsLong = 32;  // keys per thread of clustered units (up to 8 * kItemsLong * kThreads elements)

struct SelectResult {
  uint32_t thresh;  // key of the last element taken
  int ties;         // how many elements equal to thresh are taken (lowest positions first)
  int all;          // 1: every eligible element is taken (fewer eligible than requested)
  int none;         // 1: nothing is taken
};

constexpr int kCandCap = 2048;  // candidates a split unit finishes locally

struct SelectShared {
  uint32_t hist[256];
  uint32_t prefix, mask;
  int remaining;
  int done_all;
  int ncand;  // elements in the digit bin the threshold fell into: the candidates of the next pass
  __align__(16) uint32_t warp_cnt[kWarps];  // per warp: definite count (low 16 bits) | tie count (high 16 bits)
  // range of the eligible keys: per warp (smallest, largest, how many), and per CTA of a cluster
  uint32_t wmin[kWarps], wmax[kWarps], wnum[kWarps];
  uint32_t cl_range[8][4];
  // long sequences are split over the CTAs of a cluster: histogram of the whole unit (on rank 0, two buffers
  // alternating by pass) and every CTA's (definite, tie) totals
  uint32_t ghist[2][256];
  int totals[8][2];
  // ordered write of a unit whose keys sit in registers: bitmaps of the definite and of the tie elements in position
  // order (word e covers positions 32e .. 32e+31 of this CTA's slice)
  // (a row of kWarps words per chunk, padded by one word so that the 32 rows a warp writes fall into 32 banks)
  uint32_t bdef[kItemsLong * (kWarps + 1)], btie[kItemsLong * (kWarps + 1)];
  uint32_t wtot[kWarps];
  uint32_t total;
  // a unit split over a cluster: once few candidates are left, their keys are collected (on rank 0, then copied by
  // every CTA) and the remaining passes run on that list inside each CTA, without cluster barriers
  uint32_t cand_n;
  uint32_t cand_keys[kCandCap];
};
constexpr int kSelectCluster = 8;  // CTAs per unit when a sequence is longer than kItems * kThreads

// Keys of a unit are read once into registers when the unit is short enough (kItems per thread), else they are
// re-read from L2 on every sweep in batches whose loads are all issued before the first use.
constexpr int kItems = 16;
constexpr int kBatch = 8;
static_assert(kItems % 8 == 0 && kItemsLong % 8 == 0, "the cached load works in groups of 8 keys per thread");
template <int ITEMS>
struct KeyCache {
  uint32_t key[ITEMS];
  uint32_t elig;  // bit `it`: element tid + it*kThreads exists and is eligible
};

template <class KeyFn, int ITEMS>
__device__ __forceinline__ void fill_cache(int n, KeyFn key_of, KeyCache<ITEMS>& kc) {
  kc.elig = 0;
#pragma unroll
  for (int it = 0; it < ITEMS; ++it) {
    const int i = (int)threadIdx.x + it * kThreads;
    kc.key[it] = 0;
    if (i < n && key_of(i, kc.key[it])) kc.elig |= 1u << it;
  }
}

// Calls body(i, exists, eligible, key) for every element slot in ascending chunks of kThreads; every thread of the
// block makes the same number of calls (the body may hold block-wide barriers).
template <bool CACHED, class KeyFn, class Body, int ITEMS>
__device__ __forceinline__ void sweep(int n, KeyFn key_of, const KeyCache<ITEMS>& kc, Body body) {
  const int tid = threadIdx.x;
  if (CACHED) {
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      if (it * kThreads < n) {
        const int i = tid + it * kThreads;
        body(i, i < n, ((kc.elig >> it) & 1u) != 0, kc.key[it]);
      }
    }
  } else {
    for (int base = 0; base < n; base += kBatch * kThreads) {
      uint32_t k[kBatch];
      uint32_t e = 0;
#pragma unroll
      for (int b = 0; b < kBatch; ++b) {
        const int i = base + b * kThreads + tid;
        k[b] = 0;
        if (i < n && key_of(i, k[b])) e |= 1u << b;
      }
#pragma unroll
      for (int b = 0; b < kBatch; ++b) {
        if (base + b * kThreads < n) {
          const int i = base + b * kThreads + tid;
          body(i, i < n, ((e >> b) & 1u) != 0, k[b]);
        }
      }
    }
  }
}

// Top-`want` of the eligible elements of [0, n) by key. All threads of the block must call it; the result is uniform
// across the block.
template <bool CACHED, int CL, class KeyFn, int ITEMS>
__device__ SelectResult block_radix_select(int n, int want, KeyFn key_of, const KeyCache<ITEMS>& kc, SelectShared& sh) {
  SelectResult r;
  r.thresh = 0;
  r.ties = 0;
  r.all = 0;
  r.none = (want <= 0);
  if (r.none) return r;
  const int tid = threadIdx.x, lane = tid & 31;
  if (tid == 0) {
    sh.prefix = 0;
    sh.mask = 0;
    sh.remaining = want;
    sh.done_all = 0;
  }
  uint32_t* ghist0 = nullptr;
  if (CL > 1) ghist0 = cg::this_cluster().map_shared_rank(&sh.ghist[0][0], 0);
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (tid < 256) {
      sh.hist[tid] = 0;
      if (CL > 1) sh.ghist[pass & 1][tid] = 0;  // only rank 0's copy is used; its readers of two passes ago are done
    }
    if (CL > 1) cg::this_cluster().sync();
    else __syncthreads();
    const uint32_t prefix = sh.prefix, mask = sh.mask;
    sweep<CACHED>(n, key_of, kc, [&](int, bool, bool elig, uint32_t key) {
      const int bin = (elig && (key & mask) == prefix) ? (int)((key >> shift) & 255u) : -1;
      // after the first pass most warps hold no candidate at all: a ballot is far cheaper than match.any
      const unsigned have = __ballot_sync(0xffffffffu, bin >= 0);
      if (have == 0u) return;
      if ((have & (have - 1u)) == 0u) {  // a single candidate in the warp
        if (bin >= 0) atomicAdd(&sh.hist[bin], 1u);
        return;
      }
      const unsigned peers = __match_any_sync(0xffffffffu, bin);
      if (bin >= 0 && lane == __ffs(peers) - 1) atomicAdd(&sh.hist[bin], (uint32_t)__popc(peers));
    });
    __syncthreads();
    const uint32_t* hist = sh.hist;
    if (CL > 1) {  // merge the slices' histograms on rank 0, then every CTA takes the same decision from the sum
      uint32_t* gh = ghist0 + (pass & 1) * 256;
      if (tid < 256 && sh.hist[tid]) atomicAdd(&gh[tid], sh.hist[tid]);
      cg::this_cluster().sync();
      hist = gh;
    }
    if (tid < 32) {
      // lane l owns bins [8l, 8l+8); walk from the top bin down until `remaining` elements are covered
      uint32_t hl[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) hl[k] = hist[8 * lane + k];
      uint32_t tot = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) tot += hl[k];
      uint32_t above = 0;  // elements in lanes above this one
      {
        uint32_t run = tot;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const uint32_t o = __shfl_down_sync(0xffffffffu, run, off);
          if (lane + off < 32) run += o;
        }
        above = run - tot;
      }
      const int remaining = sh.remaining;
      const uint32_t total = __shfl_sync(0xffffffffu, above + tot, 0);
      if (pass == 0 && total < (uint32_t)remaining) {
        if (lane == 0) sh.done_all = 1;
      } else {
        const bool mine = above < (uint32_t)remaining && (uint32_t)remaining <= above + tot;
        if (mine) {
          uint32_t cum = above;
          int k = 7;
#pragma unroll
          for (int kk = 7; kk > 0; --kk) {
            if (k == kk && cum + hl[kk] < (uint32_t)remaining) {
              cum += hl[kk];
              k = kk - 1;
            }
          }
          const int bin = 8 * lane + k;
          sh.remaining = remaining - (int)cum;
          sh.prefix = prefix | ((uint32_t)bin << shift);
          sh.mask = mask | (255u << shift);
        }
      }
    }
    __syncthreads();
    if (sh.done_all) {
      r.all = 1;
      return r;
    }
  }
  r.thresh = sh.prefix;
  r.ties = sh.remaining;
  return r;
}

// A unit split over a cluster, keys in registers: clears the state that peers will add to and arrives at the
// cluster barrier whose wait opens cached_radix_select(); the loads of the keys run in between.
template <int CL>
__device__ __forceinline__ void split_unit_begin(SelectShared& sh) {
  if (CL > 1) {
    const int tid = threadIdx.x;
    if (tid < 256) {
      sh.ghist[0][tid] = 0;
      sh.ghist[1][tid] = 0;
    }
    if (tid == 0) sh.cand_n = 0;
    cg::this_cluster().barrier_arrive();
  }
}

// Shared step of the radix passes: warp 0 walks the 256-bin histogram from the top bin down until `remaining`
// elements are covered and publishes the bin it stops in (sh.prefix gets the digit at `shift`, sh.remaining what is
// still to take inside that bin, sh.ncand the bin's population). Called by all threads of warp 0.
__device__ __forceinline__ void radix_walk(const uint32_t* hist, int shift, uint32_t digit_mask, uint32_t prefix,
                                           uint32_t mask, SelectShared& sh) {
  const int lane = threadIdx.x & 31;
  // lane l owns bins [8l, 8l+8)
  uint32_t hl[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) hl[k] = hist[8 * lane + k];
  uint32_t tot = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) tot += hl[k];
  uint32_t run = tot;  // inclusive sum over this lane and the lanes above it
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t o = __shfl_down_sync(0xffffffffu, run, off);
    if (lane + off < 32) run += o;
  }
  const uint32_t above = run - tot;
  const uint32_t remaining = (uint32_t)sh.remaining;
  if (above < remaining && remaining <= above + tot) {
    uint32_t cum = above;
    int k = 7;
#pragma unroll
    for (int kk = 7; kk > 0; --kk) {
      if (k == kk && cum + hl[kk] < remaining) {
        cum += hl[kk];
        k = kk - 1;
      }
    }
    uint32_t pop = hl[0];
#pragma unroll
    for (int kk = 1; kk < 8; ++kk)
      if (k == kk) pop = hl[kk];
    const int bin = 8 * lane + k;
    sh.remaining = (int)(remaining - cum);
    sh.ncand = (int)pop;
    sh.prefix = prefix | ((uint32_t)bin << shift);
    sh.mask = mask | (digit_mask << shift);
  }
}

// The remaining radix passes over the m candidate keys in sh.cand_keys (all of them match `prefix` under `mask`),
// with block barriers only. On return prefix/remaining describe the threshold as at the end of the register passes.
__device__ __forceinline__ void list_radix_finish(int m, int bits, int done, uint32_t& prefix, uint32_t& mask,
                                                  int& remaining, SelectShared& sh) {
  const int tid = threadIdx.x;
  constexpr int kPer = (kCandCap + kThreads - 1) / kThreads;
  uint32_t lk[kPer];
  uint32_t live = 0;
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    const int j = tid + q * kThreads;
    lk[q] = j < m ? sh.cand_keys[j] : 0u;
    if (j < m) live |= 1u << q;
  }
  if (tid == 0) sh.remaining = remaining;
  while (done < bits) {
    const int width = min(8, bits - done), shift = bits - done - width;
    const uint32_t digit_mask = (1u << width) - 1u;
    if (tid < 256) sh.hist[tid] = 0;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kPer; ++q) {
      if ((live >> q) & 1u) {
        if ((lk[q] & mask) != prefix) live &= ~(1u << q);
        else atomicAdd(&sh.hist[(lk[q] >> shift) & digit_mask], 1u);
      }
    }
    __syncthreads();
    if (tid < 32) radix_walk(sh.hist, shift, digit_mask, prefix, mask, sh);
    __syncthreads();
    prefix = sh.prefix;
    mask = sh.mask;
    remaining = sh.remaining;
    const int ncand = sh.ncand;
    done += width;
    if (ncand == remaining) break;
  }
}

// Top-`want` of the eligible elements when the keys sit in registers. The eligible keys' range is taken first: the
// bits above the highest bit in which two of them differ are common to all and need no pass, so the first 8-bit
// digit already spreads the keys over the whole histogram (utilities of one unit span a few binades: the top byte of
// a float alone would put most of them into two or three bins). The first pass counts every eligible element
// (match.any merges equal digits of a warp into one shared-memory atomic); from then on each thread keeps a bit mask
// of its elements that are still candidates, and the passes touch those only. The passes stop as soon as the
// candidates left are exactly as many as are still to take. n_unit is the length of the whole unit (n is this CTA's
// slice when CL > 1).
template <int CL, int ITEMS>
__device__ SelectResult cached_radix_select(int n, int n_unit, int want, const KeyCache<ITEMS>& kc, SelectShared& sh) {
  SelectResult r;
  r.thresh = 0;
  r.ties = 0;
  r.all = 0;
  r.none = (want <= 0);
  // the cluster barrier that split_unit_begin() arrived at before the keys were loaded: from here on every CTA of the
  // cluster is known to run (its shared memory may be written) and to have zeroed its ghist and cand_n
  if (CL > 1) cg::this_cluster().barrier_wait();
  if (r.none) return r;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned lt = (1u << lane) - 1u;
  uint32_t cand = kc.elig;
  uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
  for (int it = 0; it < ITEMS; ++it) {
    if ((cand >> it) & 1u) {
      kmin = min(kmin, kc.key[it]);
      kmax = max(kmax, kc.key[it]);
    }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  uint32_t num = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(cand));
  if (lane == 0) {
    sh.wmin[warp] = kmin;
    sh.wmax[warp] = kmax;
    sh.wnum[warp] = num;
  }
  if (tid == 0) sh.remaining = want;
  __syncthreads();
  static_assert(kWarps <= 32, "one lane per warp in the second reduction step");
  kmin = __reduce_min_sync(0xffffffffu, lane < kWarps ? sh.wmin[lane] : 0xffffffffu);
  kmax = __reduce_max_sync(0xffffffffu, lane < kWarps ? sh.wmax[lane] : 0u);
  num = __reduce_add_sync(0xffffffffu, lane < kWarps ? sh.wnum[lane] : 0u);
  uint32_t* ghist0 = nullptr;
  if (CL > 1) {
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    ghist0 = cluster.map_shared_rank(&sh.ghist[0][0], 0);
    if (tid < CL) {
      uint32_t* peer = cluster.map_shared_rank(&sh.cl_range[0][0], tid);
      peer[rank * 4 + 0] = kmin;
      peer[rank * 4 + 1] = kmax;
      peer[rank * 4 + 2] = num;
    }
    cluster.sync();
    kmin = 0xffffffffu;
    kmax = 0u;
    num = 0u;
#pragma unroll
    for (int q = 0; q < CL; ++q) {
      kmin = min(kmin, sh.cl_range[q][0]);
      kmax = max(kmax, sh.cl_range[q][1]);
      num += sh.cl_range[q][2];
    }
  }
  if (num < (uint32_t)want) {  // fewer eligible elements than requested: all of them
    r.all = 1;
    return r;
  }
  const uint32_t diff = kmin ^ kmax;
  if (diff == 0u) {  // all eligible keys are equal
    r.thresh = kmin;
    r.ties = want;
    return r;
  }
  const int bits = 32 - __clz(diff);  // low bits still to resolve
  uint32_t mask = bits == 32 ? 0u : (0xffffffffu << bits);
  uint32_t prefix = kmax & mask;
  int remaining = want;
  int ncand = (int)num;
  int done = 0, pass = 0;
  while (done < bits) {
    if (CL > 1 && ncand <= kCandCap) {
      // Few candidates left (uniform over the cluster: ncand comes from the merged histogram, or is the number of
      // eligible elements before the first pass). Every CTA appends its own to the list on rank 0; after one cluster
      // barrier every CTA copies the list and finishes alone. The list's order does not matter: only the multiset of
      // keys decides the threshold, so all CTAs arrive at the same one.
      cg::cluster_group cluster = cg::this_cluster();
      uint32_t* list0 = cluster.map_shared_rank(&sh.cand_keys[0], 0);
      uint32_t* count0 = cluster.map_shared_rank(&sh.cand_n, 0);
      uint32_t mine = 0;
      if (cand != 0u) {
#pragma unroll
        for (int it = 0; it < ITEMS; ++it)
          if (((cand >> it) & 1u) && (kc.key[it] & mask) == prefix) mine |= 1u << it;
      }
      // one remote atomic per warp reserves the warp's range of the list
      const uint32_t cnt = (uint32_t)__popc(mine);
      uint32_t incl = cnt;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
      }
      const uint32_t warp_n = __shfl_sync(0xffffffffu, incl, 31);
      uint32_t base = 0;
      if (lane == 0 && warp_n != 0u) base = atomicAdd(count0, warp_n);
      base = __shfl_sync(0xffffffffu, base, 0);
      uint32_t slot = base + incl - cnt;
      if (mine != 0u) {
#pragma unroll
        for (int it = 0; it < ITEMS; ++it) {
          if ((mine >> it) & 1u) {
            if (slot < (uint32_t)kCandCap) list0[slot] = kc.key[it];
            ++slot;
          }
        }
      }
      cluster.sync();
      if (cluster.block_rank() != 0)
        for (int j = tid; j < ncand; j += kThreads) sh.cand_keys[j] = list0[j];
      __syncthreads();
      list_radix_finish(ncand, bits, done, prefix, mask, remaining, sh);
      break;
    }
    const int width = min(8, bits - done), shift = bits - done - width;
    const uint32_t digit_mask = (1u << width) - 1u;
    if (tid < 256) sh.hist[tid] = 0;
    if (CL > 1 && pass >= 2) {
      // rank 0's merged histogram alternates between two buffers, both zero at the start; from the third pass on the
      // buffer is cleared again (its readers of two passes ago are done) and the clearing made visible
      if (tid < 256) sh.ghist[pass & 1][tid] = 0;
      cg::this_cluster().sync();
    } else {
      __syncthreads();
    }
    if (pass == 0 || ncand * 4 > n_unit) {  // most elements are candidates (uniform over the unit's CTAs)
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        if (it * kThreads < n) {
          const bool c = ((cand >> it) & 1u) != 0 && (kc.key[it] & mask) == prefix;
          if (!c) cand &= ~(1u << it);
          const int bin = c ? (int)((kc.key[it] >> shift) & digit_mask) : -1;
          const unsigned peers = __match_any_sync(0xffffffffu, bin);
          if (c && (peers & lt) == 0u) atomicAdd(&sh.hist[bin], (uint32_t)__popc(peers));
        }
      }
    } else if (cand != 0u) {
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        if ((cand >> it) & 1u) {
          if ((kc.key[it] & mask) != prefix) cand &= ~(1u << it);
          else atomicAdd(&sh.hist[(kc.key[it] >> shift) & digit_mask], 1u);
        }
      }
    }
    __syncthreads();
    const uint32_t* hist = sh.hist;
    if (CL > 1) {  // merge the slices' histograms on rank 0, then every CTA takes the same decision from the sum
      uint32_t* gh = ghist0 + (pass & 1) * 256;
      if (tid < 256 && sh.hist[tid]) atomicAdd(&gh[tid], sh.hist[tid]);
      cg::this_cluster().sync();
      hist = gh;
    }
    if (tid < 32) radix_walk(hist, shift, digit_mask, prefix, mask, sh);
    __syncthreads();
    prefix = sh.prefix;
    mask = sh.mask;
    remaining = sh.remaining;
    ncand = sh.ncand;
    done += width;
    ++pass;
    if (ncand == remaining) break;  // every candidate left is taken: the low bits need no pass
  }
  r.thresh = prefix;  // with the unresolved low bits zero: candidates above it are definite, equal ones are ties
  r.ties = remaining;
  return r;
}

// Ordered pass over [0, n): classify(i, eligible, key, def, tie) marks element i `definite` (taken for sure) or a
// `tie` (taken while ties last). Calls emit(i, rank) for every taken element with its rank in ascending position
// order. Returns the number taken.
template <bool CACHED, class KeyFn, class ClassFn, class EmitFn, int ITEMS>
__device__ int block_ordered_emit(int n, int ties_allowed, KeyFn key_of, const KeyCache<ITEMS>& kc, ClassFn classify,
                                  EmitFn emit, SelectShared& sh, int def_base = 0, int tie_base = 0,
                                  int* def_total_out = nullptr, int* tie_total_out = nullptr) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int def0 = def_base, tie0 = tie_base;
  sweep<CACHED>(n, key_of, kc, [&](int i, bool exists, bool elig, uint32_t key) {
    bool def = false, tie = false;
    if (exists) classify(i, elig, key, def, tie);
    const unsigned bd = __ballot_sync(0xffffffffu, def), bt = __ballot_sync(0xffffffffu, tie);
    const unsigned lt = (1u << lane) - 1u;
    if (lane == 0) sh.warp_cnt[warp] = (uint32_t)__popc(bd) | ((uint32_t)__popc(bt) << 16);
    __syncthreads();
    uint32_t before = 0, total = 0;
    const uint4* wc = reinterpret_cast<const uint4*>(sh.warp_cnt);
#pragma unroll
    for (int q = 0; q < kWarps / 4; ++q) {
      const uint4 c4 = wc[q];
      const uint32_t cs[4] = {c4.x, c4.y, c4.z, c4.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        total += cs[e];
        if (4 * q + e < warp) before += cs[e];
      }
    }
    const int def_before = (int)(before & 0xffffu) + __popc(bd & lt);
    const int ties_seen = tie_base + (int)(before >> 16) + __popc(bt & lt);
    if (def)
      emit(i, def_base + def_before + min(ties_seen, ties_allowed));
    else if (tie && ties_seen < ties_allowed)
      emit(i, def_base + def_before + ties_seen);
    def_base += (int)(total & 0xffffu);
    tie_base += (int)(total >> 16);
    __syncthreads();
  });
  if (def_total_out) *def_total_out = def_base - def0;
  if (tie_total_out) *tie_total_out = tie_base - tie0;
  return def_base + min(tie_base, ties_allowed);
}

// Bit `it` set for every chunk in which this thread's slot (tid + it * kThreads) lies inside [0, n).
__device__ __forceinline__ uint32_t exist_mask(int n) {
  const int tid = threadIdx.x;
  const int cnt = n > tid ? (n - tid + kThreads - 1) / kThreads : 0;
  return cnt >= 32 ? 0xffffffffu : ((1u << cnt) - 1u);
}

// Transpose of a 32 x 32 bit matrix held one row per lane: on return lane i holds, in bit l, what was bit i of lane l.
// Five butterfly steps, each swapping the off-diagonal blocks of size s with the lane s away.
__device__ __forceinline__ uint32_t warp_transpose32(uint32_t x, int lane) {
#pragma unroll
  for (int s = 16; s >= 1; s >>= 1) {
    const uint32_t m = s == 16 ? 0x0000ffffu : s == 8 ? 0x00ff00ffu : s == 4 ? 0x0f0f0f0fu : s == 2 ? 0x33333333u : 0x55555555u;
    const uint32_t y = __shfl_xor_sync(0xffffffffu, x, s);
    x = (lane & s) ? ((x & ~m) | ((y >> s) & m)) : ((x & m) | ((y << s) & ~m));
  }
  return x;
}

// The ordered pass when the keys sit in registers (ITEMS chunks of kThreads elements, element tid + it*kThreads in
// chunk it). One sweep classifies every element (each thread collects its own 32 bits, one in-warp bit transpose turns
// them into what 32 ballots would give) and leaves two bitmaps in shared memory, definite and tie, in position
// order: the bits of warp w in chunk it are word it*kWarps + w and cover positions 32 * word .. + 31.
// From there on thread j owns word j: a block-wide exclusive scan over the words' populations gives it the number
// of definite and of tie elements before its 32 positions, and it writes its taken positions itself (two per word on
// average) -- no key is needed for that. Three block barriers (and one cluster barrier for the totals of the lower
// ranks). emit may run on another thread than the one that holds the element's key.
template <int CL, class EmitFn, int ITEMS>
__device__ int cached_ordered_emit(int n, const SelectResult& r, const KeyCache<ITEMS>& kc, uint32_t always,
                                   EmitFn emit, SelectShared& sh) {
  static_assert(ITEMS <= kItemsLong && ITEMS <= 32, "per-thread masks hold one bit per chunk");
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunks = (n + kThreads - 1) / kThreads;
  // per thread: bit `it` of mdef / mtie = its element of chunk `it` is definite / a tie. `always` marks the elements
  // taken whatever their key (not eligible for the search); eligible ones are definite above the threshold and ties
  // at it. The elig bits exist only for elements inside the unit.
  const int ties_allowed = r.ties;
  uint32_t mdef = always, mtie = 0;
  if (!r.none) {
    if (r.all) {
      mdef |= kc.elig;
    } else {
      uint32_t above = 0, equal = 0;
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        if (it < chunks) {
          above |= kc.key[it] > r.thresh ? (1u << it) : 0u;
          equal |= kc.key[it] == r.thresh ? (1u << it) : 0u;
        }
      }
      mdef |= kc.elig & above;
      mtie = kc.elig & equal;
    }
  }
  // the warp's 32 x 32 bits transposed: lane `it` then holds the ballot of chunk `it` (bit l = lane l's element)
  mdef = warp_transpose32(mdef, lane);
  mtie = warp_transpose32(mtie, lane);
  if (lane < chunks) {
    sh.bdef[lane * (kWarps + 1) + warp] = mdef;
    sh.btie[lane * (kWarps + 1) + warp] = mtie;
  }
  __syncthreads();
  // exclusive scan of the packed populations over the chunks * kWarps words (word tid belongs to thread tid)
  static_assert(kItemsLong * kWarps <= kThreads, "one word per thread");
  const bool owner = tid < chunks * kWarps;
  const int slot = tid + tid / kWarps;  // word tid = (chunk tid / kWarps, warp tid % kWarps) in the padded rows
  const uint32_t wd = owner ? sh.bdef[slot] : 0u, wt = owner ? sh.btie[slot] : 0u;
  const uint32_t mine = (uint32_t)__popc(wd) | ((uint32_t)__popc(wt) << 16);
  uint32_t run = mine;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const uint32_t o = __shfl_up_sync(0xffffffffu, run, off);
    if (lane >= off) run += o;
  }
  const uint32_t warp_total = __shfl_sync(0xffffffffu, run, 31);
  if (lane == 0) sh.wtot[warp] = warp_total;
  __syncthreads();
  uint32_t before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kWarps; ++w) {
    const uint32_t t = sh.wtot[w];
    if (w < warp) before += t;
    all += t;
  }
  const uint32_t ex = before + run - mine;
  int def_base = 0, tie_base = 0;
  int def_all = (int)(all & 0xffffu), tie_all = (int)(all >> 16);
  if (CL > 1) {
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    if (tid < CL) {
      int* peer = cluster.map_shared_rank(&sh.totals[0][0], tid);
      peer[rank * 2 + 0] = def_all;
      peer[rank * 2 + 1] = tie_all;
    }
    cluster.sync();
    def_all = 0;
    tie_all = 0;
#pragma unroll
    for (int r = 0; r < CL; ++r) {
      if (r < rank) {
        def_base += sh.totals[r][0];
        tie_base += sh.totals[r][1];
      }
      def_all += sh.totals[r][0];
      tie_all += sh.totals[r][1];
    }
  }
  int def_before = def_base + (int)(ex & 0xffffu);
  int ties_seen = tie_base + (int)(ex >> 16);
  uint32_t m = wd | wt;
  while (m) {
    const int bit = __ffs((int)m) - 1;
    m &= m - 1u;
    const int i = 32 * tid + bit;
    if ((wd >> bit) & 1u) {
      emit(i, def_before + min(ties_seen, ties_allowed));
      ++def_before;
    } else {
      if (ties_seen < ties_allowed) emit(i, def_before + ties_seen);
      ++ties_seen;
    }
  }
  return def_all + min(tie_all, ties_allowed);
}

// The ordered pass for a unit split over CL CTAs (rank r owns a contiguous, ascending slice): a counting sweep
// gives every CTA its (definite, tie) totals, the totals are exchanged through distributed shared memory, and the
// emitting sweep starts from the sums of the lower ranks. Returns the number taken over the whole unit.
template <bool CACHED, int CL, class KeyFn, class ClassFn, class EmitFn, int ITEMS>
__device__ int cluster_ordered_emit(int n, int ties_allowed, KeyFn key_of, const KeyCache<ITEMS>& kc, ClassFn classify,
                                    EmitFn emit, SelectShared& sh) {
  static_assert(!CACHED, "keys in registers: call cached_ordered_emit");
  if (CL == 1) return block_ordered_emit<CACHED>(n, ties_allowed, key_of, kc, classify, emit, sh);
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = (int)cluster.block_rank();
  int dt = 0, tt = 0;
  block_ordered_emit<CACHED>(n, 0, key_of, kc, classify, [](int, int) {}, sh, 0, 0, &dt, &tt);
  if (threadIdx.x < CL) {
    int* peer = cluster.map_shared_rank(&sh.totals[0][0], threadIdx.x);
    peer[rank * 2 + 0] = dt;
    peer[rank * 2 + 1] = tt;
  }
  cluster.sync();
  int def_base = 0, tie_base = 0, def_all = 0, tie_all = 0;
#pragma unroll
  for (int r = 0; r < CL; ++r) {
    if (r < rank) {
      def_base += sh.totals[r][0];
      tie_base += sh.totals[r][1];
    }
    def_all += sh.totals[r][0];
    tie_all += sh.totals[r][1];
  }
  block_ordered_emit<CACHED>(n, ties_allowed, key_of, kc, classify, emit, sh, def_base, tie_base);
  return def_all + min(tie_all, ties_allowed);
}

// Slice [lo, hi) of a unit of n elements owned by this CTA when the unit is split over CL CTAs (whole chunks of
// kThreads elements per CTA so that the slices stay aligned).
template <int CL>
__device__ __forceinline__ void unit_slice(int n, int& lo, int& hi) {
  if (CL == 1) {
    lo = 0;
    hi = n;
    return;
  }
  const int rank = (int)cg::this_cluster().block_rank();
  const int per = ((n + CL - 1) / CL + kThreads - 1) / kThreads * kThreads;
  lo = min(n, rank * per);
  hi = min(n, lo + per);
}

struct SeqInfo {
  int start, n, K_eff, s_take, r_take, p;
  bool bad;  // the sequence does not lie inside the token arrays (cu_seqlens is device data the host cannot check)
};

__device__ __forceinline__ SeqInfo seq_info(const ta_seq_desc& seq, int b, int K, int n_sink, int n_recent,
                                            int k_protected) {
  SeqInfo s;
  s.start = ta_seq_begin(seq, b);
  s.n = (seq.cu ? seq.cu[b + 1] : s.start + seq.n_uniform) - s.start;
  s.bad = s.n < 0 || s.n > seq.max_n || s.start < 0 || (long long)s.start + s.n > seq.total;
  if (s.bad) s.n = 0;
  s.K_eff = min(K, s.n);
  int p = k_protected < 0 ? s.K_eff - n_sink - n_recent : k_protected;
  p = max(0, min(p, s.K_eff));
  s.p = p;
  const int K_main = s.K_eff - p;
  // mandatory list: sinks 0.. then recents n-1, n-2, .. (no duplicates), truncated to K_main entries
  const int sinks = min(n_sink, s.n);
  const int recents = max(0, min(n_recent, s.n - sinks));
  s.s_take = min(sinks, K_main);
  s.r_take = min(recents, K_main - s.s_take);
  return s;
}

template <bool CACHED, int CL, int ITEMS = kItems>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads) ta_forced_kernel(ta_seq_desc seq, int K, int n_sink, int n_recent,
                                                             int k_protected, const float* __restrict__ voucher,
                                                             uint8_t* __restrict__ forced,
                                                             int32_t* __restrict__ r_main, ta_dev_status* status,
                                                             const int32_t* __restrict__ class_K, ta_static_out so) {
  __shared__ SelectShared sh;
  ta_wait_for_prior_grid();
  // grid.x = classes * sequences * CL; without budget classes there is one class and K is the argument
  const int b = (blockIdx.x / CL) % seq.batch;
  const int cls = (blockIdx.x / CL) / seq.batch;
  if (class_K) {
    K = class_K[cls];
    forced += (long long)cls * seq.total;
    r_main += cls * seq.batch;
  }
  const SeqInfo s = seq_info(seq, b, K, n_sink, n_recent, k_protected);
  if (so.out && cls == 0) {  // the static utilities of this CTA's slice (a rejected sequence has s.n == 0)
    int slo, shi;
    unit_slice<CL>(s.n, slo, shi);
    // eight tokens per thread and step: their loads (id, then count of that id, flags, voucher) are in flight together
    for (int i0 = slo + (int)threadIdx.x; i0 < shi; i0 += 8 * kThreads) {
      int id[8], c[8];
      uint8_t fl[8];
      float V[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int i = i0 + q * kThreads;
        const long long tok = (long long)s.start + i;
        id[q] = i < shi ? so.ids[tok] : -1;
        fl[q] = i < shi ? so.flags[tok] : (uint8_t)0;
        V[q] = i < shi ? voucher[tok] : 0.0f;
      }
#pragma unroll
      for (int q = 0; q < 8; ++q) c[q] = (id[q] >= 0 && id[q] < so.vocab) ? so.hist[(long long)b * so.vocab + id[q]] : 0;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int i = i0 + q * kThreads;
        if (i < shi)
          so.out[(long long)s.start + i] = ta_static_utility(i, s.n, c[q], (fl[q] & TA_FLAG_ANCHOR_TOKEN) != 0, V[q],
                                                             so.beta, so.gamma, so.lambda);
      }
    }
  }
  if (s.bad) {
    if (threadIdx.x == 0) {
      if (atomicCAS(&status->code, 0, (int)TA_ERR_DEVICE_BOUNDS) == 0) {
        status->where = 3;
        status->detail0 = b;
        status->detail1 = s.start;
      }
      r_main[b] = -2;  // poisoned: the select kernel writes an empty result
    }
    return;
  }
  if (s.K_eff == s.n) {
    if (threadIdx.x == 0) r_main[b] = -1;  // keep everything
    return;
  }
  int lo, hi;
  unit_slice<CL>(s.n, lo, hi);
  const float* V = voucher + s.start + lo;  // this CTA's slice; local index il <-> position lo + il
  auto mandatory = [&](int i) { return i < s.s_take || i >= s.n - s.r_take; };
  auto key_of = [&](int il, uint32_t& key) {
    const float v = V[il];
    key = sortable_key(v);
    return v > 0.0f && !mandatory(lo + il);
  };
  KeyCache<ITEMS> kc;
  if constexpr (CACHED) split_unit_begin<CL>(sh);
  if (CACHED) fill_cache(hi - lo, key_of, kc);
  SelectResult r;
  if constexpr (CACHED) r = cached_radix_select<CL>(hi - lo, s.n, s.p, kc, sh);
  else r = block_radix_select<CACHED, CL>(hi - lo, s.p, key_of, kc, sh);
  uint8_t* f = forced + s.start + lo;
  // ordered pass: mandatory tokens and vouchers above the threshold are forced for sure; vouchers equal to the
  // threshold are forced while protected slots last, lowest position first
  auto classify = [&](int il, bool cand, uint32_t key, bool& def, bool& tie) {
    def = mandatory(lo + il) || (cand && !r.none && (r.all || key > r.thresh));
    tie = !def && cand && !r.none && !r.all && key == r.thresh;
    f[il] = 0;  // set by emit when taken (later, after a block barrier; possibly by another thread)
  };
  auto emit = [&](int il, int rank) { f[il] = 1; };
  int taken;
  if constexpr (CACHED) {
    uint32_t always = 0;  // the mandatory tokens; every flag is cleared here and set by emit after a block barrier
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
      const int il = (int)threadIdx.x + it * kThreads;
      if (il < hi - lo) {
        f[il] = 0;
        if (mandatory(lo + il)) always |= 1u << it;
      }
    }
    taken = cached_ordered_emit<CL>(hi - lo, r, kc, always, emit, sh);
  } else {
    taken = cluster_ordered_emit<CACHED, CL>(hi - lo, r.ties, key_of, kc, classify, emit, sh);
  }
  if (threadIdx.x == 0 && blockIdx.x % CL == 0) r_main[b] = s.K_eff - taken;
}

struct UnitSrc {  // where a unit's utility comes from
  const float* u;         // fused: [L][Hkv][total]
  const float* A;         // unfused
  const float* P;
  const float* u_static;  // per token
  float alpha, delta;
};

__device__ __forceinline__ float unit_utility(const UnitSrc& src, long long unit_off, long long tok) {
  const float u0 = src.u_static[tok];
  if (src.u) return __fadd_rn(src.u[unit_off + tok], u0);
  if (!src.A) return u0;
  const float aA = __fmul_rn(src.alpha, src.A[unit_off + tok]);
  const float dP = __fmul_rn(src.delta, src.P ? src.P[unit_off + tok] : 0.0f);
  return __fadd_rn(__fadd_rn(aA, dP), u0);
}

// Small budgets and few units: the block that selected a unit also moves its retained K and V rows (Algorithm 1
// step 9), which saves the launch of the gather kernel where that launch costs more than the copy. Same result as ta_compact_kernel:
// rows at and beyond the retained count, and rows whose index lies outside the sequence, are zero.
struct GatherDst {
  ta_bf16_view k, v;
  uint4* k_out;
  uint4* v_out;
};
constexpr int kGatherMaxK = 16;  // one 16-byte piece per thread

__device__ __forceinline__ void gather_unit(const GatherDst& gd, const ta_seq_desc& seq, int unit, int l, int b, int g,
                                            int n, int K, const int32_t* out, int taken) {
  constexpr int kLanesPerRow = TA_HEAD_DIM * 2 / 16;
  __syncthreads();  // the unit's indices were written by other threads of this block
  for (int t = threadIdx.x; t < K * 2 * kLanesPerRow; t += kThreads) {
    const int r = t / (2 * kLanesPerRow), which = (t / kLanesPerRow) & 1, lane16 = t % kLanesPerRow;
    const ta_bf16_view& src = which ? gd.v : gd.k;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (r < taken) {
      const int i = out[r];
      if (i >= 0 && i < n) {
        const long long base = (long long)l * src.stride_l + (long long)g * src.stride_h +
                               (seq.cu ? (long long)seq.cu[b] * src.stride_n : (long long)b * src.stride_b);
        val = __ldg(reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(src.ptr) + base +
                                                   (long long)i * src.stride_n) + lane16);
      }
    }
    (which ? gd.v_out : gd.k_out)[((long long)unit * K + r) * kLanesPerRow + lane16] = val;
  }
}

// grid.x = units. scored: unit = (l*B + b)*Hkv + g; fast: unit = b.
template <bool CACHED, int CL, int ITEMS = kItems, bool GATHER = false>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads) ta_select_kernel(ta_seq_desc seq, int n_layers, int Hkv, int K, int fast,
                                                             UnitSrc src, const uint8_t* __restrict__ forced,
                                                             const int32_t* __restrict__ r_main,
                                                             int32_t* __restrict__ idx, int32_t* __restrict__ count,
                                                             GatherDst gd, const int32_t* __restrict__ class_of) {
  __shared__ SelectShared sh;
  ta_wait_for_prior_grid();
  const int unit = blockIdx.x / CL;
  const bool lead = blockIdx.x % CL == 0;
  int b, l = 0, g = 0;
  if (fast) {
    b = unit;
  } else {
    g = unit % Hkv;
    b = (unit / Hkv) % seq.batch;
    l = unit / (Hkv * seq.batch);
  }
  if (class_of) {  // budgets per (layer, head): the forced set and the main-pool size of this pair's class
    const int cls = class_of[l * Hkv + g];
    forced += (long long)cls * seq.total;
    r_main += cls * seq.batch;
  }
  const int start = ta_seq_begin(seq, b);
  const int n = (seq.cu ? seq.cu[b + 1] : start + seq.n_uniform) - start;
  int32_t* out = idx + (long long)unit * K;
  const int want = r_main[b];
  const int tid = threadIdx.x;
  if (want == -2) {  // sequence rejected by ta_forced_kernel
    if (lead) {
      for (int r = tid; r < K; r += kThreads) out[r] = -1;
      if (tid == 0) count[unit] = 0;
    }
    if constexpr (GATHER) gather_unit(gd, seq, unit, l, b, g, n, K, out, 0);
    return;
  }
  if (want == -1) {  // K >= n: keep everything
    if (lead) {
      for (int r = tid; r < K; r += kThreads) out[r] = r < n ? r : -1;
      if (tid == 0) count[unit] = n;
    }
    if constexpr (GATHER) gather_unit(gd, seq, unit, l, b, g, n, K, out, n);
    return;
  }
  const long long unit_off = fast ? 0 : ((long long)l * Hkv + g) * seq.total;
  int lo, hi;
  unit_slice<CL>(n, lo, hi);
  const uint8_t* f = forced + start + lo;
  auto key_of = [&](int il, uint32_t& key) {
    key = sortable_key(unit_utility(src, unit_off, (long long)start + lo + il));
    return f[il] == 0;
  };
  KeyCache<ITEMS> kc;
  if constexpr (CACHED) {
    split_unit_begin<CL>(sh);
    if (src.u) {
      // the attention part comes from HBM, the per-token arrays mostly from L2: issue all loads of the former first
      // (they land in the registers that hold the keys afterwards), so one memory latency covers the whole unit
      const int nl = hi - lo;
      const float* up = src.u + unit_off + start + lo;
      const float* sp = src.u_static + start + lo;
      kc.elig = 0;
      // loads as selects, never under a branch: nothing then keeps them from being in flight together
      float uu[ITEMS];
#pragma unroll
      for (int it = 0; it < ITEMS; ++it) {
        const int i = tid + it * kThreads;
        uu[it] = i < nl ? up[i] : 0.0f;
      }
      // the per-token values in groups of 8 (registers: a group's loads are in flight together, no more)
#pragma unroll
      for (int g0 = 0; g0 < ITEMS; g0 += 8) {
        float us[8];
        uint8_t ff[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int i = tid + (g0 + q) * kThreads;
          us[q] = i < nl ? sp[i] : 0.0f;
          ff[q] = i < nl ? f[i] : (uint8_t)1;
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
          const int it = g0 + q;
          const bool in = tid + it * kThreads < nl;
          kc.key[it] = in ? sortable_key(__fadd_rn(uu[it], us[q])) : 0u;
          kc.elig |= (in && ff[q] == 0) ? (1u << it) : 0u;
        }
        asm volatile("" ::: "memory");  // keeps the next group's loads behind this group's use
      }
    } else {
      fill_cache(hi - lo, key_of, kc);
    }
  }
  SelectResult r;
  if constexpr (CACHED) r = cached_radix_select<CL>(hi - lo, n, want, kc, sh);
  else r = block_radix_select<CACHED, CL>(hi - lo, want, key_of, kc, sh);
  auto classify = [&](int, bool elig, uint32_t key, bool& def, bool& tie) {
    def = !elig || (!r.none && (r.all || key > r.thresh));
    tie = !def && !r.none && !r.all && key == r.thresh;
  };
  auto emit = [&](int il, int rank) {
    if (rank < K) out[rank] = lo + il;
  };
  int taken;
  if constexpr (CACHED)  // forced tokens (not eligible, inside the unit) are taken whatever their key
    taken = cached_ordered_emit<CL>(hi - lo, r, kc, exist_mask(hi - lo) & ~kc.elig, emit, sh);
  else
    taken = cluster_ordered_emit<CACHED, CL>(hi - lo, r.ties, key_of, kc, classify, emit, sh);
  if (!lead) return;
  for (int q = taken + tid; q < K; q += kThreads) out[q] = -1;
  if (tid == 0) count[unit] = taken;
  if constexpr (GATHER) gather_unit(gd, seq, unit, l, b, g, n, K, out, min(taken, K));
}

}  // namespace TA_SEL_NS
