// Step 4 of the retention path: eviction as a gather of the retained K and V rows into a compact cache
// (Algorithm 1 step 9; "index_select on KV tensors along the sequence dimension", Section 3.2).
//
// Pure data movement: a row is head_dim bf16 = 256 bytes = 16 lanes x 128 bits. Each thread moves four
// independent 16-byte pieces (four rows of the same unit) so that enough loads are in flight to cover HBM latency;
// source rows are read once through the non-coherent path and written with streaming stores.
#include "ta_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kLanesPerRow = TA_HEAD_DIM * 2 / 16;           // 16
constexpr int kRowsPerIter = kThreads / kLanesPerRow;        // 16
constexpr int kUnroll = 4;
constexpr int kRowsPerBlock = kRowsPerIter * kUnroll;        // 64

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) {
  asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
               : "memory");
}

// grid.x = units (l, b, g), grid.y = ceil(K / 64) row blocks, grid.z = 2 (K cache, V cache)
__global__ void __launch_bounds__(kThreads) ta_compact_kernel(ta_seq_desc seq, int Hkv, int K, ta_bf16_view kv0,
                                                              ta_bf16_view kv1, const int32_t* __restrict__ idx,
                                                              const int32_t* __restrict__ count,
                                                              uint4* __restrict__ out0, uint4* __restrict__ out1) {
  ta_wait_for_prior_grid();
  const int unit = blockIdx.x;
  const int g = unit % Hkv;
  const int b = (unit / Hkv) % seq.batch;
  const int l = unit / (Hkv * seq.batch);
  const ta_bf16_view src = blockIdx.z ? kv1 : kv0;
  uint4* out = (blockIdx.z ? out1 : out0) + (long long)unit * K * kLanesPerRow;
  const int32_t* uidx = idx + (long long)unit * K;
  const int cnt = count[unit];
  const int n = seq.cu ? seq.cu[b + 1] - seq.cu[b] : seq.n_uniform;
  const long long base = (long long)l * src.stride_l + (long long)g * src.stride_h +
                         (seq.cu ? (long long)seq.cu[b] * src.stride_n : (long long)b * src.stride_b);
  const uint16_t* sp = reinterpret_cast<const uint16_t*>(src.ptr) + base;
  const int lane16 = threadIdx.x % kLanesPerRow;
  const int r0 = blockIdx.y * kRowsPerBlock + threadIdx.x / kLanesPerRow;

  uint4 v[kUnroll];
  int rows[kUnroll];
#pragma unroll
  for (int j = 0; j < kUnroll; ++j) {
    const int r = r0 + j * kRowsPerIter;
    rows[j] = r;
    v[j] = make_uint4(0u, 0u, 0u, 0u);
    if (r < K && r < cnt) {
      const int i = uidx[r];
      if (i >= 0 && i < n)  // an index outside the sequence is skipped, never dereferenced
        v[j] = ld_stream(reinterpret_cast<const uint4*>(sp + (long long)i * src.stride_n) + lane16);
    }
  }
#pragma unroll
  for (int j = 0; j < kUnroll; ++j)
    if (rows[j] < K) st_stream(out + (long long)rows[j] * kLanesPerRow + lane16, v[j]);
}

}  // namespace

cudaError_t ta_launch_compact(const ta_compact_args& a, int sm_count, cudaStream_t stream) {
  (void)sm_count;
  const int units = a.n_layers * a.seq.batch * a.Hkv;
  if (units == 0 || a.K == 0) return cudaSuccess;
  dim3 grid(units, (a.K + kRowsPerBlock - 1) / kRowsPerBlock, 2);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  if (a.pdl) ta_pdl_attribute(&attr[0]);
  cfg.attrs = attr;
  cfg.numAttrs = a.pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, ta_compact_kernel, a.seq, a.Hkv, a.K, a.k, a.v, a.idx, a.count,
                            reinterpret_cast<uint4*>(a.k_out), reinterpret_cast<uint4*>(a.v_out));
}
