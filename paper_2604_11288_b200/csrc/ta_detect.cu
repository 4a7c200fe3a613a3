// Embedding-based anchor detector (Section 3.2 "Anchor detection", instantiation 3; Section 5.4): the confidence of a
// token is the largest cosine similarity between its input embedding and a handful of anchor-concept embeddings.
//
// The work is one pass over the embeddings (D bf16 values per token, read once; nothing else is large), so the kernel
// is built around that stream: a warp takes 16 tokens; per 32 dimensions every lane reads 16 contiguous bytes of two
// token rows straight from global memory (four lanes cover 64 contiguous bytes of a row: whole sectors, each fetched
// once), the dot products with the (at most 8) concepts run as m16n8k16 tensor-core products against concept
// fragments kept in shared memory, and the squared norms of the rows are accumulated from the same registers. The
// order of the dimensions inside a product is free as long as both operands use the same one, so a lane's 8
// consecutive dimensions serve as its fragment columns of two products. The contraction has N = 8: far too small for a
// tcgen05 tile to pay; the memory stream is what bounds it (2*D bytes per token against about 20 instructions per 16
// tokens and 16 dimensions).
#include <cuda_bf16.h>

#include "ta_internal.cuh"

namespace {

constexpr int kWarps = 8;
constexpr int kMaxConcepts = 8;

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float sq2(uint32_t w) {  // sum of squares of a bf16 pair
  const float lo = __uint_as_float(w << 16), hi = __uint_as_float(w & 0xffff0000u);
  return fmaf(lo, lo, hi * hi);
}

__global__ void __launch_bounds__(kWarps * 32)
ta_embed_conf_kernel(long long total, const __nv_bfloat16* __restrict__ emb, long long stride, int D,
                     const __nv_bfloat16* __restrict__ concepts, int C, float* __restrict__ conf) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int ld = D + 32;  // padded row: consecutive rows start 64 bytes apart modulo 128 (conflict-free 16-byte loads)
  __nv_bfloat16* s_c = reinterpret_cast<__nv_bfloat16*>(smem);           // [8][D + 32], unused concepts are zero
  float* s_inv = reinterpret_cast<float*>(smem + (size_t)kMaxConcepts * ld * 2);  // 1 / |concept|, 0 for zero vectors
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < kMaxConcepts * ld; i += blockDim.x) {
    const int c = i / ld, k = i - c * ld;
    s_c[i] = (c < C && k < D) ? concepts[(size_t)c * D + k] : __float2bfloat16(0.0f);
  }
  __syncthreads();
  if (warp < kMaxConcepts) {  // one warp per concept norm
    float acc = 0.0f;
    for (int k = lane; k < D; k += 32) {
      const float x = __bfloat162float(s_c[warp * ld + k]);
      acc = fmaf(x, x, acc);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) s_inv[warp] = acc > 0.0f ? rsqrtf(acc) : 0.0f;
  }
  __syncthreads();

  const int r = lane >> 2, q = lane & 3;  // fragment row (and row + 8), column pair
  const long long groups = (total + 15) / 16;
  for (long long g = (long long)blockIdx.x * kWarps + warp; g < groups; g += (long long)gridDim.x * kWarps) {
    const long long t0 = g * 16 + r, t1 = t0 + 8;
    // rows past the end re-read the last token; their results are not written
    const uint4* e0 = reinterpret_cast<const uint4*>(emb + (t0 < total ? t0 : total - 1) * stride) + q;
    const uint4* e1 = reinterpret_cast<const uint4*>(emb + (t1 < total ? t1 : total - 1) * stride) + q;
    const uint4* cb = reinterpret_cast<const uint4*>(s_c + (size_t)r * ld) + q;  // concept r, dimensions 8q .. 8q+7
    // two accumulator sets taken in turn: the tensor core's fp32 accumulation does not round to nearest, and its
    // error grows with the length of one accumulation chain
    float dA[4] = {0.0f, 0.0f, 0.0f, 0.0f}, dB[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    float n0 = 0.0f, n1 = 0.0f;
#pragma unroll 4
    for (int k = 0; k < D; k += 32) {  // 32 dimensions = 4 x uint4 per row
      const uint4 v0 = __ldg(e0 + (k >> 3)), v1 = __ldg(e1 + (k >> 3));
      const uint4 vb = cb[k >> 3];
      const uint32_t a0[4] = {v0.x, v1.x, v0.y, v1.y}, a1[4] = {v0.z, v1.z, v0.w, v1.w};
      mma_bf16_16816(dA, a0, vb.x, vb.y);
      mma_bf16_16816(dB, a1, vb.z, vb.w);
      n0 += (sq2(v0.x) + sq2(v0.y)) + (sq2(v0.z) + sq2(v0.w));
      n1 += (sq2(v1.x) + sq2(v1.y)) + (sq2(v1.z) + sq2(v1.w));
    }
    float d[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) d[x] = dA[x] + dB[x];
    // the four lanes of a row hold its norm in parts, and its dot products with concepts 2q and 2q + 1
    n0 += __shfl_xor_sync(0xffffffffu, n0, 1);
    n0 += __shfl_xor_sync(0xffffffffu, n0, 2);
    n1 += __shfl_xor_sync(0xffffffffu, n1, 1);
    n1 += __shfl_xor_sync(0xffffffffu, n1, 2);
    const float i0 = n0 > 0.0f ? rsqrtf(n0) : 0.0f, i1 = n1 > 0.0f ? rsqrtf(n1) : 0.0f;
    const float ca = s_inv[2 * q], cbv = s_inv[2 * q + 1];
    // concepts beyond C are zero vectors with similarity 0: they must not win over negative similarities
    float m0 = -INFINITY, m1 = -INFINITY;
    if (2 * q < C) {
      m0 = d[0] * i0 * ca;
      m1 = d[2] * i1 * ca;
    }
    if (2 * q + 1 < C) {
      m0 = fmaxf(m0, d[1] * i0 * cbv);
      m1 = fmaxf(m1, d[3] * i1 * cbv);
    }
    // NaN must survive the maximum (a NaN confidence is "no anchor" downstream): fmaxf drops it, so carry a flag
    bool bad0 = !(d[0] == d[0]) || !(d[1] == d[1]) || !(n0 == n0), bad1 = !(d[2] == d[2]) || !(d[3] == d[3]) || !(n1 == n1);
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
      m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
      bad0 = bad0 || __shfl_xor_sync(0xffffffffu, (int)bad0, o);
      bad1 = bad1 || __shfl_xor_sync(0xffffffffu, (int)bad1, o);
    }
    if (q == 0) {
      if (t0 < total) conf[t0] = bad0 ? NAN : m0;
      if (t1 < total) conf[t1] = bad1 ? NAN : m1;
    }
  }
}

}  // namespace

cudaError_t ta_launch_embed_conf(int sm_count, long long total, const void* emb, long long stride, int D,
                                 const void* concepts, int C, float* conf, cudaStream_t stream) {
  if (total == 0) return cudaSuccess;
  const size_t smem = (size_t)kMaxConcepts * (D + 32) * 2 + kMaxConcepts * sizeof(float);
  static bool attr_set[64] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (!attr_set[dev & 63]) {
    e = cudaFuncSetAttribute(ta_embed_conf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  const long long groups = (total + 15) / 16;
  long long blocks = (groups + kWarps - 1) / kWarps;
  const long long cap = (long long)sm_count * (smem > 100 * 1024 ? 1 : 2) * 2;  // persistent-ish: a few waves at most
  if (blocks > cap) blocks = cap;
  ta_embed_conf_kernel<<<(int)blocks, kWarps * 32, smem, stream>>>(total, reinterpret_cast<const __nv_bfloat16*>(emb),
                                                                  stride, D, reinterpret_cast<const __nv_bfloat16*>(concepts),
                                                                  C, conf);
  return cudaGetLastError();
}
