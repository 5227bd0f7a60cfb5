// RMSNorm (Sec. 3.1) fused with the LoRA shrink T[m] = (alpha/r) * h[m] A_a(m)^T  (first half of the
// low-rank term of Eq. 1-4), the adapter gathered per row from the run-time pointer table (Sec. 3.2 (c)).
// One CTA per (row, slice of the rank indices): the row is normalised (or loaded), kept in shared memory,
// and each warp forms rank-r inner products with 128-bit loads of A and a warp-level reduction.
#include "common.cuh"

namespace mlora {

constexpr int SHRINK_THREADS = 256;
constexpr int SHRINK_JCHUNK = 8;   // rank indices per CTA

__global__ void __launch_bounds__(SHRINK_THREADS) norm_shrink_kernel(const ShrinkArgs p, const int jchunks) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* hrow = reinterpret_cast<__half*>(smem_raw);          // [K]
  __shared__ float red[SHRINK_THREADS / 32];
  const int m = blockIdx.x;
  const int K = p.K;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (p.x_f32 != nullptr) {
    const float* x = p.x_f32 + (size_t)m * K;
    float ss = 0.f;
    for (int k = threadIdx.x * 4; k < K; k += SHRINK_THREADS * 4) {
      const float4 v = *reinterpret_cast<const float4*>(x + k);
      ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if (lane == 0) red[warp] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < SHRINK_THREADS / 32; ++w) tot += red[w];
    const float inv = rsqrtf(tot / (float)K + p.eps);
    for (int k = threadIdx.x * 4; k < K; k += SHRINK_THREADS * 4) {
      const float4 v = *reinterpret_cast<const float4*>(x + k);
      const uint2 gv = *reinterpret_cast<const uint2*>(p.gain + k);
      const float2 g01 = __half22float2(u32_as_h2(gv.x)), g23 = __half22float2(u32_as_h2(gv.y));
      const __half2 o01 = __floats2half2_rn(v.x * inv * g01.x, v.y * inv * g01.y);
      const __half2 o23 = __floats2half2_rn(v.z * inv * g23.x, v.w * inv * g23.y);
      const uint2 o = make_uint2(h2_as_u32(o01), h2_as_u32(o23));
      *reinterpret_cast<uint2*>(hrow + k) = o;
      if (blockIdx.y == 0) *reinterpret_cast<uint2*>(p.h_out + (size_t)m * K + k) = o;
    }
  } else {
    const __half* h = p.h_in + (size_t)m * K;
    for (int k = threadIdx.x * 8; k < K; k += SHRINK_THREADS * 8)
      *reinterpret_cast<uint4*>(hrow + k) = *reinterpret_cast<const uint4*>(h + k);
  }
  __syncthreads();

  if (p.lora.adapter_idx == nullptr) return;
  const int r = p.lora.rank;
  const int a = p.lora.adapter_idx[m / p.lora.rows_per_stream];
  const int seg = blockIdx.y / jchunks;
  const int jc = blockIdx.y % jchunks;
  const int j0 = jc * SHRINK_JCHUNK, j1 = min(r, j0 + SHRINK_JCHUNK);
  float* T = p.lora.T + ((size_t)m * p.lora.nseg + seg) * r;
  const __half* A = nullptr;
  if (a >= 0 && a < p.lora.n_slots) A = p.lora.tabA[(size_t)a * p.lora.tab_stride + p.lora.seg[seg].proj_index];
  if (A == nullptr) {
    for (int j = j0 + threadIdx.x; j < j1; j += SHRINK_THREADS) T[j] = 0.f;
    return;
  }
  const float s = p.lora.scale[a];
  for (int j = j0 + warp; j < j1; j += SHRINK_THREADS / 32) {
    const __half* arow = A + (size_t)j * K;
    float acc = 0.f;
    for (int k = lane * 8; k < K; k += 32 * 8) {
      const uint4 av = *reinterpret_cast<const uint4*>(arow + k);
      const uint4 hv = *reinterpret_cast<const uint4*>(hrow + k);
      const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
      const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 af = __half22float2(u32_as_h2(aw[e])), hf = __half22float2(u32_as_h2(hw[e]));
        acc = fmaf(af.x, hf.x, acc);
        acc = fmaf(af.y, hf.y, acc);
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) T[j] = s * acc;
  }
}

cudaError_t init_shrink() {
  return cudaFuncSetAttribute(norm_shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
}

cudaError_t launch_shrink(const ShrinkArgs& a, cudaStream_t st) {
  int jchunks = 1, gy = 1;
  if (a.lora.adapter_idx != nullptr) {
    jchunks = (a.lora.rank + SHRINK_JCHUNK - 1) / SHRINK_JCHUNK;
    gy = jchunks * a.lora.nseg;
  }
  dim3 grid(a.M, gy);
  norm_shrink_kernel<<<grid, SHRINK_THREADS, (size_t)a.K * sizeof(__half), st>>>(a, jchunks);
  return cudaGetLastError();
}

}  // namespace mlora
