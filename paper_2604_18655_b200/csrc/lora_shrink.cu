// RMSNorm (Sec. 3.1) fused with the LoRA shrink T[m] = (alpha/r) * h[m] A_a(m)^T  (first half of the
// low-rank term of Eq. 1-4), the adapter gathered per row from the run-time pointer table (Sec. 3.2 (c)).
// One CTA per (row, slice of the rank indices): the row is normalised (or loaded), kept in shared memory,
// and each warp forms rank-r inner products with 128-bit loads of A and a warp-level reduction.
#include "common.cuh"

namespace mlora {

constexpr int SHRINK_THREADS = 256;
constexpr int SHRINK_JCHUNK = 8;   // rank indices per CTA

__global__ void __launch_bounds__(SHRINK_THREADS) norm_shrink_kernel(const ShrinkArgs p, const int jchunks) {
  // (the tensor-core projection launched after this kernel may start streaming its weights now)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

// LoRA shrink on mma.sync for passes whose rows come in runs of 16 that share an adapter (rows_per_stream a multiple
// of 16: DS2D trees of 16 or 32 nodes).  One CTA per (16 rows, segment, 8 rank indices); its sixteen warps split K in
// contiguous ranges and the partial fragments are added in warp order.  Per 16 features a thread loads 8 consecutive
// features of an activation row (rows g and g+8 of the tile) and of an A row (rank index j0 + g): the two k16 steps
// use features {0,1 | 2,3} and {4,5 | 6,7} of that piece for the fragment's (k 2t.. | k 2t+8..) slots -- any pairing of
// slots with features is valid as long as both operands use the same one.  The activations are the fp16 rows the
// GEMM reads (written by the norm pass before), so the A matrix of a stream is fetched once per 16 rows.
constexpr int SHRINK_MMA_WARPS = 16;
__global__ void __launch_bounds__(SHRINK_MMA_WARPS * 32) shrink_mma_kernel(const ShrinkArgs p, const __half* __restrict__ h) {
  // (the tensor-core projection launched after this kernel may start streaming its weights now)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ float red[SHRINK_MMA_WARPS][32][4];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int m0 = blockIdx.x * 16, r = p.lora.rank, K = p.K;
  const int jtiles = (r + 7) / 8;
  const int seg = blockIdx.y / jtiles, j0 = (blockIdx.y % jtiles) * 8;
  const int mA = m0 + g, mB = mA + 8;
  const int a = p.lora.adapter_idx[m0 / p.lora.rows_per_stream];
  const __half* A = nullptr;
  if (a >= 0 && a < p.lora.n_slots) A = p.lora.tabA[(size_t)a * p.lora.tab_stride + p.lora.seg[seg].proj_index];
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  if (A != nullptr) {
    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
    // a warp takes a contiguous range of 64-feature blocks; per block a thread reads 32 contiguous bytes of each of
    // its three rows, so a warp fetches whole 128-byte lines
    const int nblk = K / 64, per = (nblk + SHRINK_MMA_WARPS - 1) / SHRINK_MMA_WARPS;
    const int b0 = warp * per, b1 = min(nblk, b0 + per);
    const uint4* hA = reinterpret_cast<const uint4*>(h + (size_t)min(mA, p.M - 1) * K) + 2 * t;
    const uint4* hB = reinterpret_cast<const uint4*>(h + (size_t)min(mB, p.M - 1) * K) + 2 * t;
    const uint4* Ar = reinterpret_cast<const uint4*>(A + (size_t)min(j0 + g, r - 1) * K) + 2 * t;
    const bool okA = mA < p.M, okB = mB < p.M, okJ = j0 + g < r;
    auto block = [&](const uint4 (&va)[2], const uint4 (&vb)[2], const uint4 (&vw)[2]) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint32_t f0[4] = {va[q].x, vb[q].x, va[q].y, vb[q].y}, f1[4] = {va[q].z, vb[q].z, va[q].w, vb[q].w};
        mma_16816(acc, f0, vw[q].x, vw[q].y);
        mma_16816(acc, f1, vw[q].z, vw[q].w);
      }
    };
    int b = b0;
    for (; b + 2 <= b1; b += 2) {                              // two blocks' loads in flight
      uint4 va[2][2], vb[2][2], vw[2][2];
#pragma unroll
      for (int u = 0; u < 2; ++u)
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int o = (b + u) * 8 + q;
          va[u][q] = okA ? __ldg(hA + o) : zero; vb[u][q] = okB ? __ldg(hB + o) : zero; vw[u][q] = okJ ? __ldg(Ar + o) : zero;
        }
      block(va[0], vb[0], vw[0]);
      block(va[1], vb[1], vw[1]);
    }
    for (; b < b1; ++b) {
      uint4 va[2], vb[2], vw[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const int o = b * 8 + q;
        va[q] = okA ? __ldg(hA + o) : zero; vb[q] = okB ? __ldg(hB + o) : zero; vw[q] = okJ ? __ldg(Ar + o) : zero;
      }
      block(va, vb, vw);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) red[warp][lane][e] = acc[e];
  __syncthreads();
  if (warp == 0) {
    const float s = (A != nullptr) ? p.lora.scale[a] : 0.f;
    float tot[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int w = 0; w < SHRINK_MMA_WARPS; ++w)
#pragma unroll
      for (int e = 0; e < 4; ++e) tot[e] += red[w][lane][e];
    // fragment: [0],[1] = row mA, rank j0 + 2t, +1;  [2],[3] = row mB
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int m = (e < 2) ? mA : mB, j = j0 + 2 * t + (e & 1);
      if (m < p.M && j < r) p.lora.T[((size_t)m * p.lora.nseg + seg) * r + j] = s * tot[e];
    }
  }
}

cudaError_t init_shrink() {
  return cudaFuncSetAttribute(norm_shrink_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
}

cudaError_t launch_shrink(const ShrinkArgs& a, cudaStream_t st) {
  // Runs of 16 rows share an adapter: the norm (if any) as its own pass, the shrink on mma.sync from the fp16 rows.
  // With a norm this costs a second launch, which pays only when the shrink is large.
  const bool big = (long long)a.lora.rank * a.lora.nseg * a.K >= 150000;
  if (a.lora.adapter_idx != nullptr && a.lora.rows_per_stream % 16 == 0 && a.M >= 32 && (a.x_f32 == nullptr || big)) {
    const __half* h = a.h_in;
    if (a.x_f32 != nullptr) {
      ShrinkArgs n = a;
      n.lora.adapter_idx = nullptr;
      dim3 grid(a.M, 1);
      norm_shrink_kernel<<<grid, SHRINK_THREADS, (size_t)a.K * sizeof(__half), st>>>(n, 1);
      const cudaError_t e = cudaGetLastError();
      if (e != cudaSuccess) return e;
      h = a.h_out;
    }
    dim3 grid((a.M + 15) / 16, a.lora.nseg * ((a.lora.rank + 7) / 8));
    shrink_mma_kernel<<<grid, SHRINK_MMA_WARPS * 32, 0, st>>>(a, h);
    return cudaGetLastError();
  }
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
