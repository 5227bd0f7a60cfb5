// The paper's own precision regime for a single projection (Sec. 3.3 "LLM Quantization": activations quantised
// per tensor to Int8, weights per channel to Int4): y[m][n] = (sum_k qx[m][k] * qw[n][k]) * (x_scale * w_scale[n]) with
// the contraction in exact integer arithmetic on the tensor cores (mma.sync m16n8k32, s8 x s8 -> s32).
//
// Few rows (M <= 64), so the weights are the 16-row operand: a CTA owns 16 output channels, its eight warps split K in
// spans of 256 inputs, and within a span thread (g, t) of a warp reads the 64 inputs [64 t, 64 t + 64) of channels g
// and g + 8 (two 16-byte loads each: the INT4 bytes as they are stored, channel-major) and of activation row g of
// every 8-row tile.  Which input lands in which k slot of an MMA does not matter for a dot product as long as both
// operands agree, and here the slot depends on t alone: one 32-bit word of nibbles (inputs 8i .. 8i+7) splits into the
// even inputs (low nibbles) and the odd ones (high nibbles), the activation bytes are zipped the same way (prmt).
// Integer partial sums are added across warps in shared memory (any order: exact), then scaled in float32.
#include "common.cuh"

namespace mlora {

constexpr int WA_WARPS = 8;
constexpr int WA_THREADS = WA_WARPS * 32;
constexpr int WA_CH = 16;            // output channels per CTA
constexpr int WA_SPAN = 256;         // inputs per warp step

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 ldg_nc16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// four stored nibbles (q + 8) in the low halves of four bytes -> four int8 values q
__device__ __forceinline__ uint32_t nib_to_s8(uint32_t v) { return __vsub4(v & 0x0f0f0f0fu, 0x08080808u); }

template <int NT>
__global__ void __launch_bounds__(WA_THREADS) w4a8_kernel(const unsigned char* __restrict__ qw, const __half* __restrict__ w_scale,
                                                         const signed char* __restrict__ qx, float x_scale, int M, int K, int N,
                                                         float* __restrict__ y) {
  __shared__ int red[WA_WARPS][NT][32][4];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n0 = blockIdx.x * WA_CH;
  int acc[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0;
  const unsigned char* w_lo = qw + (size_t)(n0 + g) * (K / 2);
  const unsigned char* w_hi = qw + (size_t)(n0 + g + 8) * (K / 2);
  const int spans = K / WA_SPAN;
#pragma unroll 2
  for (int sp = warp; sp < spans; sp += WA_WARPS) {
    const int k0 = sp * WA_SPAN + t * 64;
    uint32_t wl[8], wh[8];
    *reinterpret_cast<uint4*>(wl) = ldg_nc16(w_lo + k0 / 2);
    *reinterpret_cast<uint4*>(wl + 4) = ldg_nc16(w_lo + k0 / 2 + 16);
    *reinterpret_cast<uint4*>(wh) = ldg_nc16(w_hi + k0 / 2);
    *reinterpret_cast<uint4*>(wh + 4) = ldg_nc16(w_hi + k0 / 2 + 16);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int row = nt * 8 + g;
      uint32_t xs[16];
      if (row < M) {
        const signed char* xr = qx + (size_t)row * K + k0;
#pragma unroll
        for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(xs + 4 * q) = __ldg(reinterpret_cast<const uint4*>(xr) + q);
      } else {
#pragma unroll
        for (int q = 0; q < 16; ++q) xs[q] = 0u;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // inputs 8i .. 8i+7 of the thread's 64: even ones in k slots 4t .. 4t+3, odd ones in slots 16+4t .. 16+4t+3
        const uint32_t b0 = __byte_perm(xs[2 * i], xs[2 * i + 1], 0x6420);
        const uint32_t b1 = __byte_perm(xs[2 * i], xs[2 * i + 1], 0x7531);
        mma_s8(acc[nt], nib_to_s8(wl[i]), nib_to_s8(wh[i]), nib_to_s8(wl[i] >> 4), nib_to_s8(wh[i] >> 4), b0, b1);
      }
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
    *reinterpret_cast<int4*>(red[warp][nt][lane]) = make_int4(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3]);
  __syncthreads();
  for (int i = threadIdx.x; i < NT * 32 * 4; i += WA_THREADS) {
    const int e = i & 3, ln = (i >> 2) & 31, nt = i >> 7;
    int sum = 0;
#pragma unroll
    for (int w = 0; w < WA_WARPS; ++w) sum += red[w][nt][ln][e];
    // accumulator element e of lane (g', t'): channel g' (+8 for e >= 2), activation row 8 nt + 2 t' + (e & 1)
    const int n = n0 + (ln >> 2) + ((e & 2) ? 8 : 0);
    const int row = nt * 8 + 2 * (ln & 3) + (e & 1);
    if (row < M) y[(size_t)row * N + n] = (float)sum * (x_scale * __half2float(w_scale[n]));
  }
}

// per-tensor INT8 activations: q = clip(round_half_even(x / scale), -127, 127), the division in float32
__global__ void quant_act_kernel(const __half* __restrict__ x, long long count, float scale, signed char* __restrict__ out) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  int q = __float2int_rn(__fdiv_rn(__half2float(x[i]), scale));
  q = q > 127 ? 127 : (q < -127 ? -127 : q);
  out[i] = (signed char)q;
}

cudaError_t launch_quant_act(const __half* x, long long count, float scale, signed char* out, cudaStream_t st) {
  quant_act_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(x, count, scale, out);
  return cudaGetLastError();
}

bool w4a8_shape_ok(int M, int K, int N) {
  // 127 * 8 * K must stay below 2^31 for the 32-bit accumulators
  return M >= 1 && M <= 64 && K >= WA_SPAN && K % WA_SPAN == 0 && N >= WA_CH && N % WA_CH == 0 &&
         (long long)K * 127 * 8 < (1ll << 31);
}

cudaError_t launch_w4a8(const unsigned char* w, const __half* ws, const signed char* x, float x_scale, int M, int K, int N,
                        float* y, cudaStream_t st) {
  const dim3 grid((unsigned)(N / WA_CH));
  if (M <= 8) w4a8_kernel<1><<<grid, WA_THREADS, 0, st>>>(w, ws, x, x_scale, M, K, N, y);
  else if (M <= 16) w4a8_kernel<2><<<grid, WA_THREADS, 0, st>>>(w, ws, x, x_scale, M, K, N, y);
  else if (M <= 32) w4a8_kernel<4><<<grid, WA_THREADS, 0, st>>>(w, ws, x, x_scale, M, K, N, y);
  else w4a8_kernel<8><<<grid, WA_THREADS, 0, st>>>(w, ws, x, x_scale, M, K, N, y);
  return cudaGetLastError();
}

}  // namespace mlora
