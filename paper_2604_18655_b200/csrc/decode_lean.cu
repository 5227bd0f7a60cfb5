// Decode step (at most 8 rows) as one small kernel per projection group, with nothing between them but the kernel
// boundary: no normalisation pass, no shrink pass, no exchange of intermediate sums through waits.
//
//  * A projection kernel reads its input rows as fp16 (x * gain of the RMSNorm ahead of it, not yet normalised; or
//    the attention / SwiGLU output), streams its 16 output columns' INT4 weights straight from global memory into
//    registers (one 16-byte load per lane and k-tile in the fragment-major layout; eight warps split K), dequantises
//    in registers (exactly fp16(q * scale)) and multiplies on the tensor cores (mma.sync m16n8k16, weights as the
//    16-wide operand, the rows as the 8-wide one).  The rows' 1/rms factor multiplies the finished sums: RMSNorm
//    (Sec. 3.1) is linear up to that factor.
//  * LoRA (Eq. 1-4): the expand y += T B happens in the epilogue; the shrink T = s x A^T of the NEXT projection is
//    computed by the kernel that PRODUCES x -- every CTA multiplies its 16 fresh columns with the matching columns of
//    A and adds the partial sums into 64-bit fixed-point accumulators with integer atomics (integer addition is
//    associative: the total is bit-reproducible), as it does for the rows' sums of squares.  By the time the next
//    kernel starts, T and the norm factors are complete.
//  * The accumulators of a whole step are zeroed by one memset at its start.
#include "../../include/mlora.h"
#include "common.cuh"

namespace mlora {

constexpr int LN_WARPS = 8;
constexpr int LN_THREADS = LN_WARPS * 32;
constexpr float LN_FIX = 4294967296.f, LN_UNFIX = 1.f / 4294967296.f;

__device__ __forceinline__ unsigned long long ln_fix(float v) { return (unsigned long long)__float2ll_rn(v * LN_FIX); }
__device__ __forceinline__ float ln_unfix(unsigned long long q) { return __ll2float_rn((long long)q) * LN_UNFIX; }
__device__ __forceinline__ void ln_red_add(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint4 ln_ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

__device__ __forceinline__ void ln_cp_async16(void* smem, const void* gmem, bool valid) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  const int sz = valid ? 16 : 0;                          // 0: the 16 bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(sa), "l"(gmem), "r"(sz) : "memory");
}

// The adapter slices a CTA needs at its end, asked for at its start (cp.async, behind the main loop):
//   sB [NTILE][M][r][16]: rows of B of this group for the CTA's columns (the expand);
//   sA [M][next_nseg][r][16]: rows of A of the consuming group for the CTA's output columns (its partial shrink).
// A missing adapter or matrix gives zeros.
// x = q * rank + j by shifts where the rank is a power of two (runtime divisions cost tens of instructions each, and
// these index computations sit at the start of every CTA and behind its main loop)
__device__ __forceinline__ void ln_divmod_rank(const LeanArgs& a, int x, int& q, int& j) {
  if (a.rank_log2 >= 0) { q = x >> a.rank_log2; j = x & (a.rank - 1); }
  else { q = x / a.rank; j = x - q * a.rank; }
}

// Items run over all CHAIN_MAX_ROWS rows (row = low three bits of the quotient; rows past M are skipped), so that no
// index needs a division by the row count.
template <int NTILE>
__device__ __forceinline__ void lean_prefetch_slices(const LeanArgs& a, const StepPhase& ph, int tile0, int n_out0, bool lora,
                                                     __half* sB, __half* sA) {
  const int r = a.rank, M = a.M;
  const int nB = lora ? NTILE * CHAIN_MAX_ROWS * r * 2 : 0;
  const int nA = (ph.next_nseg > 0 && a.adapter_idx != nullptr) ? ph.next_nseg * CHAIN_MAX_ROWS * r * 2 : 0;
  for (int it = threadIdx.x; it < nB; it += blockDim.x) {
    int q, j;
    ln_divmod_rank(a, it >> 1, q, j);
    const int hf = it & 1, m = q & (CHAIN_MAX_ROWS - 1), u = q >> 3;
    if (m >= M) continue;
    const int ad = a.rows_direct ? m : a.adapter_idx[m];
    int seg, col;
    map_col(ph.mode, (tile0 + u) * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
    const __half* B = (ad >= 0 && ad < a.n_slots) ? a.tabB[(size_t)ad * a.tab_stride + ph.lora_proj[seg]] : nullptr;
    ln_cp_async16(sB + (((size_t)u * M + m) * r + j) * 16 + hf * 8, B ? B + (size_t)j * ph.lora_n[seg] + col + hf * 8 : (const __half*)ph.w,
                  B != nullptr);
  }
  for (int it = threadIdx.x; it < nA; it += blockDim.x) {
    int q, j;
    ln_divmod_rank(a, it >> 1, q, j);
    const int hf = it & 1, m = q & (CHAIN_MAX_ROWS - 1), seg = q >> 3;
    if (m >= M) continue;
    const int ad = a.rows_direct ? m : a.adapter_idx[m];
    const __half* A = (ad >= 0 && ad < a.n_slots) ? a.tabA[(size_t)ad * a.tab_stride + ph.next_proj[seg]] : nullptr;
    ln_cp_async16(sA + (((size_t)m * ph.next_nseg + seg) * r + j) * 16 + hf * 8,
                  A ? A + (size_t)j * ph.next_ld + n_out0 + hf * 8 : (const __half*)ph.w, A != nullptr);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
}

// partial shrink of the consuming group over this CTA's fresh fp16 outputs vals[8][16]: one item per (row, segment,
// rank index), the A slices in shared memory
__device__ __forceinline__ void lean_shrink_partial(const LeanArgs& a, const StepPhase& ph, const __half (*vals)[16], const __half* sA) {
  if (ph.next_nseg == 0 || a.adapter_idx == nullptr) return;
  const int r = a.rank;
  for (int it = threadIdx.x; it < ph.next_nseg * CHAIN_MAX_ROWS * r; it += blockDim.x) {
    int q, j;
    ln_divmod_rank(a, it, q, j);
    const int m = q & (CHAIN_MAX_ROWS - 1), seg = q >> 3;
    if (m >= a.M) continue;
    const __half2* av = reinterpret_cast<const __half2*>(sA + (((size_t)m * ph.next_nseg + seg) * r + j) * 16);
    const __half2* xv = reinterpret_cast<const __half2*>(vals[m]);
    float s = 0.f;
#pragma unroll
    for (int q2 = 0; q2 < 8; ++q2) {
      const float2 x = __half22float2(xv[q2]), w = __half22float2(av[q2]);
      s = fmaf(x.x, w.x, s); s = fmaf(x.y, w.y, s);
    }
    ln_red_add(a.tacc + ((size_t)ph.t_out * CHAIN_MAX_ROWS + m) * 3 * r + seg * r + j, ln_fix(s));
  }
}

// NTILE = 1: 16 physical columns per CTA; NTILE = 2: a gate tile and its up tile (SwiGLU pair)
// Launched with programmatic stream serialisation: everything ahead of pdl_wait() -- the first weights, the adapter
// slices -- depends on no earlier kernel and is in flight while the kernel before this one finishes.
// Timeline of a traced step (the TRACE instantiations of the kernels; the others carry none of it): thread 0 of the
// first and of the last CTA stamp the GPU's global nanosecond timer into their launch's slots -- 0 start, 1 wait
// returned, 2 main loop done, 3 end -- and every CTA's thread 0 raises slot 4 of the first CTA's row to its own end.
__device__ __forceinline__ long long ln_now() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
template <bool TRACE>
__device__ __forceinline__ void ln_stamp(const LeanArgs& a, int slot) {
  if constexpr (TRACE) {
    if (threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
      const long long now = ln_now();
      if (blockIdx.x == 0) a.trace0[slot] = now;
      if (blockIdx.x == gridDim.x - 1) a.trace1[slot] = now;
    }
    if (slot == 3 && threadIdx.x == 0) atomicMax(reinterpret_cast<unsigned long long*>(a.trace0 + 4), (unsigned long long)ln_now());
  }
}

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <int NTILE, int WARPS, bool TRACE>
__global__ void __launch_bounds__(WARPS * 32, WARPS == 8 ? 3 : 1)
lean_gemm_kernel(const LeanArgs a, const __grid_constant__ StepPhase ph) {
  constexpr int THREADS = WARPS * 32;
  __shared__ float red[WARPS][NTILE][32][4];
  __shared__ float s_inv[CHAIN_MAX_ROWS];
  __shared__ float s_T[CHAIN_MAX_ROWS][3 * 64];
  __shared__ float s_y[NTILE][CHAIN_MAX_ROWS][16];
  __shared__ __align__(16) __half s_vals[CHAIN_MAX_ROWS][16];
  __shared__ float s_sq[CHAIN_MAX_ROWS][16];
  extern __shared__ __align__(16) unsigned char ln_dyn[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  ln_stamp<TRACE>(a, 0);
  pdl_launch_dependents();
  const int M = a.M, K = ph.K, r = a.rank;
  const WLayout L = make_wlayout(K, ph.N, ph.G);
  const int tile0 = blockIdx.x * NTILE;
  // ---- ahead of the wait: adapter slices and the first weights (immutable data)
  const bool lora = ph.lora_nseg > 0 && a.adapter_idx != nullptr;
  __half* sB = reinterpret_cast<__half*>(ln_dyn);                          // [NTILE][M][r][16]
  __half* sA = sB + (size_t)NTILE * CHAIN_MAX_ROWS * r * 16;               // [M][next_nseg][r][16]
  const int n_out0 = ph.epi == EPI_SWIGLU ? (tile0 >> 1) * TILE_N : tile0 * TILE_N;   // first column the CTA produces
  const int kt0 = (L.KT * warp) / WARPS, kt1 = (L.KT * (warp + 1)) / WARPS;
  const unsigned char* unit[NTILE];
#pragma unroll
  for (int u = 0; u < NTILE; ++u) unit[u] = ph.w + (size_t)(tile0 + u) * L.unit_bytes;
  constexpr int PF = 4;                                                    // k-tiles in flight per warp
  uint4 wv[PF][NTILE];
  uint32_t sv[PF][NTILE];
  auto load_weights = [&](int kb) {
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      const int kt = kb + i;
      if (kt < kt1) {
#pragma unroll
        for (int u = 0; u < NTILE; ++u) {
          wv[i][u] = ln_ldg_stream(unit[u] + wl_tile_off(L, kt) + lane * 16);
          sv[i][u] = __ldg(reinterpret_cast<const uint32_t*>(unit[u] + wl_scale_off(L, kt)) + g);
        }
      }
    }
  };
  load_weights(kt0);                                                       // (first: the longest latency)
  // this CTA's share of the next projection group's weights, asked for in L2: that kernel's CTAs mostly start only
  // when this kernel's leave their SMs, and then find their weights a short trip away
  if (threadIdx.x == 32 && ph.pf_bytes != 0) {
    const unsigned long long per = ((ph.pf_bytes / gridDim.x) + 15ull) & ~15ull;
    const unsigned long long b0 = per * blockIdx.x, b1 = b0 + per < ph.pf_bytes ? b0 + per : (ph.pf_bytes & ~15ull);
    for (unsigned long long o = b0; o < b1; o += 16384ull) {
      const uint32_t n = (uint32_t)(b1 - o < 16384ull ? b1 - o : 16384ull);
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ph.pf_w + o), "r"(n) : "memory");
    }
  }
  lean_prefetch_slices<NTILE>(a, ph, tile0, n_out0, lora, sB, sA);
  pdl_wait();
  ln_stamp<TRACE>(a, 1);
  // ---- what earlier kernels produced: the old residual, norm factors, T of this group, the input rows
  float x_old = 0.f, gain_nx = 1.f;
  if (ph.epi == EPI_RESID && threadIdx.x < 128 && (threadIdx.x >> 4) < M) {
    x_old = __ldcg(a.X + (size_t)(threadIdx.x >> 4) * ph.N + n_out0 + (threadIdx.x & 15));
    if (ph.gain_next != nullptr) gain_nx = __half2float(__ldg(ph.gain_next + n_out0 + (threadIdx.x & 15)));
  }
  if (threadIdx.x < CHAIN_MAX_ROWS) {
    float inv = 1.f;
    if (ph.norm_in >= 0 && threadIdx.x < M)
      inv = rsqrtf(ln_unfix(__ldcg(a.ssq + (size_t)ph.norm_in * CHAIN_MAX_ROWS + threadIdx.x)) / (float)K + a.eps);
    s_inv[threadIdx.x] = inv;
  }
  auto load_T = [&]() {
    for (int i = threadIdx.x; i < ph.lora_nseg * CHAIN_MAX_ROWS * r; i += THREADS) {
      int q, j;
      ln_divmod_rank(a, i, q, j);
      const int m = q & (CHAIN_MAX_ROWS - 1), rest = (q >> 3) * r + j;
      if (m >= M) continue;
      const int ad = a.rows_direct ? m : a.adapter_idx[m];
      float v = 0.f;
      if (ad >= 0 && ad < a.n_slots)
        v = ln_unfix(__ldcg(a.tacc + ((size_t)ph.t_in * CHAIN_MAX_ROWS + m) * 3 * r + rest)) * a.scale[ad];
      s_T[m][rest] = v;
    }
  };
  if (lora && !a.late_wait) load_T();
  // ---- main loop: warp w takes the k-tiles [kt0, kt1)
  float acc[NTILE][4];
#pragma unroll
  for (int u = 0; u < NTILE; ++u) acc[u][0] = acc[u][1] = acc[u][2] = acc[u][3] = 0.f;
  const __half* xrow = ph.in16 + (size_t)g * K + 16 * t;
  const bool row_live = g < M;
#pragma unroll 1
  for (int kb = kt0; kb < kt1; kb += PF) {
    uint4 x0[PF], x1[PF];
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      const int kt = kb + i;
      if (kt < kt1 && row_live) {
        // (ordinary cached loads: the CTAs that share an SM read the same rows, and loads behind the wait see what
        // the kernel ahead wrote)
        x0[i] = *(reinterpret_cast<const uint4*>(xrow + (size_t)kt * TILE_K));
        x1[i] = *(reinterpret_cast<const uint4*>(xrow + (size_t)kt * TILE_K) + 1);
      } else {
        x0[i] = make_uint4(0, 0, 0, 0);
        x1[i] = make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      if (kb + i < kt1) {
#pragma unroll
        for (int u = 0; u < NTILE; ++u) {
          __half2 s_lo, s_hi;
          split_scales(sv[i][u], s_lo, s_hi);
          uint32_t af[4][4];
          dequant8(wv[i][u].x, s_lo, s_hi, af[0]);
          dequant8(wv[i][u].y, s_lo, s_hi, af[1]);
          dequant8(wv[i][u].z, s_lo, s_hi, af[2]);
          dequant8(wv[i][u].w, s_lo, s_hi, af[3]);
          mma_16816(acc[u], af[0], x0[i].x, x0[i].y);
          mma_16816(acc[u], af[1], x0[i].z, x0[i].w);
          mma_16816(acc[u], af[2], x1[i].x, x1[i].y);
          mma_16816(acc[u], af[3], x1[i].z, x1[i].w);
        }
      }
    }
    if (kb + PF < kt1) load_weights(kb + PF);
  }
  if (a.late_wait) {
    pdl_wait();
    if (lora) load_T();
  }
  ln_stamp<TRACE>(a, 2);
#pragma unroll
  for (int u = 0; u < NTILE; ++u)
    *reinterpret_cast<float4*>(red[warp][u][lane]) = make_float4(acc[u][0], acc[u][1], acc[u][2], acc[u][3]);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // ---- one thread per (tile, row, column): sum of the warps' parts in warp order, LoRA expand, norm factor
  for (int o = threadIdx.x; o < NTILE * 128; o += THREADS) {
    const int u = o >> 7, m = (o >> 4) & 7, c = o & 15;
    // accumulator layout of m16n8k16: lane (g,t) holds (out g, row 2t), (g, 2t+1), (g+8, 2t), (g+8, 2t+1)
    const int src_lane = (c & 7) * 4 + (m >> 1), e = (c >> 3) * 2 + (m & 1);
    float y = 0.f;
    if (m < M) {
#pragma unroll
      for (int w = 0; w < WARPS; ++w) y += red[w][u][src_lane][e];
      if (lora) {
        int seg, col;
        map_col(ph.mode, (tile0 + u) * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
        const float* T = s_T[m] + seg * r;
        const __half* Bs = sB + ((size_t)u * M + m) * r * 16 + c;           // (zeros where the row has no adapter)
        float ex = 0.f;
        for (int j = 0; j < r; ++j) ex = fmaf(T[j], __half2float(Bs[(size_t)j * 16]), ex);
        y += ex;
      }
      y *= s_inv[m];
    }
    s_y[u][m][c] = y;
  }
  __syncthreads();

  const int n0 = tile0 * TILE_N;                                            // first physical column (NTILE = 1)
  if (ph.epi == EPI_F32 && ph.out_f32 == nullptr && a.amax != nullptr) {
    // lm_head without a logits destination: the row argmax (Sec. 3.5: greedy tokens; lowest column on ties) is all that
    // is wanted.  Key = order-preserving image of the value (NaN lowest) over the complemented column: the CTA's best
    // per row goes to a global maximum -- tried only when it beats what is there already.
    if (threadIdx.x < M) {
      const int m = threadIdx.x;
      unsigned long long best = 0ull;
#pragma unroll
      for (int u = 0; u < NTILE; ++u)
        for (int c = 0; c < 16; ++c) {
          float v = s_y[u][m][c];
          if (v == 0.f) v = 0.f;
          const unsigned b = __float_as_uint(v);
          const unsigned ord = (v != v) ? 0u : ((b & 0x80000000u) ? ~b : (b | 0x80000000u));
          const unsigned long long k = ((unsigned long long)ord << 32) | (unsigned)(0xffffffffu - (unsigned)((tile0 + u) * TILE_N + c));
          best = k > best ? k : best;
        }
      if (best > __ldcg(a.amax + m)) atomicMax(a.amax + m, best);
    }
    ln_stamp<TRACE>(a, 3);
    return;
  }
  if (ph.epi == EPI_F32) {
    float* out = ph.out_f32 != nullptr ? ph.out_f32 : a.logits;
    for (int o = threadIdx.x; o < NTILE * 128; o += THREADS) {
      const int u = o >> 7, m = (o >> 4) & 7, c = o & 15;
      if (m < M) out[(size_t)m * ph.ldo + (tile0 + u) * TILE_N + c] = s_y[u][m][c];
    }
    ln_stamp<TRACE>(a, 3);
    return;
  }
  if (ph.epi == EPI_RESID) {
    // new residual; x * gain for the norm that follows; the rows' sums of squares; the next group's partial shrink
    if (threadIdx.x < 128) {
      const int m = threadIdx.x >> 4, c = threadIdx.x & 15;
      float xn = 0.f;
      __half hv = __float2half_rn(0.f);
      if (m < M) {
        xn = x_old + s_y[0][m][c];
        a.X[(size_t)m * ph.N + n0 + c] = xn;
        if (ph.gain_next != nullptr) {
          hv = __float2half_rn(xn * gain_nx);
          ph.out16[(size_t)m * ph.N + n0 + c] = hv;
        }
      }
      s_vals[m][c] = hv;
      s_sq[m][c] = xn * xn;
    }
    __syncthreads();
    if (ph.ssq_out >= 0 && threadIdx.x < M) {
      float sq = 0.f;
#pragma unroll
      for (int c = 0; c < 16; ++c) sq += s_sq[threadIdx.x][c];
      ln_red_add(a.ssq + (size_t)ph.ssq_out * CHAIN_MAX_ROWS + threadIdx.x, ln_fix(sq));
    }
    lean_shrink_partial(a, ph, s_vals, sA);
    ln_stamp<TRACE>(a, 3);
    return;
  }
  // EPI_SWIGLU: tile0 is the gate tile, tile0 + 1 the up tile of 16 features
  if (NTILE == 2) {
    const int f0 = (tile0 >> 1) * TILE_N, F = ph.N / 2;
    if (threadIdx.x < 128) {
      const int m = threadIdx.x >> 4, c = threadIdx.x & 15;
      __half hv = __float2half_rn(0.f);
      if (m < M) {
        const float gt = s_y[0][m][c], up = s_y[NTILE - 1][m][c];
        hv = __float2half_rn(gt / (1.f + __expf(-gt)) * up);
        ph.out16[(size_t)m * F + f0 + c] = hv;
      }
      s_vals[m][c] = hv;
    }
    __syncthreads();
    lean_shrink_partial(a, ph, s_vals, sA);
  }
  ln_stamp<TRACE>(a, 3);
}

// The lm_head (or any wide projection without adapters: EPI_F32, K of at most LM_PF k-tiles per warp) as a persistent
// loop: a CTA takes the column tiles b, b + grid, b + 2 grid, ...; the input rows' fragments are fetched once and stay in
// registers; the packed weights of the CTA's next LM_DEPTH tiles are always in flight (cp.async into a shared-memory
// ring in which every thread owns the slots it copies into and reads back only those: no barrier); the cross-warp sums
// go through two alternating buffers (one barrier per tile); in row-maxima mode every thread keeps the best key of its
// (row, column of the tile) across its tiles: one atomic per row and CTA at the end.  2000 short-lived CTAs of the
// one-tile kernel took 20 us for the 33 MB of a 32000 x 2048 lm_head (4.5 waves, each paying the trip to HBM).
constexpr int LM_PF = 4;
constexpr int LM_DEPTH = 4;
constexpr size_t lm_smem_bytes(int threads) { return (size_t)LM_DEPTH * LM_PF * threads * (16 + 4); }
template <int WARPS, bool TRACE>
__global__ void __launch_bounds__(WARPS * 32, 2) lean_lmhead_kernel(const LeanArgs a, const __grid_constant__ StepPhase ph) {
  constexpr int THREADS = WARPS * 32;
  extern __shared__ __align__(16) unsigned char lm_dyn[];
  uint4* const wring = reinterpret_cast<uint4*>(lm_dyn);                                  // [LM_DEPTH][LM_PF][THREADS]
  uint32_t* const sring = reinterpret_cast<uint32_t*>(wring + (size_t)LM_DEPTH * LM_PF * THREADS);   // the same shape
  __shared__ float red[2][WARPS][32][4];
  __shared__ float s_inv[CHAIN_MAX_ROWS];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  ln_stamp<TRACE>(a, 0);
  pdl_launch_dependents();
  const int M = a.M, K = ph.K;
  const WLayout L = make_wlayout(K, ph.N, ph.G);
  const int kt0 = (L.KT * warp) / WARPS, kt1 = (L.KT * (warp + 1)) / WARPS;   // at most LM_PF k-tiles (the launcher checks)
  // this thread's pieces of a tile: offsets inside the tile's unit and slots inside a ring stage, fixed for the kernel
  uint32_t woff[LM_PF], soff[LM_PF];
#pragma unroll
  for (int i = 0; i < LM_PF; ++i) {
    const int kt = kt0 + i < kt1 ? kt0 + i : kt0;
    woff[i] = (uint32_t)wl_tile_off(L, kt) + lane * 16;
    soff[i] = (uint32_t)wl_scale_off(L, kt) + g * 4;
  }
  const uint32_t wslot = (uint32_t)__cvta_generic_to_shared(wring + threadIdx.x), sslot = (uint32_t)__cvta_generic_to_shared(sring + threadIdx.x);
  // one cp.async group per tile (an empty one past the last tile, so that the group count stays in step)
  auto issue = [&](int stage, int tile) {
    if (tile < L.NT) {
      const unsigned char* unit = ph.w + (size_t)tile * L.unit_bytes;
#pragma unroll
      for (int i = 0; i < LM_PF; ++i) {
        if (kt0 + i < kt1) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(wslot + (uint32_t)((stage * LM_PF + i) * THREADS * 16)), "l"(unit + woff[i]) : "memory");
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sslot + (uint32_t)((stage * LM_PF + i) * THREADS * 4)), "l"(unit + soff[i]) : "memory");
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  int tile = blockIdx.x;
#pragma unroll
  for (int d = 0; d < LM_DEPTH; ++d) issue(d, tile + d * (int)gridDim.x);
  if (threadIdx.x == 32 && ph.pf_bytes != 0) {               // the next projection group's weights, a share per CTA
    const unsigned long long per = ((ph.pf_bytes / gridDim.x) + 15ull) & ~15ull;
    const unsigned long long b0 = per * blockIdx.x, b1 = b0 + per < ph.pf_bytes ? b0 + per : (ph.pf_bytes & ~15ull);
    for (unsigned long long o = b0; o < b1; o += 16384ull) {
      const uint32_t n = (uint32_t)(b1 - o < 16384ull ? b1 - o : 16384ull);
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(ph.pf_w + o), "r"(n) : "memory");
    }
  }
  pdl_wait();
  ln_stamp<TRACE>(a, 1);
  if (threadIdx.x < CHAIN_MAX_ROWS) {
    float inv = 1.f;
    if (ph.norm_in >= 0 && threadIdx.x < M)
      inv = rsqrtf(ln_unfix(__ldcg(a.ssq + (size_t)ph.norm_in * CHAIN_MAX_ROWS + threadIdx.x)) / (float)K + a.eps);
    s_inv[threadIdx.x] = inv;
  }
  uint4 x0[LM_PF], x1[LM_PF];
  {
    const __half* xrow = ph.in16 + (size_t)g * K + 16 * t;
#pragma unroll
    for (int i = 0; i < LM_PF; ++i) {
      const int kt = kt0 + i;
      if (kt < kt1 && g < M) {
        x0[i] = *(reinterpret_cast<const uint4*>(xrow + (size_t)kt * TILE_K));
        x1[i] = *(reinterpret_cast<const uint4*>(xrow + (size_t)kt * TILE_K) + 1);
      } else {
        x0[i] = make_uint4(0, 0, 0, 0);
        x1[i] = make_uint4(0, 0, 0, 0);
      }
    }
  }
  __syncthreads();                                            // s_inv
  const bool maxima = ph.out_f32 == nullptr && a.amax != nullptr;
  float* const out = ph.out_f32 != nullptr ? ph.out_f32 : a.logits;
  // this thread's (row, column of the tile) in the epilogue, and where that sum sits in the warps' accumulators
  const int em = (threadIdx.x >> 4) & 7, ec = threadIdx.x & 15;
  const int src_lane = (ec & 7) * 4 + (em >> 1), e = (ec >> 3) * 2 + (em & 1);
  const float inv_m = s_inv[em];
  unsigned long long best = 0ull;
  int par = 0, stage = 0;
#pragma unroll 1
  for (; tile < L.NT; tile += gridDim.x) {
    asm volatile("cp.async.wait_group %0;" ::"n"(LM_DEPTH - 1) : "memory");   // this thread's pieces of the oldest tile are there
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int i = 0; i < LM_PF; ++i) {
      if (kt0 + i < kt1) {
        const uint4 wv = wring[((size_t)stage * LM_PF + i) * THREADS + threadIdx.x];
        const uint32_t sv = sring[((size_t)stage * LM_PF + i) * THREADS + threadIdx.x];
        __half2 s_lo, s_hi;
        split_scales(sv, s_lo, s_hi);
        uint32_t af[4][4];
        dequant8(wv.x, s_lo, s_hi, af[0]);
        dequant8(wv.y, s_lo, s_hi, af[1]);
        dequant8(wv.z, s_lo, s_hi, af[2]);
        dequant8(wv.w, s_lo, s_hi, af[3]);
        mma_16816(acc, af[0], x0[i].x, x0[i].y);
        mma_16816(acc, af[1], x0[i].z, x0[i].w);
        mma_16816(acc, af[2], x1[i].x, x1[i].y);
        mma_16816(acc, af[3], x1[i].z, x1[i].w);
      }
    }
    issue(stage, tile + LM_DEPTH * (int)gridDim.x);          // refills the slots just read (this thread's own)
    stage = stage + 1 == LM_DEPTH ? 0 : stage + 1;
    *reinterpret_cast<float4*>(red[par][warp][lane]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    __syncthreads();
    if (threadIdx.x < 128 && em < M) {
      float y = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) y += red[par][w][src_lane][e];
      y *= inv_m;
      const int col = tile * TILE_N + ec;
      if (maxima) {
        if (y == 0.f) y = 0.f;
        const unsigned b = __float_as_uint(y);
        const unsigned ord = (y != y) ? 0u : ((b & 0x80000000u) ? ~b : (b | 0x80000000u));
        const unsigned long long key = ((unsigned long long)ord << 32) | (unsigned)(0xffffffffu - (unsigned)col);
        best = key > best ? key : best;
      } else {
        out[(size_t)em * ph.ldo + col] = y;
      }
    }
    par ^= 1;
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  ln_stamp<TRACE>(a, 2);
  if (maxima && threadIdx.x < 128) {
    // the best key of a row: over its 16 columns' threads (half a warp), then one atomic per row and CTA
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
      best = other > best ? other : best;
    }
    if (ec == 0 && em < M && best > __ldcg(a.amax + em)) atomicMax(a.amax + em, best);
  }
  ln_stamp<TRACE>(a, 3);
}

// Embedding (or hidden-state input) of the step's rows: residual fp32, x * gain of the first norm as fp16, the rows'
// sums of squares, and the shrink sums of the first q,k,v group.  CTA (m, part): row m; part 0 also writes the row.
__global__ void __launch_bounds__(LN_THREADS) lean_embed_kernel(const LeanArgs a, const __grid_constant__ StepPhase ph,
                                                               const int32_t* __restrict__ tokens,
                                                               const __half* __restrict__ embed, int vocab,
                                                               const __half* __restrict__ hidden_in, int* __restrict__ status) {
  extern __shared__ __align__(16) unsigned char ln_smem[];
  __half* xg = reinterpret_cast<__half*>(ln_smem);                         // [d]
  __shared__ float s_part[LN_WARPS];
  pdl_launch_dependents();
  const int m = blockIdx.x, part = blockIdx.y, d = ph.N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const __half* src;
  if (hidden_in != nullptr) src = hidden_in + (size_t)m * d;
  else {
    int tok = tokens[m];
    if (tok < 0 || tok >= vocab) {
      if (threadIdx.x == 0 && part == 0) atomicCAS(status, 0, -1);
      tok = 0;
    }
    src = embed + (size_t)tok * d;
  }
  float sq = 0.f;
  for (int k = threadIdx.x * 2; k < d; k += LN_THREADS * 2) {
    const float2 v = __half22float2(*reinterpret_cast<const __half2*>(src + k));
    const float2 gn = ph.gain_next ? __half22float2(*reinterpret_cast<const __half2*>(ph.gain_next + k)) : make_float2(1.f, 1.f);
    const __half2 hv = __floats2half2_rn(v.x * gn.x, v.y * gn.y);
    *reinterpret_cast<__half2*>(xg + k) = hv;
    sq += v.x * v.x + v.y * v.y;
    if (part == 0) {
      if (a.X) *reinterpret_cast<float2*>(a.X + (size_t)m * d + k) = v;
      if (ph.out16) *reinterpret_cast<__half2*>(ph.out16 + (size_t)m * d + k) = hv;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
  if (lane == 0) s_part[warp] = sq;
  __syncthreads();
  if (part == 0 && threadIdx.x == 0 && ph.ssq_out >= 0) {
    float tot = 0.f;
    for (int w = 0; w < LN_WARPS; ++w) tot += s_part[w];
    ln_red_add(a.ssq + (size_t)ph.ssq_out * CHAIN_MAX_ROWS + m, ln_fix(tot));
  }
  if (ph.next_nseg == 0 || a.adapter_idx == nullptr) return;
  const int ad = a.rows_direct ? m : a.adapter_idx[m];
  if (ad < 0 || ad >= a.n_slots) return;
  const int r = a.rank;
  // the CTA's share of the (segment, rank index, 1024-element piece of the row) partial dot products, a warp each
  // (ph.pad_ = 1: whole dot products, stored: the sums need no zeroing then -- the single-projection call)
  const int KC = ph.pad_ ? 1 : (d + 1023) / 1024, items = ph.next_nseg * r * KC;
  for (int it = part * LN_WARPS + warp; it < items; it += gridDim.y * LN_WARPS) {
    const int kc = it % KC, j = (it / KC) % r, seg = it / (KC * r);
    const __half* A = a.tabA[(size_t)ad * a.tab_stride + ph.next_proj[seg]];
    if (A == nullptr) {
      if (ph.pad_ && lane == 0) a.tacc[((size_t)ph.t_out * CHAIN_MAX_ROWS + m) * 3 * r + seg * r + j] = 0ull;
      continue;
    }
    const __half* arow = A + (size_t)j * ph.next_ld;
    const int k1 = ph.pad_ ? d : min(d, (kc + 1) * 1024);
    float s = 0.f;
    for (int k = kc * 1024 + lane * 8; k < k1; k += 32 * 8) {
      const uint4 av = __ldg(reinterpret_cast<const uint4*>(arow + k));
      const uint4 xv = *reinterpret_cast<const uint4*>(xg + k);
      const __half2* ap = reinterpret_cast<const __half2*>(&av);
      const __half2* xp = reinterpret_cast<const __half2*>(&xv);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float2 x = __half22float2(xp[q]), w = __half22float2(ap[q]);
        s = fmaf(x.x, w.x, s); s = fmaf(x.y, w.y, s);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) {
      unsigned long long* dst = a.tacc + ((size_t)ph.t_out * CHAIN_MAX_ROWS + m) * 3 * r + seg * r + j;
      if (ph.pad_) *dst = ln_fix(s);
      else ln_red_add(dst, ln_fix(s));
    }
  }
}

// the greedy tokens from the lm_head's row maxima, and the suffix lengths one further
__global__ void lean_finish_kernel(const unsigned long long* __restrict__ amax, int32_t* __restrict__ out_next,
                                   int32_t* __restrict__ suffix_len, int n) {
  const int m = threadIdx.x;
  if (m >= n) return;
  const unsigned long long k = amax[m];
  out_next[m] = k == 0ull ? 0 : (int32_t)(0xffffffffu - (unsigned)(k & 0xffffffffull));
  suffix_len[m] += 1;
}

cudaError_t launch_lean_finish(const unsigned long long* amax, int32_t* out_next, int32_t* suffix_len, int n, cudaStream_t st) {
  lean_finish_kernel<<<1, 32, 0, st>>>(amax, out_next, suffix_len, n);
  return cudaGetLastError();
}

// The adapter matrices of every row, looked up once per call: rowA/rowB[m][p] = A/B of row m's adapter for
// projection p (nullptr: none), rowscale[m] its scale.  The per-projection kernels then index by row and skip the
// adapter-index load that every pointer lookup would otherwise wait for.
__global__ void lean_rowptr_kernel(const int32_t* __restrict__ adapter_idx, const __half* const* __restrict__ tabA,
                                   const __half* const* __restrict__ tabB, const float* __restrict__ scale, int n_slots,
                                   int tab_stride, int M, const __half** rowA, const __half** rowB, float* rowscale) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= CHAIN_MAX_ROWS * tab_stride) return;
  const int m = i / tab_stride, p = i % tab_stride;
  const int ad = (m < M && adapter_idx != nullptr) ? adapter_idx[m] : -1;
  const bool ok = ad >= 0 && ad < n_slots;
  rowA[i] = ok ? tabA[(size_t)ad * tab_stride + p] : nullptr;
  rowB[i] = ok ? tabB[(size_t)ad * tab_stride + p] : nullptr;
  if (p == 0) rowscale[m] = ok ? scale[ad] : 0.f;
}

cudaError_t launch_lean_rowptr(const int32_t* adapter_idx, const __half* const* tabA, const __half* const* tabB, const float* scale,
                               int n_slots, int tab_stride, int M, const __half** rowA, const __half** rowB, float* rowscale,
                               cudaStream_t st) {
  const int total = CHAIN_MAX_ROWS * tab_stride;
  lean_rowptr_kernel<<<(total + 255) / 256, 256, 0, st>>>(adapter_idx, tabA, tabB, scale, n_slots, tab_stride, M, rowA, rowB, rowscale);
  return cudaGetLastError();
}

bool lean_shapes_ok(int d_model, int d_ffn, int Nq, int Nkv, int rank) {
  // whole 16-column tiles, rows cut into 8-element pieces, T of a row within the kernels' shared arrays
  return d_model % 64 == 0 && d_ffn % 64 == 0 && Nq % 64 == 0 && Nkv % 16 == 0 && rank <= 64 && d_model <= 16384;
}

cudaError_t launch_lean_embed(const LeanArgs& a, const StepPhase& ph, const int32_t* tokens, const __half* embed, int vocab,
                              const __half* hidden_in, int* status, cudaStream_t st) {
  // a warp per (segment, rank index, 1024-element piece): enough CTAs per row to give every item its own warp
  const int items = (a.adapter_idx != nullptr ? ph.next_nseg * a.rank : 0) * (ph.pad_ ? 1 : (ph.N + 1023) / 1024);
  const int gy = items <= LN_WARPS ? 1 : (items + LN_WARPS - 1) / LN_WARPS > 32 ? 32 : (items + LN_WARPS - 1) / LN_WARPS;
  lean_embed_kernel<<<dim3((unsigned)a.M, (unsigned)gy), LN_THREADS, (size_t)ph.N * sizeof(__half), st>>>(a, ph, tokens, embed, vocab, hidden_in, status);
  return cudaGetLastError();
}

template <bool TRACE>
static cudaError_t init_lean_variant() {
  // room for the adapter slices at rank 64: 5 x 16 KB
  cudaError_t e = cudaFuncSetAttribute(lean_gemm_kernel<1, 8, TRACE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(lean_gemm_kernel<1, 16, TRACE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(lean_lmhead_kernel<LN_WARPS, TRACE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lm_smem_bytes(LN_THREADS));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(lean_gemm_kernel<2, 8, TRACE>, cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
}
cudaError_t init_lean() {
  const cudaError_t e = init_lean_variant<false>();
  return e != cudaSuccess ? e : init_lean_variant<true>();
}

template <bool TRACE>
static cudaError_t launch_lean_gemm_variant(const LeanArgs& a, const StepPhase& ph, cudaStream_t st) {
  const int tiles = ph.N / TILE_N, mode = ph.mode;
  // B slices of up to two tiles and A slices of up to three consuming segments, 8 rows x rank x 16 columns each
  const size_t slice = (size_t)CHAIN_MAX_ROWS * (a.rank > 0 ? a.rank : 1) * 16 * sizeof(__half);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(mode == MODE_GATEUP ? tiles / 2 : tiles));
  const bool wide = mode != MODE_GATEUP && ph.K >= 4096 && tiles <= 148;   // a long K on few tiles: sixteen warps split it
  cfg.blockDim = dim3(wide ? 512 : LN_THREADS);
  cfg.dynamicSmemBytes = (mode == MODE_GATEUP ? 5 : 4) * slice;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start while the kernel before it drains
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // wide projections without adapters (the lm_head): persistent CTAs, two per SM, that loop over the column tiles
  static const int sms = [] { int d = 0, n = 0; cudaGetDevice(&d); cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, d); return n; }();
  if (mode == MODE_PLAIN && ph.epi == EPI_F32 && ph.lora_nseg == 0 && tiles >= 4 * sms && sms > 0 &&
      (ph.K / TILE_K + LN_WARPS - 1) / LN_WARPS <= LM_PF) {
    cfg.gridDim = dim3((unsigned)(2 * sms < tiles ? 2 * sms : tiles));
    cfg.blockDim = dim3(LN_THREADS);
    cfg.dynamicSmemBytes = lm_smem_bytes(LN_THREADS);
    return cudaLaunchKernelEx(&cfg, lean_lmhead_kernel<LN_WARPS, TRACE>, a, ph);
  }
  if (mode == MODE_GATEUP) return cudaLaunchKernelEx(&cfg, lean_gemm_kernel<2, 8, TRACE>, a, ph);
  if (wide) return cudaLaunchKernelEx(&cfg, lean_gemm_kernel<1, 16, TRACE>, a, ph);
  return cudaLaunchKernelEx(&cfg, lean_gemm_kernel<1, 8, TRACE>, a, ph);
}

// (a.trace0 set: the instantiations that stamp the step's timeline)
cudaError_t launch_lean_gemm(const LeanArgs& a, const StepPhase& ph, cudaStream_t st) {
  return a.trace0 != nullptr ? launch_lean_gemm_variant<true>(a, ph, st) : launch_lean_gemm_variant<false>(a, ph, st);
}

}  // namespace mlora
