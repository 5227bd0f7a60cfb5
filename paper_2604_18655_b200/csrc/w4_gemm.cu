// INT4 group-quantised GEMM for few rows with the per-row LoRA expand fused in (paper Eq. 1-4,
// Sec. 3.2 approach (c), Sec. 3.3): y[m] = h[m] Wdeq + T[m] B_a(m), where T = (alpha/r) h A_a^T comes
// from the shrink kernel.  Weights stream once from HBM as 128-bit loads in fragment order, are
// dequantised in registers and multiplied on the tensor cores (mma.sync m16n8k16, weights as the
// 16-wide operand, the rows as the 8-wide one).  Work is split over output blocks and over K; split
// results are combined in a fixed order by the last CTA to arrive, which also runs the epilogue.
#include "common.cuh"

namespace mlora {

// ----------------------------------------------------------------------------- repack (create time)
// One thread per (tile, lane): builds the lane's 16 bytes from the canonical nibbles.
__global__ void repack_kernel(const uint8_t* __restrict__ qw, const __half* __restrict__ scales, const WLayout L,
                              unsigned char* __restrict__ w, int tile_off, int tile_stride) {
  const int K = L.K, N = L.N, G = L.G;
  const int KT = L.KT, NT = L.NT;
  const long long total = (long long)NT * KT * 32;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int lane = (int)(i & 31);
    const int kt = (int)((i >> 5) % KT);
    const int nt = (int)((i >> 5) / KT);
    const int g = lane >> 2, t = lane & 3;
    uint32_t words[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t wd = 0;
#pragma unroll
      for (int nib = 0; nib < 8; ++nib) {
        const int a = nib & 3, hi = nib >> 2;
        const int n = nt * TILE_N + g + 8 * (a & 1);
        const int k = kt * TILE_K + 16 * t + 4 * j + 2 * (a >> 1) + hi;
        const uint8_t byte = qw[(size_t)k * (N / 2) + (n >> 1)];
        const uint32_t u = (n & 1) ? (byte >> 4) : (byte & 0xF);
        wd |= u << (4 * nib);
      }
      words[j] = wd;
    }
    const int pt = tile_off + nt * tile_stride;
    unsigned char* unit = w + (size_t)pt * L.unit_bytes;
    *reinterpret_cast<uint4*>(unit + wl_tile_off(L, kt) + lane * 16) = make_uint4(words[0], words[1], words[2], words[3]);
  }
  // scales: one entry per (n-tile, group, g); a group lies inside one chunk
  const int KG = K / G;
  const long long stotal = (long long)KG * NT * 8;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < stotal;
       i += (long long)gridDim.x * blockDim.x) {
    const int g = (int)(i & 7);
    const int nt = (int)((i >> 3) % NT);
    const int kg = (int)((i >> 3) / NT);
    const __half lo = scales[(size_t)kg * N + nt * TILE_N + g];
    const __half hi = scales[(size_t)kg * N + nt * TILE_N + g + 8];
    const uint32_t v = (uint32_t)__half_as_ushort(lo) | ((uint32_t)__half_as_ushort(hi) << 16);
    const int pt = tile_off + nt * tile_stride;
    unsigned char* unit = w + (size_t)pt * L.unit_bytes;
    // every chunk the group covers gets a copy (a group longer than a chunk spans several chunks)
    const int kt_first = (kg * G) / TILE_K, kt_last = ((kg + 1) * G) / TILE_K - 1;
    for (int c = kt_first / CHUNK_KT; c <= kt_last / CHUNK_KT; ++c) {
      const int kt = max(kt_first, c * CHUNK_KT);
      *reinterpret_cast<uint32_t*>(unit + wl_scale_off(L, kt) + g * 4) = v;
    }
  }
}

cudaError_t launch_repack(const uint8_t* qweight, const __half* scales, int K, int N, int G, unsigned char* w,
                          int dst_tile_off, int dst_tile_stride, cudaStream_t st) {
  const WLayout L = make_wlayout(K, N, G);
  const long long total = (long long)L.NT * L.KT * 32;
  int blocks = (int)((total + 255) / 256);
  if (blocks > 148 * 16) blocks = 148 * 16;
  repack_kernel<<<blocks, 256, 0, st>>>(qweight, scales, L, w, dst_tile_off, dst_tile_stride);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- dequant through the GEMM's unpack path
// One warp per tile: same loads, same dequant8() as the GEMM; writes fp16 [K][N] of the logical matrix.
__global__ void dequant_kernel(const unsigned char* __restrict__ w, const WLayout L, int tile_off, int tile_stride,
                               __half* __restrict__ out) {
  const int KT = L.KT, NT = L.NT, N = L.N;
  const int lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long tile = blockIdx.x * (long long)(blockDim.x >> 5) + (threadIdx.x >> 5); tile < (long long)NT * KT;
       tile += warps) {
    const int kt = (int)(tile % KT), nt = (int)(tile / KT);
    const int pt = tile_off + nt * tile_stride;
    const unsigned char* unit = w + (size_t)pt * L.unit_bytes;
    const uint4 wv = ldg_stream(reinterpret_cast<const uint4*>(unit + wl_tile_off(L, kt)) + lane);
    const uint32_t sw = ldg_nc_u32(reinterpret_cast<const uint32_t*>(unit + wl_scale_off(L, kt)) + g);
    __half2 s_lo, s_hi;
    split_scales(sw, s_lo, s_hi);
    const uint32_t words[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t a[4];
      dequant8(words[j], s_lo, s_hi, a);
      const int k = kt * TILE_K + 16 * t + 4 * j;
      const int n = nt * TILE_N + g;
      const __half2 a0 = u32_as_h2(a[0]), a1 = u32_as_h2(a[1]), a2 = u32_as_h2(a[2]), a3 = u32_as_h2(a[3]);
      out[(size_t)(k + 0) * N + n] = __low2half(a0);
      out[(size_t)(k + 1) * N + n] = __high2half(a0);
      out[(size_t)(k + 0) * N + n + 8] = __low2half(a1);
      out[(size_t)(k + 1) * N + n + 8] = __high2half(a1);
      out[(size_t)(k + 2) * N + n] = __low2half(a2);
      out[(size_t)(k + 3) * N + n] = __high2half(a2);
      out[(size_t)(k + 2) * N + n + 8] = __low2half(a3);
      out[(size_t)(k + 3) * N + n + 8] = __high2half(a3);
    }
  }
}

// K, N: logical shape of the projection being written out; the physical matrix may hold other projections too
cudaError_t launch_dequant(const unsigned char* w, int K, int N, int G, int tile_off, int tile_stride, __half* out,
                           cudaStream_t st) {
  const WLayout L = make_wlayout(K, N, G);
  const long long tiles = (long long)L.NT * L.KT;
  int blocks = (int)((tiles + 7) / 8);
  if (blocks > 148 * 8) blocks = 148 * 8;
  dequant_kernel<<<blocks, 256, 0, st>>>(w, L, tile_off, tile_stride, out);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- GEMM
struct GemmPlan {
  int ksplit, kts_per_split, kc_tiles, m_blocks, n_blocks, mt;
  size_t smem;
};

template <int MT>
__global__ void __launch_bounds__(GEMM_THREADS) w4_gemm_kernel(const GemmArgs p, const int ksplit,
                                                               const int kts_per_split, const int kc_tiles) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int ROWS = MT * 8;
  const int KC = kc_tiles * TILE_K;
  const int hs_stride = KC + 8;                                  // halves; +16 B keeps 128-bit reads conflict-free
  __half* hs = reinterpret_cast<__half*>(smem_raw);
  float* tile = reinterpret_cast<float*>(smem_raw + (size_t)ROWS * hs_stride * sizeof(__half));
  const int tile_stride = GEMM_NB + 4;
  __shared__ int s_is_last;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int KT = p.K / TILE_K;
  const int NTILES = p.N / TILE_N;
  const int nt = blockIdx.x * GEMM_WARPS + warp;
  const bool active = nt < NTILES;
  const int split = blockIdx.y;
  const int m0 = blockIdx.z * ROWS;
  const int rows = min(ROWS, p.M - m0);
  const int kt_begin = split * kts_per_split;
  const int kt_end = min(KT, kt_begin + kts_per_split);
  const int nk = kt_end - kt_begin;

  float acc[MT][4];
#pragma unroll
  for (int i = 0; i < MT; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

  // weight / scale prefetch ring (independent of the activations)
  const WLayout L = make_wlayout(p.K, p.N, p.G);
  const unsigned char* unit = p.w + (size_t)(active ? nt : 0) * L.unit_bytes;
  auto w_at = [&](int kt) { return ldg_stream(reinterpret_cast<const uint4*>(unit + wl_tile_off(L, kt)) + lane); };
  auto s_at = [&](int kt) { return ldg_nc_u32(reinterpret_cast<const uint32_t*>(unit + wl_scale_off(L, kt)) + g); };
  uint4 wr[GEMM_PF];
  uint32_t sr[GEMM_PF];
#pragma unroll
  for (int i = 0; i < GEMM_PF; ++i) {
    if (active && i < nk) {
      wr[i] = w_at(kt_begin + i);
      sr[i] = s_at(kt_begin + i);
    } else {
      wr[i] = make_uint4(0, 0, 0, 0);
      sr[i] = 0;
    }
  }

  for (int k0 = 0; k0 < nk; k0 += GEMM_PF) {
    if (k0 % kc_tiles == 0) {
      // stage the next KC input features of the CTA's rows: fp16 [ROWS][KC], zero beyond the valid rows / K range
      __syncthreads();
      const int kbase = (kt_begin + k0) * TILE_K;
      const int kvalid = min(KC, kt_end * TILE_K - kbase);
      const int vec_per_row = KC / 8;
      for (int i = threadIdx.x; i < ROWS * vec_per_row; i += GEMM_THREADS) {
        const int r = i / vec_per_row, c = (i % vec_per_row) * 8;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < rows && c < kvalid) v = *reinterpret_cast<const uint4*>(p.h + (size_t)(m0 + r) * p.K + kbase + c);
        *reinterpret_cast<uint4*>(hs + (size_t)r * hs_stride + c) = v;
      }
      __syncthreads();
    }
    const int kl0 = (k0 % kc_tiles) * TILE_K;
#pragma unroll
    for (int i = 0; i < GEMM_PF; ++i) {
      if (k0 + i < nk) {             // uniform across the CTA
        if (active) {
          const uint4 w = wr[i];
          __half2 s_lo, s_hi;
          split_scales(sr[i], s_lo, s_hi);
          const int nxt = k0 + i + GEMM_PF;
          if (nxt < nk) {
            wr[i] = w_at(kt_begin + nxt);
            sr[i] = s_at(kt_begin + nxt);
          }
          uint32_t a[4][4];
          dequant8(w.x, s_lo, s_hi, a[0]);
          dequant8(w.y, s_lo, s_hi, a[1]);
          dequant8(w.z, s_lo, s_hi, a[2]);
          dequant8(w.w, s_lo, s_hi, a[3]);
          const __half* hrow = hs + kl0 + i * TILE_K + 16 * t;
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const uint4 b01 = *reinterpret_cast<const uint4*>(hrow + (size_t)(mt * 8 + g) * hs_stride);
            const uint4 b23 = *reinterpret_cast<const uint4*>(hrow + (size_t)(mt * 8 + g) * hs_stride + 8);
            mma_16816(acc[mt], a[0], b01.x, b01.y);
            mma_16816(acc[mt], a[1], b01.z, b01.w);
            mma_16816(acc[mt], a[2], b23.x, b23.y);
            mma_16816(acc[mt], a[3], b23.z, b23.w);
          }
        }
      }
    }
  }

  // accumulators -> shared tile [ROWS][GEMM_NB] (row-major, rows = activations rows)
  __syncthreads();
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) {
    const int r = mt * 8 + 2 * t;
    const int c = warp * TILE_N + g;
    tile[(size_t)(r + 0) * tile_stride + c] = acc[mt][0];
    tile[(size_t)(r + 1) * tile_stride + c] = acc[mt][1];
    tile[(size_t)(r + 0) * tile_stride + c + 8] = acc[mt][2];
    tile[(size_t)(r + 1) * tile_stride + c + 8] = acc[mt][3];
  }
  __syncthreads();

  const int nb0 = blockIdx.x * GEMM_NB;
  const int ncols = min(GEMM_NB, p.N - nb0);
  constexpr int QUADS = GEMM_NB / 4;

  // LoRA expand: this split's share of the rank-r sum, added to its partial tile (Eq. 1-4, second term)
  if (p.lora.adapter_idx != nullptr) {
    const int r = p.lora.rank;
    const int j0 = (int)(((long long)r * split) / ksplit), j1 = (int)(((long long)r * (split + 1)) / ksplit);
    if (j1 > j0) {
      for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
        const int m = i / QUADS, cq = (i % QUADS) * 4;
        if (cq >= ncols) continue;
        const int a = p.lora.adapter_idx[(m0 + m) / p.lora.rows_per_stream];
        if (a < 0 || a >= p.lora.n_slots) continue;
        int seg, col;
        map_col(p.mode, nb0 + cq, p.seg_n0, p.seg_n1, seg, col);
        const __half* B = p.lora.tabB[(size_t)a * p.lora.tab_stride + p.lora.seg[seg].proj_index];
        if (B == nullptr) continue;
        const int ldb = p.lora.seg[seg].n;
        const float* T = p.lora.T + ((size_t)(m0 + m) * p.lora.nseg + seg) * r;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
        for (int j = j0; j < j1; ++j) {
          const float tj = T[j];
          const uint2 bv = *reinterpret_cast<const uint2*>(B + (size_t)j * ldb + col);
          const float2 b01 = __half22float2(u32_as_h2(bv.x)), b23 = __half22float2(u32_as_h2(bv.y));
          s0 = fmaf(tj, b01.x, s0); s1 = fmaf(tj, b01.y, s1);
          s2 = fmaf(tj, b23.x, s2); s3 = fmaf(tj, b23.y, s3);
        }
        float* tp = tile + (size_t)m * tile_stride + cq;
        tp[0] += s0; tp[1] += s1; tp[2] += s2; tp[3] += s3;
      }
      __syncthreads();
    }
  }

  if (ksplit > 1) {
    // publish this split's tile, then the last CTA of the (n-block, m-block) sums all splits in split order
    float* mine = p.partial + (size_t)split * p.M * p.N;
    for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
      const int m = i / QUADS, cq = (i % QUADS) * 4;
      if (cq >= ncols) continue;
      const float* tp = tile + (size_t)m * tile_stride + cq;
      __stcg(reinterpret_cast<float4*>(mine + (size_t)(m0 + m) * p.N + nb0 + cq), make_float4(tp[0], tp[1], tp[2], tp[3]));
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned* ctr = p.counters + blockIdx.z * gridDim.x + blockIdx.x;
      const unsigned prev = atomicAdd(ctr, 1u);
      s_is_last = (prev == (unsigned)(ksplit - 1));
      if (s_is_last) *ctr = 0u;                                  // ready for the next launch on this stream
    }
    __syncthreads();
    if (!s_is_last) return;
    __threadfence();
    for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
      const int m = i / QUADS, cq = (i % QUADS) * 4;
      if (cq >= ncols) continue;
      float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int sp2 = 0; sp2 < ksplit; ++sp2) {
        const float4 v = __ldcg(reinterpret_cast<const float4*>(p.partial + ((size_t)sp2 * p.M + m0 + m) * p.N + nb0 + cq));
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
      float* tp = tile + (size_t)m * tile_stride + cq;
      tp[0] = s.x; tp[1] = s.y; tp[2] = s.z; tp[3] = s.w;
    }
    __syncthreads();
  }

  // epilogue on the complete sums
  if (p.epi == EPI_F32) {
    for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
      const int m = i / QUADS, cq = (i % QUADS) * 4;
      if (cq >= ncols) continue;
      const float* tp = tile + (size_t)m * tile_stride + cq;
      *reinterpret_cast<float4*>(p.out_f32 + (size_t)(m0 + m) * p.ldo + nb0 + cq) = make_float4(tp[0], tp[1], tp[2], tp[3]);
    }
  } else if (p.epi == EPI_RESID) {
    for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
      const int m = i / QUADS, cq = (i % QUADS) * 4;
      if (cq >= ncols) continue;
      const float* tp = tile + (size_t)m * tile_stride + cq;
      float4* xp = reinterpret_cast<float4*>(p.resid + (size_t)(m0 + m) * p.N + nb0 + cq);
      float4 x = *xp;
      x.x += tp[0]; x.y += tp[1]; x.z += tp[2]; x.w += tp[3];
      *xp = x;
    }
  } else {                                                       // EPI_SWIGLU: even 16-col tiles = gate, odd = up
    const int F = p.N / 2;
    for (int i = threadIdx.x; i < rows * QUADS; i += GEMM_THREADS) {
      const int m = i / QUADS, cq = (i % QUADS) * 4;
      if (cq >= ncols || ((cq >> 4) & 1)) continue;
      const float* gp = tile + (size_t)m * tile_stride + cq;
      const float* up = gp + 16;
      const int f = (((nb0 + cq) >> 5) << 4) | (cq & 15);
      __half2 o01, o23;
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = gp[e] / (1.f + __expf(-gp[e])) * up[e];
      o01 = __floats2half2_rn(v[0], v[1]);
      o23 = __floats2half2_rn(v[2], v[3]);
      *reinterpret_cast<uint2*>(p.out_f16 + (size_t)(m0 + m) * F + f) = make_uint2(h2_as_u32(o01), h2_as_u32(o23));
    }
  }
}

static int pick_mt(int M) {
  int mt = 1;
  while (mt < GEMM_MAX_MT && mt * 8 < M) mt *= 2;
  return mt;
}

static GemmPlan make_plan(int K, int N, int M, size_t partial_capacity) {
  GemmPlan pl;
  pl.mt = pick_mt(M);
  const int rows = pl.mt * 8;
  pl.m_blocks = (M + rows - 1) / rows;
  pl.n_blocks = (N + GEMM_NB - 1) / GEMM_NB;
  const int KT = K / TILE_K;
  // enough CTAs for ~4 per SM on 148 SMs, but never fewer than GEMM_PF/2 k-tiles per split
  const int target = 148 * 4;
  int ksplit = target / (pl.n_blocks * pl.m_blocks);
  if (ksplit < 1) ksplit = 1;
  int max_split = KT / 4;
  if (max_split < 1) max_split = 1;
  if (ksplit > max_split) ksplit = max_split;
  while (ksplit > 1 && (size_t)ksplit * M * N > partial_capacity) --ksplit;
  pl.kts_per_split = (KT + ksplit - 1) / ksplit;
  pl.ksplit = (KT + pl.kts_per_split - 1) / pl.kts_per_split;
  // K chunk staged in shared memory: multiple of GEMM_PF tiles, bounded by ~64 KB of activations
  int kc = (pl.kts_per_split + GEMM_PF - 1) / GEMM_PF * GEMM_PF;
  const int max_kc = ((64 * 1024) / (rows * 2 * TILE_K)) / GEMM_PF * GEMM_PF;
  if (kc > max_kc) kc = max_kc < GEMM_PF ? GEMM_PF : max_kc;
  pl.kc_tiles = kc;
  pl.smem = (size_t)rows * (kc * TILE_K + 8) * sizeof(__half) + (size_t)rows * (GEMM_NB + 4) * sizeof(float);
  return pl;
}

int gemm_pick_split(int K, int N, int M, size_t partial_capacity) { return make_plan(K, N, M, partial_capacity).ksplit; }

template <int MT>
static cudaError_t launch_mt(const GemmArgs& a, const GemmPlan& pl, cudaStream_t st) {
  dim3 grid(pl.n_blocks, pl.ksplit, pl.m_blocks);
  w4_gemm_kernel<MT><<<grid, GEMM_THREADS, pl.smem, st>>>(a, pl.ksplit, pl.kts_per_split, pl.kc_tiles);
  return cudaGetLastError();
}

template <int MT>
static cudaError_t set_attr() {
  return cudaFuncSetAttribute(w4_gemm_kernel<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
}

cudaError_t init_gemm() {
  cudaError_t e;
  if ((e = set_attr<1>()) != cudaSuccess) return e;
  if ((e = set_attr<2>()) != cudaSuccess) return e;
  if ((e = set_attr<4>()) != cudaSuccess) return e;
  if ((e = set_attr<8>()) != cudaSuccess) return e;
  return set_attr<16>();
}

cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st) {
  const GemmPlan pl = make_plan(a.K, a.N, a.M, a.partial_capacity);
  switch (pl.mt) {
    case 1: return launch_mt<1>(a, pl, st);
    case 2: return launch_mt<2>(a, pl, st);
    case 4: return launch_mt<4>(a, pl, st);
    case 8: return launch_mt<8>(a, pl, st);
    default: return launch_mt<16>(a, pl, st);
  }
}

}  // namespace mlora
