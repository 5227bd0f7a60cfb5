// Decode / tree-verify attention over one shared prompt KV segment plus one private segment per stream
// (Sec. 3.4, App. A.1: a stream's rows see the prefill segment and their own segment only) with the DS2D
// tree-ancestor mask on the rows being verified (Sec. 3.5, App. A.2).  No mask tensor exists: stream
// isolation is the addressing, the tree mask is one 64-bit word per row.
//
// Split-K online softmax: the key range is cut into chunks; a CTA takes (kv head, chunk, block of 64 query
// rows) and produces un-normalised partial outputs with their running max and sum; a merge kernel combines
// the chunks of a row by log-sum-exp.  A shared-prefix chunk is loaded once and used by the rows of ALL
// streams and all query heads of the kv head; an own-segment chunk is used by that stream's rows.
// QK^T and PV run on the tensor cores (mma.sync m16n8k16, fp32 accumulate), K/V tiles are staged through
// shared memory with a two-stage cp.async pipeline.
#include <cuda.h>
#include <cudaTypedefs.h>

#include "pipe.cuh"

namespace mlora {

constexpr int ATT_WARPS = 4;
constexpr int ATT_THREADS = ATT_WARPS * 32;
constexpr int ATT_ROWS = ATT_WARPS * 16;   // query rows per CTA
constexpr int ATT_KEYS = 32;               // keys per pipeline tile

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sa), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(sa));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem) {
  const uint32_t sa = (uint32_t)__cvta_generic_to_shared(smem);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(sa));
}

struct AttnItem {
  int is_own, s, chunk, row_block;
};

__device__ __forceinline__ AttnItem decode_item(const AttnArgs& p, int item, int rb_all, int rb_own) {
  AttnItem it;
  const int n_prefix_items = p.n_prefix_chunks * rb_all;
  if (item < n_prefix_items) {
    it.is_own = 0; it.s = 0;
    it.chunk = item / rb_all;
    it.row_block = item % rb_all;
  } else {
    item -= n_prefix_items;
    it.is_own = 1;
    it.row_block = item % rb_own;
    item /= rb_own;
    it.chunk = item % p.n_own_chunks;
    it.s = item / p.n_own_chunks;
  }
  return it;
}

template <int HD>
__device__ __forceinline__ void attn_partial_body(const AttnArgs& p, const int rb_all, const int rb_own,
                                                  const float scale_log2) {
  constexpr int STRIDE = HD + 8;                      // halves per shared-memory row
  constexpr int KSTEPS = HD / 16;
  constexpr int DT = HD / 8;                          // output n8-tiles
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* Qs = reinterpret_cast<__half*>(smem_raw);                   // [ATT_ROWS][STRIDE]
  __half* Ks = Qs + ATT_ROWS * STRIDE;                                // [2][ATT_KEYS][STRIDE]
  __half* Vs = Ks + 2 * ATT_KEYS * STRIDE;                            // [2][ATT_KEYS][STRIDE]

  const int kh = blockIdx.y;
  const int g_heads = p.Hq / p.Hkv;
  const bool fused = p.qkv_f32 != nullptr;
  const AttnItem it = decode_item(p, blockIdx.x, rb_all, rb_own);
  const int rows_per_stream = p.T * g_heads;
  const int R_all = p.n * rows_per_stream;

  int key_begin, key_end, S = 0;
  const __half *kbase, *vbase;
  int row_lo, row_hi;                                                  // virtual rows [row_lo, row_hi) within the kv head
  if (!it.is_own) {
    key_begin = it.chunk * p.prefix_chunk;
    key_end = min(p.P, key_begin + p.prefix_chunk);
    kbase = p.prefix_k + (size_t)kh * p.prefix_head_stride;
    vbase = p.prefix_v + (size_t)kh * p.prefix_head_stride;
    row_lo = it.row_block * ATT_ROWS;
    row_hi = min(R_all, row_lo + ATT_ROWS);
  } else {
    S = p.suffix_len[it.s];
    key_begin = it.chunk * p.own_chunk;
    key_end = min(S + p.T, key_begin + p.own_chunk);
    kbase = p.own_k + (size_t)it.s * p.own_stream_stride + (size_t)kh * p.own_head_stride;
    vbase = p.own_v + (size_t)it.s * p.own_stream_stride + (size_t)kh * p.own_head_stride;
    row_lo = it.s * rows_per_stream + it.row_block * ATT_ROWS;
    row_hi = min((it.s + 1) * rows_per_stream, row_lo + ATT_ROWS);
  }
  if (key_begin >= key_end) return;                                    // nothing here (merge skips this slot too)
  const int slot = it.is_own ? p.n_prefix_chunks + it.chunk : it.chunk;
  const int slots = p.n_prefix_chunks + p.n_own_chunks;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int n_tiles = (key_end - key_begin + ATT_KEYS - 1) / ATT_KEYS;

  auto load_kv_tile = [&](int tile, int stage) {
    const int k0 = key_begin + tile * ATT_KEYS;
    __half* kd = Ks + (size_t)stage * ATT_KEYS * STRIDE;
    __half* vd = Vs + (size_t)stage * ATT_KEYS * STRIDE;
    constexpr int VPR = HD / 8;                                        // 16-byte pieces per row
    for (int i = threadIdx.x; i < ATT_KEYS * VPR; i += ATT_THREADS) {
      const int r = i / VPR, c = (i % VPR) * 8;
      const int key = k0 + r;
      if (key >= key_end) {
        // rows past the end of the chunk: zeros (their scores are masked; a zero V row keeps 0 * v finite)
        *reinterpret_cast<uint4*>(kd + (size_t)r * STRIDE + c) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(vd + (size_t)r * STRIDE + c) = make_uint4(0, 0, 0, 0);
      } else if (fused && it.is_own && key >= S) {
        // a row of this pass: not in the cache yet -- build it from the projections (k rotated), use it, and let
        // the first row block of the chunk append it to the stream's own segment
        const int m = it.s * p.T + (key - S);
        const float* row = p.qkv_f32 + (size_t)m * (size_t)((p.Hq + 2 * p.Hkv) * HD);
        const float2* cs = p.cs_table + (size_t)(p.pos_base + S + p.depth[m]) * (HD / 2);
        const uint4 kv8 = head_piece_f16(row + (size_t)(p.Hq + kh) * HD, c, HD, cs);
        const uint4 vv8 = head_piece_f16(row + (size_t)(p.Hq + p.Hkv + kh) * HD, c, HD, nullptr);
        *reinterpret_cast<uint4*>(kd + (size_t)r * STRIDE + c) = kv8;
        *reinterpret_cast<uint4*>(vd + (size_t)r * STRIDE + c) = vv8;
        if (it.row_block == 0) {
          *reinterpret_cast<uint4*>(const_cast<__half*>(kbase) + (size_t)key * HD + c) = kv8;
          *reinterpret_cast<uint4*>(const_cast<__half*>(vbase) + (size_t)key * HD + c) = vv8;
        }
      } else {
        cp_async16(kd + (size_t)r * STRIDE + c, kbase + (size_t)key * HD + c);
        cp_async16(vd + (size_t)r * STRIDE + c, vbase + (size_t)key * HD + c);
      }
    }
  };

  load_kv_tile(0, 0);
  cp_async_commit();

  // query rows of this block -> shared memory (zero beyond the block's rows)
  {
    constexpr int VPR = HD / 8;
    for (int i = threadIdx.x; i < ATT_ROWS * VPR; i += ATT_THREADS) {
      const int r = i / VPR, c = (i % VPR) * 8;
      const int v = row_lo + r;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (v < row_hi) {
        const int m = v / g_heads, j = v % g_heads;
        if (fused) {
          const float* row = p.qkv_f32 + (size_t)m * (size_t)((p.Hq + 2 * p.Hkv) * HD);
          const float2* cs = p.cs_table + (size_t)(p.pos_base + p.suffix_len[m / p.T] + p.depth[m]) * (HD / 2);
          val = head_piece_f16(row + (size_t)(kh * g_heads + j) * HD, c, HD, cs);
        } else {
          val = *reinterpret_cast<const uint4*>(p.q + ((size_t)m * p.Hq + kh * g_heads + j) * HD + c);
        }
      }
      *reinterpret_cast<uint4*>(Qs + (size_t)r * STRIDE + c) = val;
    }
  }
  __syncthreads();

  const bool warp_active = (row_lo + warp * 16) < row_hi;
  uint32_t qf[KSTEPS][4];
  if (warp_active) {
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      const int mi = lane >> 3, r = lane & 7;
      ldmatrix_x4(qf[ks], Qs + (size_t)(warp * 16 + (mi & 1) * 8 + r) * STRIDE + ks * 16 + (mi >> 1) * 8);
    }
  }

  // per-row tree masks (own segment only): rows g and g+8 of the warp's tile
  unsigned long long anc0 = ~0ull, anc1 = ~0ull;
  int tq0 = -1, tq1 = -1;                                              // causal passes: the rows' own indices
  if (it.is_own) {
    const int v0 = row_lo + warp * 16 + g, v1 = v0 + 8;
    if (p.causal) {
      tq0 = (v0 < row_hi) ? (v0 / g_heads) % p.T : -1;
      tq1 = (v1 < row_hi) ? (v1 / g_heads) % p.T : -1;
    } else {
      anc0 = (v0 < row_hi) ? p.anc[v0 / g_heads] : 0ull;               // v / g_heads = global row m = s*T + t
      anc1 = (v1 < row_hi) ? p.anc[v1 / g_heads] : 0ull;
    }
  }

  float o[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  for (int tile = 0; tile < n_tiles; ++tile) {
    const int stage = tile & 1;
    if (tile + 1 < n_tiles) {
      load_kv_tile(tile + 1, stage ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    if (warp_active) {
      const __half* kt = Ks + (size_t)stage * ATT_KEYS * STRIDE;
      const __half* vt = Vs + (size_t)stage * ATT_KEYS * STRIDE;
      float sacc[ATT_KEYS / 8][4];
#pragma unroll
      for (int nt = 0; nt < ATT_KEYS / 8; ++nt) {
        sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ks += 2) {
          uint32_t kb[4];
          const int mi = lane >> 3, r = lane & 7;
          ldmatrix_x4(kb, kt + (size_t)(nt * 8 + r) * STRIDE + ks * 16 + mi * 8);
          mma_16816(sacc[nt], qf[ks], kb[0], kb[1]);
          mma_16816(sacc[nt], qf[ks + 1], kb[2], kb[3]);
        }
      }
      // scale, mask, running max
      const int k0 = key_begin + tile * ATT_KEYS;
      float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
      for (int nt = 0; nt < ATT_KEYS / 8; ++nt) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int key = k0 + nt * 8 + 2 * t + (e & 1);
          bool ok = key < key_end;
          if (it.is_own && key >= S) {
            if (p.causal) {
              ok = ok && (key - S) <= ((e & 2) ? tq1 : tq0);
            } else {
              const unsigned long long a = (e & 2) ? anc1 : anc0;
              ok = ok && ((a >> (key - S)) & 1ull);
            }
          }
          const float v = ok ? sacc[nt][e] * scale_log2 : -INFINITY;
          sacc[nt][e] = v;
          mx[e >> 1] = fmaxf(mx[e >> 1], v);
        }
      }
      float corr[2], msafe[2];
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
        mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
        const float mnew = fmaxf(mrow[h], mx[h]);
        msafe[h] = (mnew == -INFINITY) ? 0.f : mnew;
        corr[h] = exp2f(mrow[h] - msafe[h]);                           // mrow = -inf -> 0
        mrow[h] = mnew;
      }
      float ls[2] = {0.f, 0.f};
      uint32_t pf[ATT_KEYS / 16][4];
#pragma unroll
      for (int nt = 0; nt < ATT_KEYS / 8; ++nt) {
        const float p0 = exp2f(sacc[nt][0] - msafe[0]), p1 = exp2f(sacc[nt][1] - msafe[0]);
        const float p2 = exp2f(sacc[nt][2] - msafe[1]), p3 = exp2f(sacc[nt][3] - msafe[1]);
        ls[0] += p0 + p1;
        ls[1] += p2 + p3;
        pf[nt >> 1][(nt & 1) * 2 + 0] = h2_as_u32(__floats2half2_rn(p0, p1));
        pf[nt >> 1][(nt & 1) * 2 + 1] = h2_as_u32(__floats2half2_rn(p2, p3));
      }
#pragma unroll
      for (int h = 0; h < 2; ++h) lrow[h] = lrow[h] * corr[h] + ls[h];
#pragma unroll
      for (int dt = 0; dt < DT; ++dt) {
        o[dt][0] *= corr[0]; o[dt][1] *= corr[0];
        o[dt][2] *= corr[1]; o[dt][3] *= corr[1];
      }
#pragma unroll
      for (int kk = 0; kk < ATT_KEYS / 16; ++kk) {
#pragma unroll
        for (int dt = 0; dt < DT; dt += 2) {
          uint32_t vb[4];
          const int mi = lane >> 3, r = lane & 7;
          ldmatrix_x4_trans(vb, vt + (size_t)(kk * 16 + (mi & 1) * 8 + r) * STRIDE + (dt + (mi >> 1)) * 8);
          mma_16816(o[dt], pf[kk], vb[0], vb[1]);
          mma_16816(o[dt + 1], pf[kk], vb[2], vb[3]);
        }
      }
    }
    __syncthreads();                                                   // stage may be overwritten next iteration
  }

  if (!warp_active) return;
  // partial results: un-normalised output, running max (log2 domain) and the lane-group's partial sum
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const int v = row_lo + warp * 16 + g + 8 * h;
    if (v >= row_hi) continue;
    const size_t idx = ((size_t)kh * R_all + v) * slots + slot;
    float* po = p.part_o + idx * HD;
#pragma unroll
    for (int dt = 0; dt < DT; ++dt)
      *reinterpret_cast<float2*>(po + dt * 8 + 2 * t) = make_float2(o[dt][2 * h], o[dt][2 * h + 1]);
    if (t == 0) *reinterpret_cast<float2*>(p.part_ml + idx * 2) = make_float2(mrow[h], lrow[h]);
  }
}

// log-sum-exp merge of the chunks of virtual row v (row m, query head hq) of kv head kh by one warp.  The lanes
// take the chunks' (max, sum) pairs side by side; the weighted sum over chunks runs in chunk order with
// independent loads.
template <int FAST>
__device__ __forceinline__ void merge_row_fast(const AttnArgs& p, size_t base, int n_valid, __half* out, int lane) {
  // one round trip: every load is issued before the first use; the partial outputs of FAST chunks sit in registers
  const int hd = p.hd;
  float2 ml = make_float2(-INFINITY, 0.f);
  if (lane < n_valid) ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (base + lane) * 2));
  float po[FAST][4];
#pragma unroll
  for (int i = 0; i < FAST; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e)
      po[i][e] = (i < n_valid && e * 32 + lane < hd) ? __ldcg(p.part_o + (base + i) * hd + e * 32 + lane) : 0.f;
  float mmax = ml.x;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));
  const float wgt = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mmax);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float L = 0.f;
#pragma unroll
  for (int i = 0; i < FAST; ++i) {                                     // fixed order: chunk 0, 1, ...
    const float wi = __shfl_sync(0xffffffffu, wgt, i);
    L = fmaf(wi, __shfl_sync(0xffffffffu, ml.y, i), L);
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = fmaf(wi, po[i][e], acc[e]);
  }
  const float inv = 1.f / L;
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (e * 32 + lane < hd) out[e * 32 + lane] = __float2half_rn(acc[e] * inv);
}

__device__ __forceinline__ void merge_row(const AttnArgs& p, int kh, int v, int m, int hq, int lane) {
  const int g_heads = p.Hq / p.Hkv;
  const int R_all = p.n * p.T * g_heads;
  const int slots = p.n_prefix_chunks + p.n_own_chunks;
  const int s = m / p.T;
  // (no or a single own chunk: no need to wait for the suffix length)
  const int own_valid = p.n_own_chunks <= 1 ? p.n_own_chunks : min(p.n_own_chunks, (p.suffix_len[s] + p.T + p.own_chunk - 1) / p.own_chunk);
  const int n_valid = p.n_prefix_chunks + own_valid;
  const size_t base = ((size_t)kh * R_all + v) * slots;
  const int hd = p.hd;
  __half* out = p.out + ((size_t)m * p.Hq + hq) * hd;
  if (hd <= 128) {
    if (n_valid <= 12) { merge_row_fast<12>(p, base, n_valid, out, lane); return; }
    if (n_valid <= 24) { merge_row_fast<24>(p, base, n_valid, out, lane); return; }
  }
  float mmax = -INFINITY;
  for (int i = lane; i < n_valid; i += 32) mmax = fmaxf(mmax, __ldcg(p.part_ml + (base + i) * 2));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, o));
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float L = 0.f;
  for (int i0 = 0; i0 < n_valid; i0 += 32) {
    // lane i0 + lane holds the weight and the sum of its chunk
    float wgt = 0.f, lsum = 0.f;
    if (i0 + lane < n_valid) {
      const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (base + i0 + lane) * 2));
      wgt = (ml.x == -INFINITY) ? 0.f : exp2f(ml.x - mmax);
      lsum = ml.y;
    }
    const int cnt = min(32, n_valid - i0);
#pragma unroll 4
    for (int i = 0; i < cnt; ++i) {                                      // fixed order: chunk 0, 1, ...
      const float wi = __shfl_sync(0xffffffffu, wgt, i);
      L = fmaf(wi, __shfl_sync(0xffffffffu, lsum, i), L);
      const float* po = p.part_o + (base + i0 + i) * hd;
#pragma unroll
      for (int e = 0; e < 4; ++e)
        if (e * 32 + lane < hd) acc[e] = fmaf(wi, __ldcg(po + e * 32 + lane), acc[e]);
    }
  }
  const float inv = 1.f / L;
#pragma unroll
  for (int e = 0; e < 4; ++e)
    if (e * 32 + lane < hd) out[e * 32 + lane] = __float2half_rn(acc[e] * inv);
}

template <int HD>
__global__ void __launch_bounds__(ATT_THREADS, 3) attn_partial_kernel(const AttnArgs p, const int rb_all, const int rb_own,
                                                                  const float scale_log2) {
  attn_partial_body<HD>(p, rb_all, rb_own, scale_log2);
}

// One warp per (row, query head): log-sum-exp merge of the row's chunks, output in fp16.
__global__ void attn_merge_kernel(const AttnArgs p) {
  const int w = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  const int M = p.n * p.T;
  if (w >= M * p.Hq) return;
  const int m = w / p.Hq, hq = w % p.Hq;
  const int g_heads = p.Hq / p.Hkv;
  merge_row(p, hq / g_heads, m * g_heads + hq % g_heads, m, hq, lane);
}

// ----------------------------------------------------------------------------- single-pass decode attention
// One decode row per stream (T = 1) and a short context: a cluster of two CTAs per (kv head, stream) does the whole
// softmax (the CTAs take alternate tiles and the second hands its result to the first through distributed shared
// memory), so there are no partial results in global memory and no merge kernel.  The shared prefix is re-read by every stream's
// CTA, but from L2: HBM still sees it once.  The warps take 32-key tiles of (prefix ++ own segment) round-robin, each
// with its own double-buffered K/V tiles (cp.async) and its own online softmax over the kv head's query heads (one
// m16 tile, rows past the group zero); the warps' results are combined by log-sum-exp in shared memory.  The new
// K/V row of the pass is built from the projections (k rotated), used, and appended to the cache by the warp whose
// tile holds it.
constexpr int DEC_KEYS = 32;
constexpr int DEC_SPLIT = 2;                 // CTAs (one cluster) that share the tiles of a (kv head, stream)
__host__ __device__ constexpr int dec_warps(int hd) { return hd == 64 ? 8 : 4; }
__host__ __device__ constexpr size_t dec_smem_bytes(int hd) {
  return (size_t)16 * (hd + 8) * 2 + (size_t)dec_warps(hd) * 4 * DEC_KEYS * (hd + 8) * 2 +
         (size_t)dec_warps(hd) * 16 * (hd + 2) * 4 + (size_t)16 * (hd + 2) * 4 + (size_t)2 * hd * 2;
}

// (TRACE: the instantiation that stamps a traced step's timeline -- thread 0 of the first CTA writes the GPU's global
// nanosecond timer to slots 0 start, 1 wait returned, 2 key tiles done, 3 end of its launch's row; every CTA's thread 0
// raises slot 4 to its own end)
__device__ __forceinline__ long long attn_now() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
template <bool TRACE>
__device__ __forceinline__ void attn_stamp(const AttnArgs& p, int slot) {
  if constexpr (TRACE) {
    if (threadIdx.x == 0) {
      if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) p.trace0[slot] = attn_now();
      if (slot == 3) atomicMax(reinterpret_cast<unsigned long long*>(p.trace0 + 4), (unsigned long long)attn_now());
    }
  }
}
template <int HD, bool TRACE>
__global__ void __launch_bounds__(dec_warps(HD) * 32) attn_decode_kernel(const AttnArgs p, const float scale_log2) {
  constexpr int W = dec_warps(HD), STRIDE = HD + 8, KSTEPS = HD / 16, DT = HD / 8, VPR = HD / 8;
  // (programmatic launches around this kernel: the kernel after it may start its own independent loads now; nothing
  // here is read before the kernel ahead has finished -- both are no-ops in ordinary launches)
  attn_stamp<TRACE>(p, 0);
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // first phase of the cluster barrier: "this CTA runs" (waited for before the peer's shared memory is written)
  asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __half* Qs = reinterpret_cast<__half*>(smem_raw);                       // [16][STRIDE]
  __half* tiles = Qs + 16 * STRIDE;                                       // [W][2 buffers][K, V][DEC_KEYS][STRIDE]
  float* part_o = reinterpret_cast<float*>(tiles + (size_t)W * 4 * DEC_KEYS * STRIDE);   // [W][16][HD]
  float* part_ml = part_o + (size_t)W * 16 * HD;                          // [W][16][2]
  float* xch = part_ml + (size_t)W * 16 * 2;                              // [16][HD + 2]: this CTA's result for its peer
  __half (*newkv)[HD] = reinterpret_cast<__half (*)[HD]>(xch + 16 * (HD + 2));   // [2][HD]: the pass's new K (rotated) and V rows
  __half* a_sl = reinterpret_cast<__half*>(xch + 16 * (HD + 2)) + 2 * HD;  // [o_rank][g_heads * HD]: the o adapter's A rows
  const int rank = blockIdx.z;                                            // position in the cluster (1, 1, DEC_SPLIT)
  auto tile_of = [&](int li) { return li * DEC_SPLIT + rank; };          // the CTA's li-th tile

  const int kh = blockIdx.x, s = blockIdx.y;
  const int g_heads = p.Hq / p.Hkv;
  const bool fused = p.qkv_f32 != nullptr;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int n_ptiles = (p.P + DEC_KEYS - 1) / DEC_KEYS;
  int S = 0, own_keys = 0, n_tiles = n_ptiles;                            // known once suffix_len has arrived
  const __half* pk = p.prefix_k + (size_t)kh * p.prefix_head_stride;
  const __half* pv = p.prefix_v + (size_t)kh * p.prefix_head_stride;
  __half* ok = const_cast<__half*>(p.own_k) + (size_t)s * p.own_stream_stride + (size_t)kh * p.own_head_stride;
  __half* ov = const_cast<__half*>(p.own_v) + (size_t)s * p.own_stream_stride + (size_t)kh * p.own_head_stride;
  const int m = s;                                                        // the stream's row (T = 1)
  const float* prow = fused ? p.qkv_f32 + (size_t)m * (size_t)((p.Hq + 2 * p.Hkv) * HD) : nullptr;
  const float2* cs = nullptr;

  __half* my_tiles = tiles + (size_t)warp * 4 * DEC_KEYS * STRIDE;
  // (new_row_later: the pass's new row is not there yet -- the caller puts it in with fill_new_row)
  auto load_tile = [&](int ti, int buf, bool new_row_later = false) {
    __half* kd = my_tiles + (size_t)buf * 2 * DEC_KEYS * STRIDE;
    __half* vd = kd + DEC_KEYS * STRIDE;
    const bool own = ti >= n_ptiles;
    const int k0 = (own ? ti - n_ptiles : ti) * DEC_KEYS;
    const int kend = own ? own_keys : p.P;
    const __half* kb = own ? ok : pk;
    const __half* vb = own ? ov : pv;
    if (k0 + DEC_KEYS <= kend && !(fused && own && S >= k0 && S < k0 + DEC_KEYS)) {
      // a full tile of cached rows: straight copies, the addresses stepped
      constexpr int RPI = 32 / VPR;                                       // rows covered by one pass of the warp
      const int r0 = lane / VPR, c = (lane % VPR) * 8;
      const __half* ks = kb + (size_t)(k0 + r0) * HD + c;
      const __half* vs = vb + (size_t)(k0 + r0) * HD + c;
      __half* kdp = kd + (size_t)r0 * STRIDE + c;
      __half* vdp = vd + (size_t)r0 * STRIDE + c;
#pragma unroll
      for (int it = 0; it < DEC_KEYS / RPI; ++it) {
        cp_async16(kdp + (size_t)it * RPI * STRIDE, ks + (size_t)it * RPI * HD);
        cp_async16(vdp + (size_t)it * RPI * STRIDE, vs + (size_t)it * RPI * HD);
      }
      cp_async_commit();
      return;
    }
    for (int i = lane; i < DEC_KEYS * VPR; i += 32) {
      const int r = i / VPR, c = (i % VPR) * 8, key = k0 + r;
      if (key >= kend) {
        *reinterpret_cast<uint4*>(kd + (size_t)r * STRIDE + c) = make_uint4(0, 0, 0, 0);
        *reinterpret_cast<uint4*>(vd + (size_t)r * STRIDE + c) = make_uint4(0, 0, 0, 0);
      } else if (fused && own && key == S) {
        // the pass's new row: built (rotated, appended to the cache) next to the query rows, copied from there
        if (!new_row_later) {
          *reinterpret_cast<uint4*>(kd + (size_t)r * STRIDE + c) = *reinterpret_cast<const uint4*>(&newkv[0][c]);
          *reinterpret_cast<uint4*>(vd + (size_t)r * STRIDE + c) = *reinterpret_cast<const uint4*>(&newkv[1][c]);
        }
      } else {
        cp_async16(kd + (size_t)r * STRIDE + c, kb + (size_t)key * HD + c);
        cp_async16(vd + (size_t)r * STRIDE + c, vb + (size_t)key * HD + c);
      }
    }
    cp_async_commit();
  };
  // the o projection's adapter rows over this kv head's features (first CTA of the cluster; immutable: asked for
  // ahead of everything; its cp.async group is the oldest, so every later wait covers it)
  const __half* oA = nullptr;
  if (p.o_tacc != nullptr && rank == 0) {
    const int ad = p.o_direct ? s : p.o_adapter_idx[s];
    oA = (ad >= 0 && ad < p.o_n_slots) ? p.o_tabA[(size_t)ad * p.o_tab_stride + p.o_proj_index] : nullptr;
    if (oA != nullptr) {
      const int feats = g_heads * HD, ld = p.Hq * HD, pieces = feats / 8;
      for (int i = threadIdx.x; i < p.o_rank * pieces; i += W * 32) {
        const int j = i / pieces, c = (i % pieces) * 8;
        cp_async16(a_sl + (size_t)j * feats + c, oA + (size_t)j * ld + (size_t)kh * feats + c);
      }
    }
    cp_async_commit();
  }
  // a warp whose first tile lies in the shared prefix starts it before anything that depends on the stream
  if (tile_of(warp) < n_ptiles) load_tile(tile_of(warp), 0);
  // (programmatic launch: the shared prefix does not change in decode, and the suffix lengths were last written by the
  // step before this one, which an ordinary launch at the start of this step has waited for)
  S = p.suffix_len[s];
  if (fused && p.depth == nullptr) {
    // rows without a tree depth (plain decode): the rotation table row of the new position is known already -- asked
    // for now, so that the rotation behind the wait waits only for the projections
    cs = p.cs_table + (size_t)(p.pos_base + S) * (HD / 2);
    if (threadIdx.x < (HD / 2) * (int)sizeof(float2) / 128)
      asm volatile("prefetch.global.L1 [%0];" ::"l"(reinterpret_cast<const char*>(cs) + threadIdx.x * 128) : "memory");
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  attn_stamp<TRACE>(p, 1);
  own_keys = S + 1;                                                       // cached rows + this pass's row
  n_tiles = n_ptiles + (own_keys + DEC_KEYS - 1) / DEC_KEYS;
  if (fused && p.depth != nullptr) cs = p.cs_table + (size_t)(p.pos_base + S + p.depth[m]) * (HD / 2);
  // (the tile that holds the new row gets its cached rows now and the new row once that has been built: below, with
  // the query rows, so that the loads of all of them are in flight together)
  const int s_tile = fused ? n_ptiles + S / DEC_KEYS : -1;
  if (tile_of(warp) >= n_ptiles && tile_of(warp) < n_tiles) load_tile(tile_of(warp), 0, true);
  if (tile_of(warp + W) < n_tiles) load_tile(tile_of(warp + W), 1, true);
  // the warp's later tiles: ask for them in L2 now, so that their copies two iterations on do not wait for HBM
  if (lane == 0) {
    for (int li = warp + 2 * W; tile_of(li) < n_tiles; li += W) {
      const int ti = tile_of(li);
      const bool own = ti >= n_ptiles;
      const int k0 = (own ? ti - n_ptiles : ti) * DEC_KEYS;
      const int rows = min(DEC_KEYS, (own ? S : p.P) - k0);               // cached rows only
      if (rows <= 0) continue;
      const uint32_t bytes = (uint32_t)rows * HD * 2;
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"((own ? ok : pk) + (size_t)k0 * HD), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"((own ? ov : pv) + (size_t)k0 * HD), "r"(bytes) : "memory");
    }
  }

  // the group's query rows (rotated on load in fused mode), zero past the group
  for (int i = threadIdx.x; i < 16 * VPR; i += W * 32) {
    const int r = i / VPR, c = (i % VPR) * 8;
    uint4 val = make_uint4(0, 0, 0, 0);
    if (r < g_heads) {
      if (fused) val = head_piece_f16(prow + (size_t)(kh * g_heads + r) * HD, c, HD, cs);
      else val = *reinterpret_cast<const uint4*>(p.q + ((size_t)m * p.Hq + kh * g_heads + r) * HD + c);
    }
    *reinterpret_cast<uint4*>(Qs + (size_t)r * STRIDE + c) = val;
  }
  // the new K and V rows of this kv head, by the CTA whose tile they fall into (threads the query rows leave idle,
  // where there are any): rotated, appended to the stream's cache, kept for the tile
  if (fused && s_tile % DEC_SPLIT == rank) {
    const int base = (16 * VPR) % (W * 32);                              // first thread without a query piece in the last pass
    for (int i = (threadIdx.x - base + W * 32) % (W * 32); i < 2 * VPR; i += W * 32) {
      const int which = i / VPR, c = (i % VPR) * 8;
      const uint4 v8 = which == 0 ? head_piece_f16(prow + (size_t)(p.Hq + kh) * HD, c, HD, cs)
                                  : head_piece_f16(prow + (size_t)(p.Hq + p.Hkv + kh) * HD, c, HD, nullptr);
      *reinterpret_cast<uint4*>(&newkv[which][c]) = v8;
      *reinterpret_cast<uint4*>((which == 0 ? ok : ov) + (size_t)S * HD + c) = v8;
    }
  }
  __syncthreads();
  if (tile_of(warp) == s_tile || tile_of(warp + W) == s_tile) {
    __half* kd = my_tiles + (size_t)(tile_of(warp) == s_tile ? 0 : 1) * 2 * DEC_KEYS * STRIDE;
    const int r = S % DEC_KEYS;
    if (lane < 2 * VPR) {
      const int which = lane / VPR, c = (lane % VPR) * 8;
      *reinterpret_cast<uint4*>(kd + (size_t)which * DEC_KEYS * STRIDE + (size_t)r * STRIDE + c) = *reinterpret_cast<const uint4*>(&newkv[which][c]);
    }
  }
  uint32_t qf[KSTEPS][4];
#pragma unroll
  for (int ks = 0; ks < KSTEPS; ++ks) {
    const int mi = lane >> 3, r = lane & 7;
    ldmatrix_x4(qf[ks], Qs + (size_t)((mi & 1) * 8 + r) * STRIDE + ks * 16 + (mi >> 1) * 8);
  }

  float o[DT][4];
#pragma unroll
  for (int i = 0; i < DT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  int buf = 0;
  for (int li = warp; tile_of(li) < n_tiles; li += W, buf ^= 1) {
    const int ti = tile_of(li);
    if (tile_of(li + W) < n_tiles) cp_async_wait<1>();     // the next tile may still be in flight
    else cp_async_wait<0>();
    __syncwarp();
    const __half* kt = my_tiles + (size_t)buf * 2 * DEC_KEYS * STRIDE;
    const __half* vt = kt + DEC_KEYS * STRIDE;
    const bool own = ti >= n_ptiles;
    const int k0 = (own ? ti - n_ptiles : ti) * DEC_KEYS, kend = own ? own_keys : p.P;
    float sacc[DEC_KEYS / 8][4];
#pragma unroll
    for (int nt = 0; nt < DEC_KEYS / 8; ++nt) {
      sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KSTEPS; ks += 2) {
        uint32_t kb[4];
        const int mi = lane >> 3, r = lane & 7;
        ldmatrix_x4(kb, kt + (size_t)(nt * 8 + r) * STRIDE + ks * 16 + mi * 8);
        mma_16816(sacc[nt], qf[ks], kb[0], kb[1]);
        mma_16816(sacc[nt], qf[ks + 1], kb[2], kb[3]);
      }
    }
    float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
    for (int nt = 0; nt < DEC_KEYS / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = k0 + nt * 8 + 2 * t + (e & 1);
        const float v = key < kend ? sacc[nt][e] * scale_log2 : -INFINITY;
        sacc[nt][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
    float corr[2], msafe[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
      mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
      const float mnew = fmaxf(mrow[h], mx[h]);
      msafe[h] = (mnew == -INFINITY) ? 0.f : mnew;
      corr[h] = exp2f(mrow[h] - msafe[h]);
      mrow[h] = mnew;
    }
    float ls[2] = {0.f, 0.f};
    uint32_t pf[DEC_KEYS / 16][4];
#pragma unroll
    for (int nt = 0; nt < DEC_KEYS / 8; ++nt) {
      const float p0 = exp2f(sacc[nt][0] - msafe[0]), p1 = exp2f(sacc[nt][1] - msafe[0]);
      const float p2 = exp2f(sacc[nt][2] - msafe[1]), p3 = exp2f(sacc[nt][3] - msafe[1]);
      ls[0] += p0 + p1;
      ls[1] += p2 + p3;
      pf[nt >> 1][(nt & 1) * 2 + 0] = h2_as_u32(__floats2half2_rn(p0, p1));
      pf[nt >> 1][(nt & 1) * 2 + 1] = h2_as_u32(__floats2half2_rn(p2, p3));
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) lrow[h] = lrow[h] * corr[h] + ls[h];
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) {
      o[dt][0] *= corr[0]; o[dt][1] *= corr[0];
      o[dt][2] *= corr[1]; o[dt][3] *= corr[1];
    }
#pragma unroll
    for (int kk = 0; kk < DEC_KEYS / 16; ++kk) {
#pragma unroll
      for (int dt = 0; dt < DT; dt += 2) {
        uint32_t vb[4];
        const int mi = lane >> 3, r = lane & 7;
        ldmatrix_x4_trans(vb, vt + (size_t)(kk * 16 + (mi & 1) * 8 + r) * STRIDE + (dt + (mi >> 1)) * 8);
        mma_16816(o[dt], pf[kk], vb[0], vb[1]);
        mma_16816(o[dt + 1], pf[kk], vb[2], vb[3]);
      }
    }
    __syncwarp();                                        // every lane is done with the buffer: refill it
    if (tile_of(li + 2 * W) < n_tiles) load_tile(tile_of(li + 2 * W), buf);
  }

  attn_stamp<TRACE>(p, 2);
  // this warp's un-normalised output, running max (log2 domain) and sum for the group's rows
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
    const int r = g + 8 * h;
    if (r >= g_heads) continue;
    float* po = part_o + ((size_t)warp * 16 + r) * HD;
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) *reinterpret_cast<float2*>(po + dt * 8 + 2 * t) = make_float2(o[dt][2 * h], o[dt][2 * h + 1]);
    if (t == 0) *reinterpret_cast<float2*>(part_ml + ((size_t)warp * 16 + r) * 2) = make_float2(mrow[h], lrow[h]);
  }
  __syncthreads();
  // the CTA's result per (row, feature): running max, numerator, denominator over its warps (warp order: fixed)
  auto cta_result = [&](int r, int d, float& M, float& num, float& den) {
    M = -INFINITY;
#pragma unroll
    for (int w = 0; w < W; ++w) M = fmaxf(M, part_ml[((size_t)w * 16 + r) * 2]);
    num = 0.f; den = 0.f;
#pragma unroll
    for (int w = 0; w < W; ++w) {
      const float mw = part_ml[((size_t)w * 16 + r) * 2];
      if (mw == -INFINITY) continue;                       // a warp without tiles
      const float f = exp2f(mw - M);
      num += f * part_o[((size_t)w * 16 + r) * HD + d];
      den += f * part_ml[((size_t)w * 16 + r) * 2 + 1];
    }
  };
  // The second CTA of the cluster PUSHES its result into the first one's exchange area (distributed shared memory),
  // so that after the barrier the first CTA combines from its own shared memory and nothing of the second CTA's is
  // read any more: no barrier at the end.  Every thread of both CTAs takes both barrier phases (no early exit above).
  static_assert(DEC_SPLIT == 2, "one exchange area: one peer");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");       // (phase 1: the peer runs)
  float M_own = -INFINITY, num_own = 0.f, den_own = 0.f;                   // this thread's first element, ahead of the barrier
  if (rank != 0) {
    uint32_t dst;                                                          // rank 0's xch in the cluster's shared window
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(dst) : "r"((uint32_t)__cvta_generic_to_shared(xch)), "r"(0));
    auto push = [&](int idx, float v) { asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(dst + 4u * (uint32_t)idx), "f"(v) : "memory"); };
    for (int i = threadIdx.x; i < g_heads * HD; i += W * 32) {
      const int r = i / HD, d = i % HD;
      float M, num, den;
      cta_result(r, d, M, num, den);
      push(r * (HD + 2) + d, num);
      if (d == 0) { push(r * (HD + 2) + HD, M); push(r * (HD + 2) + HD + 1, den); }
    }
  } else if (threadIdx.x < g_heads * HD) {
    cta_result(threadIdx.x / HD, threadIdx.x % HD, M_own, num_own, den_own);
  }
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
  if (rank == 0) {
    for (int i = threadIdx.x; i < g_heads * HD; i += W * 32) {
      const int r = i / HD, d = i % HD;
      float M = M_own, num = num_own, den = den_own;
      if (i != (int)threadIdx.x) cta_result(r, d, M, num, den);
      if (M == -INFINITY) { num = 0.f; den = 0.f; }
      {
        const float num1 = xch[r * (HD + 2) + d], M1 = xch[r * (HD + 2) + HD], den1 = xch[r * (HD + 2) + HD + 1];
        if (M1 != -INFINITY) {                             // (a peer without tiles contributes nothing)
          const float Mn = fmaxf(M, M1);
          const float f0 = (M == -INFINITY) ? 0.f : exp2f(M - Mn), f1 = exp2f(M1 - Mn);
          num = f0 * num + f1 * num1;
          den = f0 * den + f1 * den1;
          M = Mn;
        }
      }
      const __half hv = __float2half_rn(den > 0.f ? num / den : 0.f);
      p.out[((size_t)m * p.Hq + kh * g_heads + r) * HD + d] = hv;
      Qs[(size_t)r * STRIDE + d] = hv;                     // (the query tile is long since in registers)
    }
    if (p.o_tacc != nullptr) {
      // partial shrink of the o projection's adapter (Eq. 1-4) over this kv head's output features of row m: rank
      // index j by warp; integer atomics on fixed-point sums, so the total does not depend on the arrival order
      cp_async_wait<0>();
      __syncthreads();
      if (oA != nullptr) {
        const int feats = g_heads * HD;
        for (int j = warp; j < p.o_rank; j += W) {
          const __half* arow = a_sl + (size_t)j * feats;
          float sum = 0.f;
          for (int i = lane * 2; i < feats; i += 64) {
            const float2 av = __half22float2(*reinterpret_cast<const __half2*>(arow + i));
            const float2 xv = __half22float2(*reinterpret_cast<const __half2*>(Qs + (size_t)(i / HD) * STRIDE + (i % HD)));
            sum = fmaf(xv.x, av.x, sum);
            sum = fmaf(xv.y, av.y, sum);
          }
#pragma unroll
          for (int o2 = 16; o2 > 0; o2 >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
          if (lane == 0) {
            const unsigned long long q = (unsigned long long)__float2ll_rn(sum * 4294967296.f);
            asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p.o_tacc + ((size_t)m * 3 + 0) * p.o_rank + j), "l"(q) : "memory");
          }
        }
      }
    }
  }
  attn_stamp<TRACE>(p, 3);
}


// ----------------------------------------------------------------------------- streaming decode attention
// One decode row per stream and a LONG shared prefix (Sec. 3.4, App. A.1: every stream's row attends to the same
// prefill segment): the prefix is cut into one chunk per SM and kv head, and the CTA of a chunk serves the rows of ALL
// streams and all query heads of the kv head (at most 32 rows = two m16 tiles), so the prefix crosses HBM and L2 once.
// A producer warp streams 64-key K and V tiles through a 4-stage ring with tiled TMA copies (tensor maps over the
// prefix, 128-byte swizzle, rows past the prefix zero-filled, completion on mbarriers); eight consumer warps take
// (row tile, 16 keys of the tile) each, with their own online softmax, and are combined by log-sum-exp in shared
// memory at the end of the chunk.  The first n * Hkv CTAs also take one (stream, kv head) own segment each, as further
// keys of their partial that only that stream's rows may see: its first two tiles are fetched with cp.async into the
// same swizzled layout while the prefix streams (the new row is built from the projections, rotated, and appended).
// Partial results per (row, chunk) go to the scratch that attn_merge_kernel combines.
constexpr int STR_KEYS = 64;
constexpr int STR_CWARPS = 8;
constexpr int STR_THREADS = (STR_CWARPS + 1) * 32;
constexpr int STR_STAGES = 4;
constexpr int STR_ROWS = 32;
constexpr int STR_OWN_TILES = 2;                          // own tiles fetched ahead, in shared memory of their own
constexpr long long STR_WAIT_CYCLES = 2000000000ll;       // ~1 s
__host__ __device__ constexpr size_t str_stage_bytes(int hd) { return (size_t)2 * STR_KEYS * hd * 2; }
__host__ __device__ constexpr size_t str_smem_bytes(int hd) {
  return 1024 + (STR_STAGES + STR_OWN_TILES) * str_stage_bytes(hd) + (size_t)STR_ROWS * (hd + 8) * 2 + 128;
}

__device__ __forceinline__ void tma_tile_3d(uint32_t dst, const void* tmap, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// byte offset of the 16-byte piece `piece` (0 .. hd/8 - 1) of row `row` in a [64][hd] tile stored as hd/64 column
// halves of [64 rows][128 bytes], each with the 128-byte swizzle (piece index xor row mod 8)
__device__ __forceinline__ uint32_t str_off(int row, int piece) {
  return (uint32_t)((piece >> 3) * (STR_KEYS * 128) + row * 128 + (((piece & 7) ^ (row & 7)) << 4));
}
// bounded mbarrier wait: false once the CTA has given up (the flag is shared; the first to run out sets the status)
__device__ __forceinline__ bool str_wait(uint32_t bar, uint32_t parity, volatile int* s_abort, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (int it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 127) == 127) {
      if (*s_abort) return false;
      if (clock64() - t0 > STR_WAIT_CYCLES) {
        *s_abort = 1;
        if (status) atomicCAS(status, 0, MLORA_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

// one warp: 16 query rows (fragments qf) against 16 keys (rows key16 .. key16+15 of the K and V tiles at kt / vt),
// online softmax update of (o, mrow, lrow).  n_valid = number of valid keys among the 16.
template <int HD>
__device__ __forceinline__ void str_tile16(const uint32_t (&qf)[HD / 16][4], uint32_t kt, uint32_t vt, int key16, int n_valid,
                                           bool row_lo_ok, bool row_hi_ok, float scale_log2, float (&o)[HD / 8][4],
                                           float (&mrow)[2], float (&lrow)[2]) {
  constexpr int KSTEPS = HD / 16, DT = HD / 8;
  const int lane = threadIdx.x & 31, t = lane & 3, mi = lane >> 3, r = lane & 7;
  float sacc[2][4];
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
    const int row = key16 + nt * 8 + r;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ks += 2) {
      uint32_t kb[4];
      asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                   : "=r"(kb[0]), "=r"(kb[1]), "=r"(kb[2]), "=r"(kb[3]) : "r"(kt + str_off(row, ks * 2 + mi)));
      mma_16816(sacc[nt], qf[ks], kb[0], kb[1]);
      mma_16816(sacc[nt], qf[ks + 1], kb[2], kb[3]);
    }
  }
  float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int key = nt * 8 + 2 * t + (e & 1);
      const float v = (key < n_valid && ((e & 2) ? row_hi_ok : row_lo_ok)) ? sacc[nt][e] * scale_log2 : -INFINITY;
      sacc[nt][e] = v;
      mx[e >> 1] = fmaxf(mx[e >> 1], v);
    }
  }
  float corr[2], msafe[2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
    mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
    const float mnew = fmaxf(mrow[h], mx[h]);
    msafe[h] = (mnew == -INFINITY) ? 0.f : mnew;
    corr[h] = exp2f(mrow[h] - msafe[h]);                               // both -inf: exp2(-inf) = 0 on zeros, harmless
    mrow[h] = mnew;
  }
  uint32_t pf[4];
  float ls[2] = {0.f, 0.f};
#pragma unroll
  for (int nt = 0; nt < 2; ++nt) {
    const float p0 = exp2f(sacc[nt][0] - msafe[0]), p1 = exp2f(sacc[nt][1] - msafe[0]);
    const float p2 = exp2f(sacc[nt][2] - msafe[1]), p3 = exp2f(sacc[nt][3] - msafe[1]);
    ls[0] += p0 + p1;
    ls[1] += p2 + p3;
    pf[nt * 2 + 0] = h2_as_u32(__floats2half2_rn(p0, p1));
    pf[nt * 2 + 1] = h2_as_u32(__floats2half2_rn(p2, p3));
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) lrow[h] = lrow[h] * corr[h] + ls[h];
#pragma unroll
  for (int dt = 0; dt < DT; ++dt) {
    o[dt][0] *= corr[0]; o[dt][1] *= corr[0];
    o[dt][2] *= corr[1]; o[dt][3] *= corr[1];
  }
#pragma unroll
  for (int dt = 0; dt < DT; dt += 2) {
    uint32_t vb[4];
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(vb[0]), "=r"(vb[1]), "=r"(vb[2]), "=r"(vb[3])
                 : "r"(vt + str_off(key16 + (mi & 1) * 8 + r, dt + (mi >> 1))));
    mma_16816(o[dt], pf, vb[0], vb[1]);
    mma_16816(o[dt + 1], pf, vb[2], vb[3]);
  }
}

// the consumer warps' partial results -> one (max, sum, numerator) per row, written to the scratch slot.
// Warp cw = row tile + 2 * key quarter; comb: [8 warps][16 rows][HD + 2] floats.
template <int HD>
__device__ __forceinline__ void str_combine_write(const AttnArgs& p, float* comb, int cw, const float (&o)[HD / 8][4],
                                                  const float (&mrow)[2], float (&lrow)[2], int kh, int v0, int n_rows,
                                                  int slot, int ctid) {
  constexpr int DT = HD / 8, CS = HD + 2;
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int g_heads = p.Hq / p.Hkv, R_all = p.n * g_heads, slots = p.n_prefix_chunks + p.n_own_chunks;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 1);
    lrow[h] += __shfl_xor_sync(0xffffffffu, lrow[h], 2);
  }
  float* mine = comb + (size_t)cw * 16 * CS;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float* row = mine + (size_t)(g + 8 * h) * CS;
#pragma unroll
    for (int dt = 0; dt < DT; ++dt) *reinterpret_cast<float2*>(row + dt * 8 + 2 * t) = make_float2(o[dt][2 * h], o[dt][2 * h + 1]);
    if (t == 0) { row[HD] = mrow[h]; row[HD + 1] = lrow[h]; }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
  for (int i = ctid; i < n_rows * (HD / 4); i += STR_CWARPS * 32) {
    const int r = i / (HD / 4), d = (i % (HD / 4)) * 4;
    const float* base = comb + (size_t)((r >> 4) * 16 + (r & 15)) * CS;   // key quarter 0 of the row's tile; quarter q: + 2 q warps
    float M = -INFINITY;
#pragma unroll
    for (int q = 0; q < 4; ++q) M = fmaxf(M, base[(size_t)(2 * q) * 16 * CS + HD]);
    float4 num = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
#pragma unroll
    for (int q = 0; q < 4; ++q) {                                          // fixed order
      const float* w = base + (size_t)(2 * q) * 16 * CS;
      const float mq = w[HD];
      const float f = (mq == -INFINITY) ? 0.f : exp2f(mq - M);
      num.x = fmaf(f, w[d], num.x); num.y = fmaf(f, w[d + 1], num.y);
      num.z = fmaf(f, w[d + 2], num.z); num.w = fmaf(f, w[d + 3], num.w);
      den = fmaf(f, w[HD + 1], den);
    }
    const size_t idx = ((size_t)kh * R_all + v0 + r) * slots + slot;
    *reinterpret_cast<float4*>(p.part_o + idx * HD + d) = num;
    if (d == 0) *reinterpret_cast<float2*>(p.part_ml + idx * 2) = make_float2(M, den);
  }
  asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
}

template <int HD>
__global__ void __launch_bounds__(STR_THREADS, 1)
attn_stream_kernel(const AttnArgs p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                   const float scale_log2) {
  constexpr int KSTEPS = HD / 16, DT = HD / 8, VPR = HD / 8, QSTRIDE = HD + 8;
  constexpr uint32_t TILE_BYTES = STR_KEYS * HD * 2;                      // one K (or V) tile
  constexpr uint32_t STAGE_BYTES = 2 * TILE_BYTES;
  extern __shared__ unsigned char smem_raw_[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw_) + 1023) & ~(uintptr_t)1023);
  unsigned char* ring = base;                                              // [STAGES][K tile, V tile]
  unsigned char* own_tiles_mem = ring + STR_STAGES * STAGE_BYTES;          // [OWN_TILES][K tile, V tile]
  __half* Qs = reinterpret_cast<__half*>(own_tiles_mem + STR_OWN_TILES * STAGE_BYTES);   // [32][QSTRIDE]
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<unsigned char*>(Qs) + (size_t)STR_ROWS * QSTRIDE * 2);
  float* comb = reinterpret_cast<float*>(ring);                            // after the prefix loop: [8 warps][16][HD + 2]
  __shared__ int s_abort;
  const uint32_t ring_u = smem_u32(ring), own_u = smem_u32(own_tiles_mem);
  const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STR_STAGES);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kh = blockIdx.x % p.Hkv, chunk = blockIdx.x / p.Hkv;
  const int g_heads = p.Hq / p.Hkv, R_all = p.n * g_heads;
  const bool fused = p.qkv_f32 != nullptr;
  const int NT = (p.P + STR_KEYS - 1) / STR_KEYS;
  const int t0 = (int)((long long)chunk * NT / p.n_prefix_chunks), t1 = (int)((long long)(chunk + 1) * NT / p.n_prefix_chunks);
  const int n_tiles = t1 - t0;
  const int s = chunk;                                                     // blockIdx.x = s * Hkv + kh: the CTA's own segment
  const bool has_own = s < p.n;
  const int S = has_own ? p.suffix_len[s] : 0;                             // (asked for early: used after the set-up)

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int i = 0; i < STR_STAGES; ++i) { mbar_init(full0 + 8 * i, 1); mbar_init(empty0 + 8 * i, STR_CWARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  if (warp == STR_CWARPS) {
    // ---- producer: one thread issues the tiled copies of the chunk's tiles
    if (lane == 0) {
      for (int i = 0; i < n_tiles; ++i) {
        const int st = i % STR_STAGES;
        if (i >= STR_STAGES && !str_wait(empty0 + 8 * st, (uint32_t)((i / STR_STAGES - 1) & 1), &s_abort, p.status)) break;
        const uint32_t kd = ring_u + st * STAGE_BYTES, vd = kd + TILE_BYTES, bar = full0 + 8 * st;
        mbar_expect_tx(bar, STAGE_BYTES);
        const int key0 = (t0 + i) * STR_KEYS;
#pragma unroll
        for (int half = 0; half < HD / 64; ++half) {
          tma_tile_3d(kd + half * (STR_KEYS * 128), &map_k, half * 64, key0, kh, bar);
          tma_tile_3d(vd + half * (STR_KEYS * 128), &map_v, half * 64, key0, kh, bar);
        }
      }
    }
    return;                                                                 // (the consumers wait for every copy issued)
  }

  // ---- consumers
  const int ctid = threadIdx.x;                                             // 0 .. 255
  const int rt = warp & 1, kq = warp >> 1;                                  // row tile, key quarter of a tile
  const int key_end = S + 1;                                                // own keys: cached rows + this pass's row
  __half* ok_ = const_cast<__half*>(p.own_k) + (size_t)(has_own ? s : 0) * p.own_stream_stride + (size_t)kh * p.own_head_stride;
  __half* ov_ = const_cast<__half*>(p.own_v) + (size_t)(has_own ? s : 0) * p.own_stream_stride + (size_t)kh * p.own_head_stride;
  // own tile i into (kd, vd): cached rows by cp.async, the pass's row built here, rows past the end zero
  auto fetch_own_tile = [&](int i, uint32_t kd, uint32_t vd, unsigned char* kd_g, unsigned char* vd_g) {
    for (int j = ctid; j < STR_KEYS * VPR; j += STR_CWARPS * 32) {
      const int r = j / VPR, piece = j % VPR, key = i * STR_KEYS + r;
      const uint32_t off = str_off(r, piece);
      if (key < key_end && !(fused && key == S)) {
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(kd + off), "l"(ok_ + (size_t)key * HD + piece * 8) : "memory");
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(vd + off), "l"(ov_ + (size_t)key * HD + piece * 8) : "memory");
      } else {
        uint4 kv8 = make_uint4(0, 0, 0, 0), vv8 = make_uint4(0, 0, 0, 0);
        if (key < key_end) {
          // this pass's row: built from the projections (k rotated), used, and appended to the stream's own segment
          const float* row = p.qkv_f32 + (size_t)s * (size_t)((p.Hq + 2 * p.Hkv) * HD);
          const float2* cs = p.cs_table + (size_t)(p.pos_base + S + p.depth[s]) * (HD / 2);
          kv8 = head_piece_f16(row + (size_t)(p.Hq + kh) * HD, piece * 8, HD, cs);
          vv8 = head_piece_f16(row + (size_t)(p.Hq + p.Hkv + kh) * HD, piece * 8, HD, nullptr);
          *reinterpret_cast<uint4*>(ok_ + (size_t)key * HD + piece * 8) = kv8;
          *reinterpret_cast<uint4*>(ov_ + (size_t)key * HD + piece * 8) = vv8;
        }
        *reinterpret_cast<uint4*>(kd_g + off) = kv8;
        *reinterpret_cast<uint4*>(vd_g + off) = vv8;
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const int own_tiles = has_own ? (key_end + STR_KEYS - 1) / STR_KEYS : 0;
  for (int i = 0; i < own_tiles && i < STR_OWN_TILES; ++i)
    fetch_own_tile(i, own_u + i * STAGE_BYTES, own_u + i * STAGE_BYTES + TILE_BYTES, own_tiles_mem + (size_t)i * STAGE_BYTES,
                   own_tiles_mem + (size_t)i * STAGE_BYTES + TILE_BYTES);

  // query rows v0 .. v0 + n_rows - 1 of the kv head's virtual rows (v = stream * g_heads + head in group) into dst
  auto build_q = [&](__half* dst, int rows_cap, int v0, int n_rows) {
    for (int i = ctid; i < rows_cap * VPR; i += STR_CWARPS * 32) {
      const int r = i / VPR, c = (i % VPR) * 8;
      uint4 val = make_uint4(0, 0, 0, 0);
      if (r < n_rows) {
        const int v = v0 + r, m = v / g_heads, j = v % g_heads;
        if (fused) {
          const float* row = p.qkv_f32 + (size_t)m * (size_t)((p.Hq + 2 * p.Hkv) * HD);
          const float2* cs = p.cs_table + (size_t)(p.pos_base + p.suffix_len[m] + p.depth[m]) * (HD / 2);
          val = head_piece_f16(row + (size_t)(kh * g_heads + j) * HD, c, HD, cs);
        } else {
          val = *reinterpret_cast<const uint4*>(p.q + ((size_t)m * p.Hq + kh * g_heads + j) * HD + c);
        }
      }
      *reinterpret_cast<uint4*>(dst + (size_t)r * QSTRIDE + c) = val;
    }
  };
  build_q(Qs, STR_ROWS, 0, R_all);
  asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
  uint32_t qf[KSTEPS][4];
  auto load_qf = [&](const __half* src, int row0) {
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      const int mi = lane >> 3, r = lane & 7;
      ldmatrix_x4(qf[ks], src + (size_t)(row0 + (mi & 1) * 8 + r) * QSTRIDE + ks * 16 + (mi >> 1) * 8);
    }
  };
  float o[DT][4];
  float mrow[2], lrow[2];
  auto reset_acc = [&]() {
#pragma unroll
    for (int i = 0; i < DT; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    mrow[0] = mrow[1] = -INFINITY;
    lrow[0] = lrow[1] = 0.f;
  };

  // ---- the shared-prefix chunk, for the rows of all streams
  load_qf(Qs, rt * 16);
  reset_acc();
  const bool rows_live = rt * 16 < R_all;
  for (int i = 0; i < n_tiles; ++i) {
    const int st = i % STR_STAGES;
    const bool ok = str_wait(full0 + 8 * st, (uint32_t)((i / STR_STAGES) & 1), &s_abort, p.status);
    if (ok && rows_live) {
      const uint32_t kt = ring_u + st * STAGE_BYTES, vt = kt + TILE_BYTES;
      const int key0 = (t0 + i) * STR_KEYS + kq * 16;
      str_tile16<HD>(qf, kt, vt, kq * 16, min(16, p.P - key0), true, true, scale_log2, o, mrow, lrow);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty0 + 8 * st);
    if (!ok) break;
  }

  // ---- the CTA's own segment (stream s, this kv head): more keys for the rows of stream s alone (a softmax partial
  // may cover any set of keys: these join the chunk's), masked for every other row
  if (has_own && !s_abort) {
    const int g = lane >> 2;
    const int r_lo = rt * 16 + g, r_hi = r_lo + 8;
    const bool lo_ok = r_lo / g_heads == s && r_lo < R_all, hi_ok = r_hi / g_heads == s && r_hi < R_all;
    const bool tile_has = (s * g_heads) / 16 == rt || (s * g_heads + g_heads - 1) / 16 == rt;   // warp-uniform
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
    for (int i = 0; i < own_tiles; ++i) {
      uint32_t kt = own_u + i * STAGE_BYTES;
      if (i >= STR_OWN_TILES) {
        // a long own segment: the further tiles one at a time through the start of the ring (every prefix tile has
        // been consumed by all warps: barrier above)
        kt = ring_u;
        fetch_own_tile(i, ring_u, ring_u + TILE_BYTES, ring, ring + TILE_BYTES);
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
      }
      const int key0 = i * STR_KEYS + kq * 16;
      if (tile_has && key0 < key_end)
        str_tile16<HD>(qf, kt, kt + TILE_BYTES, kq * 16, min(16, key_end - key0), lo_ok, hi_ok, scale_log2, o, mrow, lrow);
      if (i >= STR_OWN_TILES) asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");
    }
  }
  asm volatile("bar.sync 1, %0;" ::"n"(STR_CWARPS * 32) : "memory");         // every tile consumed: the ring is free
  if (!s_abort) str_combine_write<HD>(p, comb, warp, o, mrow, lrow, kh, 0, R_all, chunk, ctid);
}

// the o adapter's A rows over a kv head's features sit in shared memory beside the decode kernel's tiles
bool attn_decode_o_slice_fits(int hd, int g_heads, int rank) {
  return dec_smem_bytes(hd) + (size_t)rank * g_heads * hd * sizeof(__half) <= (size_t)227 * 1024;
}

// one decode row per stream, a context short enough for one CTA per (kv head, stream), at most 16 query heads per
// kv head
bool attn_single_pass(const AttnArgs& a) {
  return a.T == 1 && a.Hq / a.Hkv <= 16 && a.P + a.suffix_bound + 1 <= 2048 && (a.hd == 64 || a.hd == 128);
}

// one decode row per stream over a long shared prefix: the streaming kernel (one chunk of the prefix per SM and kv
// head, all streams' rows per CTA).  Shapes only: the launch checks the pointers' alignment.
static bool attn_stream_shape(const AttnArgs& a, int sm_count) {
  if (a.T != 1 || attn_single_pass(a) || (a.hd != 64 && a.hd != 128)) return false;
  const int g_heads = a.Hq / a.Hkv;
  const int chunks = sm_count / a.Hkv;                    // CTAs per kv head
  return a.n * g_heads <= STR_ROWS && g_heads <= 16 && a.P >= STR_KEYS && chunks >= a.n && a.suffix_bound + 1 <= 1024;
}

void attn_plan(AttnArgs& a, int sm_count) {
  a.stream_mode = 0;
  if (attn_stream_shape(a, sm_count)) {
    const int NT = (a.P + STR_KEYS - 1) / STR_KEYS;
    int chunks = sm_count / a.Hkv;
    if (chunks > NT) chunks = NT;
    if (chunks < a.n) chunks = a.n;                       // the first n CTAs of a kv head also take an own segment
    if (chunks <= NT) {
      a.stream_mode = 1;
      a.n_prefix_chunks = chunks;
      a.prefix_chunk = (NT + chunks - 1) / chunks * STR_KEYS;
      a.n_own_chunks = 0;                                 // the own segments' keys join the first n chunks' partials
      a.own_chunk = (a.suffix_bound + 1 + STR_KEYS - 1) / STR_KEYS * STR_KEYS;
      return;
    }
  }
  const int g_heads = a.Hq / a.Hkv;
  const int R_all = a.n * a.T * g_heads;
  const int rb_all = (R_all + ATT_ROWS - 1) / ATT_ROWS;
  const int rb_own = (a.T * g_heads + ATT_ROWS - 1) / ATT_ROWS;
  const int target = 2 * sm_count;
  // shared prefix: as many key chunks as it takes to fill the machine, at least 64 keys each
  int want = target / (a.Hkv * rb_all);
  if (want < 1) want = 1;
  int tiles = (a.P + ATT_KEYS - 1) / ATT_KEYS;
  if (tiles < 1) tiles = 1;
  if (want > tiles) want = tiles;
  int tiles_per_chunk = (tiles + want - 1) / want;
  a.prefix_chunk = tiles_per_chunk * ATT_KEYS;
  a.n_prefix_chunks = a.P > 0 ? (a.P + a.prefix_chunk - 1) / a.prefix_chunk : 0;
  // own segments: there are already n * Hkv * rb_own CTAs per chunk
  const int own_keys = a.suffix_bound + a.T;
  want = target / (a.Hkv * a.n * rb_own);
  if (want < 1) want = 1;
  tiles = (own_keys + ATT_KEYS - 1) / ATT_KEYS;
  if (want > tiles) want = tiles;
  tiles_per_chunk = (tiles + want - 1) / want;
  a.own_chunk = tiles_per_chunk * ATT_KEYS;
  a.n_own_chunks = (own_keys + a.own_chunk - 1) / a.own_chunk;
}

size_t attn_workspace_floats(const AttnArgs& a) {
  const int g_heads = a.Hq / a.Hkv;
  const size_t R_all = (size_t)a.n * a.T * g_heads;
  const size_t slots = a.n_prefix_chunks + a.n_own_chunks;
  return (size_t)a.Hkv * R_all * slots * (a.hd + 2);
}

template <int HD>
static cudaError_t launch_attn_hd(const AttnArgs& a, cudaStream_t st) {
  const size_t smem = (size_t)(ATT_ROWS + 4 * ATT_KEYS) * (HD + 8) * sizeof(__half);
  const int g_heads = a.Hq / a.Hkv;
  const int rb_all = (a.n * a.T * g_heads + ATT_ROWS - 1) / ATT_ROWS;
  const int rb_own = (a.T * g_heads + ATT_ROWS - 1) / ATT_ROWS;
  const int items = a.n_prefix_chunks * rb_all + a.n * a.n_own_chunks * rb_own;
  dim3 grid(items, a.Hkv);
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)HD);
  attn_partial_kernel<HD><<<grid, ATT_THREADS, smem, st>>>(a, rb_all, rb_own, scale_log2);
  return cudaGetLastError();
}

cudaError_t init_attention() {
  cudaError_t e = cudaFuncSetAttribute(attn_partial_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)((ATT_ROWS + 4 * ATT_KEYS) * (64 + 8) * sizeof(__half)));
  if (e != cudaSuccess) return e;
  // (+ room for the o adapter's rows over a kv head's features, up to the limit of a CTA)
  e = cudaFuncSetAttribute(attn_decode_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_decode_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_decode_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_decode_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_stream_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)str_smem_bytes(64));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(attn_stream_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)str_smem_bytes(128));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(attn_partial_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)((ATT_ROWS + 4 * ATT_KEYS) * (128 + 8) * sizeof(__half)));
}

static PFN_cuTensorMapEncodeTiled_v12000 attn_map_encoder() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = []() -> PFN_cuTensorMapEncodeTiled_v12000 {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(sym);
  }();
  return fn;
}

// rank-3 fp16 map over one side (K or V) of the shared prefix: (head_dim, P keys, kv heads); box = 64 features x 64 keys
// of one head, 128-byte swizzle; keys past P read as zeros
static cudaError_t attn_prefix_map(const __half* base, int hd, int P, int Hkv, size_t head_stride, CUtensorMap* out) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = attn_map_encoder();
  if (enc == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[3] = {(cuuint64_t)hd, (cuuint64_t)P, (cuuint64_t)Hkv};
  const cuuint64_t strides[2] = {(cuuint64_t)hd * sizeof(__half), (cuuint64_t)head_stride * sizeof(__half)};
  const cuuint32_t box[3] = {64, (cuuint32_t)STR_KEYS, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  const CUresult rc = enc(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<__half*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

static cudaError_t launch_attention_stream(const AttnArgs& a, cudaStream_t st) {
  // the tiled copies and the 16-byte copies of the own rows need aligned bases and strides
  if ((reinterpret_cast<uintptr_t>(a.prefix_k) & 15) || (reinterpret_cast<uintptr_t>(a.prefix_v) & 15) ||
      (reinterpret_cast<uintptr_t>(a.own_k) & 15) || (reinterpret_cast<uintptr_t>(a.own_v) & 15) ||
      (a.prefix_head_stride * sizeof(__half)) % 16 != 0)
    return cudaErrorMisalignedAddress;
  CUtensorMap mk, mv;
  cudaError_t e = attn_prefix_map(a.prefix_k, a.hd, a.P, a.Hkv, a.prefix_head_stride, &mk);
  if (e != cudaSuccess) return e;
  e = attn_prefix_map(a.prefix_v, a.hd, a.P, a.Hkv, a.prefix_head_stride, &mv);
  if (e != cudaSuccess) return e;
  const float scale_log2 = 1.4426950408889634f / sqrtf((float)a.hd);
  const dim3 grid((unsigned)(a.Hkv * a.n_prefix_chunks));
  if (a.hd == 64) attn_stream_kernel<64><<<grid, STR_THREADS, str_smem_bytes(64), st>>>(a, mk, mv, scale_log2);
  else attn_stream_kernel<128><<<grid, STR_THREADS, str_smem_bytes(128), st>>>(a, mk, mv, scale_log2);
  return cudaGetLastError();
}

cudaError_t launch_attention(const AttnArgs& a, cudaStream_t st) {
  if (a.stream_mode) return launch_attention_stream(a, st);
  if (attn_single_pass(a)) {
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)a.hd);
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)a.Hkv, (unsigned)a.n, DEC_SPLIT);
    cfg.blockDim = dim3((unsigned)dec_warps(a.hd) * 32);
    cfg.dynamicSmemBytes = dec_smem_bytes(a.hd) + (a.o_tacc ? (size_t)a.o_rank * (a.Hq / a.Hkv) * a.hd * sizeof(__half) : 0);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;      // the DEC_SPLIT CTAs of a (kv head, stream) form a cluster
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = DEC_SPLIT;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // its first prefix tiles may be in flight while
    attr[1].val.programmaticStreamSerializationAllowed = 1;            // the kernel ahead of it drains
    cfg.attrs = attr;
    cfg.numAttrs = a.pdl ? 2 : 1;
    if (a.trace0 != nullptr) {                              // (the instantiations that stamp the step's timeline)
      if (a.hd == 64) return cudaLaunchKernelEx(&cfg, attn_decode_kernel<64, true>, a, scale_log2);
      return cudaLaunchKernelEx(&cfg, attn_decode_kernel<128, true>, a, scale_log2);
    }
    if (a.hd == 64) return cudaLaunchKernelEx(&cfg, attn_decode_kernel<64, false>, a, scale_log2);
    return cudaLaunchKernelEx(&cfg, attn_decode_kernel<128, false>, a, scale_log2);
  }
  if (a.hd == 64) return launch_attn_hd<64>(a, st);
  if (a.hd == 128) return launch_attn_hd<128>(a, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_attention_merge(const AttnArgs& a, cudaStream_t st) {
  if (attn_single_pass(a)) return cudaSuccess;             // nothing to merge
  const int warps = a.n * a.T * a.Hq;
  attn_merge_kernel<<<(warps + 3) / 4, 128, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace mlora
