// INT4 group-quantised GEMM on the 5th-generation tensor cores for passes with many rows (DS2D verify passes
// of 128-256 rows, prefill chunks): Y^T[n][m] = sum_k Wdeq[k][n] h[m][k]  (Sec. 3.1 projections with the INT4
// weights of Sec. 3.3; "swap-AB": the 128 output features of a CTA are the UMMA M dimension, the rows the N
// dimension).  Per 64 input features a CTA
//   - dequantises its 128 x 64 weight tile from the packed INT4 layout in registers (the same dequant8() as every
//     other path: exactly fp16(q * scale)) and writes it to shared memory as a K-major tile in the 128-byte
//     swizzled layout the tensor core reads,
//   - has the rows' 64 activations copied into a second swizzled K-major tile by one TMA tile copy
//     (cp.async.bulk.tensor, 128-byte swizzle, completion counted on an mbarrier; rows past M read as zero),
//   - lets one thread issue four tcgen05.mma (M 128, N = rows, K 16, fp16 in, fp32 accumulate in tensor memory).
// The MMAs run asynchronously; a tcgen05.commit per stage tells the threads when a stage's buffers may be
// overwritten, so dequantisation of the next stages overlaps the tensor core.  The accumulator is read back with
// tcgen05.ld and written as fp32 partial sums [split][M][N]; gemm_tc_epilogue_kernel adds the K splits in a fixed
// order, adds the LoRA expand term (Eq. 1-4) and applies the projection's epilogue.
// Every mbarrier wait is bounded; a wait that runs out sets the status word and the CTA winds down (it still waits,
// bounded, for its MMAs and frees its tensor memory).
#include <cuda.h>
#include <type_traits>
#include <cudaTypedefs.h>

#include "../../include/mlora.h"
#include "common.cuh"

namespace mlora {

constexpr int TC_BM = 128;                 // output features per CTA (UMMA M)
constexpr int TC_BK = 64;                  // input features per stage: one 128-byte swizzle row of fp16
constexpr int TC_DEQ_WARPS = 8, TC_DEQ_THREADS = TC_DEQ_WARPS * 32;   // one n-tile (16 features) per warp
// dequantised-weight tiles / activation tiles / packed-weight ring depth per CTA.  Up to 128 rows two CTAs share an
// SM (<= 106 KB each); at 256 rows one CTA takes 217 KB.
__host__ __device__ constexpr int tc_nsta(int nrows) { return nrows == 256 ? 3 : 2; }
__host__ __device__ constexpr int tc_nstb(int nrows) { return nrows == 256 ? 4 : (nrows == 128 ? 3 : 4); }
__host__ __device__ constexpr int tc_wdepth(int nrows) { return nrows == 256 ? 8 : 5; }
__host__ __device__ constexpr int tc_ctas_per_sm(int nrows) { return nrows == 256 ? 1 : 2; }
__host__ __device__ constexpr size_t tc_smem_bytes(int nrows) {
  return (size_t)tc_nsta(nrows) * TC_BM * TC_BK * 2 + (size_t)tc_nstb(nrows) * nrows * TC_BK * 2 +
         (size_t)tc_wdepth(nrows) * TC_DEQ_THREADS * 20 + 1024;
}
constexpr int TC_THREADS = TC_DEQ_THREADS + 64;      // + one warp for the activation copies, one for the MMAs
constexpr long long TC_WAIT_CYCLES = 4000000000ll;

__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool tc_wait(uint32_t bar, uint32_t parity, int* status) {
  const long long t0 = clock64();
  for (int it = 0;; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (ok) return true;
    if ((it & 255) == 255 && clock64() - t0 > TC_WAIT_CYCLES) {
      if (status != nullptr) atomicCAS(status, 0, MLORA_ERR_TIMEOUT);
      return false;
    }
  }
}
// byte offset of the 16-byte piece `chunk` (8 fp16) of row `r` in a K-major tile with 128-byte rows, 128B swizzle:
// 8-row groups of 1024 bytes, the piece index XORed with the row inside the group
__device__ __forceinline__ uint32_t sw128_off(int r, int chunk) {
  return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((chunk ^ (r & 7)) << 4));
}
// shared-memory matrix descriptor: K-major, 128B swizzle, 1024 bytes between 8-row groups (descriptor version 1)
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr) {
  return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) |
         ((uint64_t)2 << 61);
}

template <int NROWS>
__global__ void __launch_bounds__(TC_THREADS, tc_ctas_per_sm(NROWS))
w4_gemm_tc_kernel(const GemmArgs p, const int kts_per_split, int* status, const __grid_constant__ CUtensorMap act_map) {
  extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
  // 1024-byte aligned tiles (the swizzle pattern is tied to address bits 7..9): NSTA weight tiles, NSTB activation
  // tiles, then the ring of packed weights (WD slots of 16 + 4 bytes per dequantising thread)
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int NSTA = tc_nsta(NROWS), NSTB = tc_nstb(NROWS), WD = tc_wdepth(NROWS);
  constexpr uint32_t A_BYTES = TC_BM * TC_BK * 2, B_BYTES = NROWS * TC_BK * 2;
  unsigned char* const act_tiles = base + (size_t)NSTA * A_BYTES;
  unsigned char* const wring = act_tiles + (size_t)NSTB * B_BYTES;
  __shared__ __align__(8) uint64_t step_done[NSTB];   // step k arrives on slot k % NSTB when its MMAs have finished
  __shared__ __align__(8) uint64_t act_full[NSTB];    // the activation tile of step k has landed in tile k % NSTB
  __shared__ __align__(8) uint64_t a_full[NSTA];      // all dequantising warps have written weight tile k % NSTA
  __shared__ __align__(8) uint64_t done_bar;
  __shared__ uint32_t tmem_base_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const int slab = blockIdx.x, split = blockIdx.y, m0 = blockIdx.z * NROWS;
  const WLayout L = make_wlayout(p.K, p.N, p.G);
  const int kt_begin = split * kts_per_split;
  const int kt_end = min(L.KT, kt_begin + kts_per_split);
  const int nk = kt_end - kt_begin;

  if (tid == 0) {
    for (int s = 0; s < NSTB; ++s) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(step_done + s)) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(act_full + s)) : "memory");
    }
    for (int s = 0; s < NSTA; ++s)
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tc_smem_u32(a_full + s)), "n"(TC_DEQ_WARPS) : "memory");
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(tc_smem_u32(&done_bar)) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    // tensor memory for the accumulator: NROWS columns of 128 lanes x fp32
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(&tmem_base_s)), "r"((uint32_t)NROWS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = tmem_base_s;
  bool alive = true;
  auto wait_step = [&](int k) {                 // the MMAs of step k have finished reading their tiles
    if (alive) alive = tc_wait(tc_smem_u32(step_done + k % NSTB), (uint32_t)((k / NSTB) & 1), status);
  };

  if (warp == TC_DEQ_WARPS) {
    // ---- activation producer (one thread).  Step j's tile: 64 features (x = kt * 64 elements: a multiple of 128
    // bytes) of NROWS rows from m0, rows >= M filled with zero; tile j % NSTB is refilled once step j - NSTB is done
    if (lane == 0) {
      // programmatic launch: set-up, tensor memory and the dequantising warps' first weight tiles (immutable data) run
      // while the kernel ahead of this one finishes; the activations are that kernel's output
      asm volatile("griddepcontrol.wait;" ::: "memory");
      int issued = 0;
      for (int j = 0; j < nk; ++j) {
        if (j >= NSTB) wait_step(j - NSTB);
        if (!alive) break;
        const uint32_t bar = tc_smem_u32(act_full + j % NSTB);
        const uint32_t dst = tc_smem_u32(act_tiles + (size_t)(j % NSTB) * B_BYTES);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(B_BYTES) : "memory");
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
            ::"r"(dst), "l"(reinterpret_cast<uint64_t>(&act_map)), "r"((kt_begin + j) * TC_BK), "r"(m0), "r"(bar) : "memory");
        issued = j + 1;
      }
      // no copy may still be in flight when the CTA ends: the newest phase of every tile (passes at once unless a
      // wait gave up somewhere)
      for (int j = max(0, issued - NSTB); j < issued; ++j)
        tc_wait(tc_smem_u32(act_full + j % NSTB), (uint32_t)((j / NSTB) & 1), status);
    }
  } else if (warp == TC_DEQ_WARPS + 1) {
    // ---- MMA issuer (one thread): per step, wait for the weight tile and the activation tile, issue, commit
    if (lane == 0) {
      // instruction descriptor: D fp32, A and B fp16, both K-major, N = NROWS, M = 128
      constexpr uint32_t IDESC = (1u << 4) | ((uint32_t)(NROWS >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
      int sa = 0; uint32_t pa = 0;
      int sb = 0; uint32_t pb = 0;
      for (int i = 0; i < nk && alive; ++i) {
        alive = tc_wait(tc_smem_u32(a_full + sa), pa, status);
        if (alive) alive = tc_wait(tc_smem_u32(act_full + sb), pb, status);
        if (!alive) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t adesc = tc_desc(tc_smem_u32(base + (size_t)sa * A_BYTES));
        const uint64_t bdesc = tc_desc(tc_smem_u32(act_tiles + (size_t)sb * B_BYTES));
#pragma unroll
        for (int kk = 0; kk < TC_BK / 16; ++kk) {
          const uint32_t acc = (i > 0 || kk > 0) ? 1u : 0u;
          // 16 features further along K: 32 bytes inside the swizzled 128-byte row (address field in 16-byte units)
          asm volatile(
              "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
              ::"r"(tmem), "l"(adesc + (uint64_t)(kk * 2)), "l"(bdesc + (uint64_t)(kk * 2)), "r"(IDESC), "r"(acc) : "memory");
        }
        // arrives on the step's barrier when the MMAs issued so far have finished reading their tiles
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(step_done + sb)) : "memory");
        if (++sa == NSTA) { sa = 0; pa ^= 1u; }
        if (++sb == NSTB) { sb = 0; pb ^= 1u; }
      }
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(&done_bar)) : "memory");
    }
  } else {
    // ---- dequantising warps: each runs on its own, up to NSTA weight tiles ahead of the tensor core
    const int nt = slab * (TC_BM / TILE_N) + warp;        // this warp's n-tile (16 output features) of the slab
    // past the last n-tile the warp reads tile 0 again: those accumulator lanes are never stored
    const unsigned char* unit = p.w + (size_t)(nt < L.NT ? nt : 0) * L.unit_bytes;
    // packed weights: each thread copies its own 16 bytes of nibbles and its scale word WD steps ahead
    // (cp.async, one group per step) and later reads back only what it copied itself, so no barrier is involved
    const uint32_t wslot0 = tc_smem_u32(wring) + (uint32_t)tid * 16, sslot0 = tc_smem_u32(wring) + TC_DEQ_THREADS * 16 + (uint32_t)tid * 4;
    constexpr uint32_t WSLOT = TC_DEQ_THREADS * 20;
    // The loop is a serial chain per warp with only two warps per scheduler to hide it, so everything that can be
    // is kept as running state: k-tile of the next fetch, ring offsets, tile indices and barrier parities.
    const int gshift = L.G == 64 ? 0 : (L.G == 128 ? 1 : (L.G == 256 ? 2 : 3));   // k-tiles per scale entry, log2
    const unsigned char* wsrc = unit + (size_t)lane * 16;
    const unsigned char* ssrc = unit + (size_t)g * 4;
    int f_kt = kt_begin;                                  // k-tile of the next fetch
    uint32_t f_off = 0;                                   // its slot's byte offset in the ring
    auto fetch_w = [&]() {
      if (f_kt < kt_end) {
        const int c = f_kt >> 3, r = f_kt & 7;
        const uint32_t cbase = (uint32_t)c * L.chunk_full;
        const uint32_t kc = (c == L.nchunks - 1) ? (uint32_t)L.kc_last : (uint32_t)CHUNK_KT;
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(wslot0 + f_off), "l"(wsrc + cbase + r * 512) : "memory");
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(sslot0 + f_off),
                     "l"(ssrc + cbase + kc * 512 + ((r >> gshift) << 5)) : "memory");
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      ++f_kt;
      f_off = (f_off + WSLOT == WD * WSLOT) ? 0u : f_off + WSLOT;
    };
#pragma unroll 1
    for (int j = 0; j < WD; ++j) fetch_w();

    // this thread's four 16-byte pieces of the weight tile (rows 16w + g and 16w + g + 8, pieces 2t and 2t + 1)
    const int r0 = warp * 16 + g, r1 = r0 + 8;
    const uint32_t a_off0 = sw128_off(r0, 2 * t), a_off1 = sw128_off(r0, 2 * t + 1);
    const uint32_t a_off2 = sw128_off(r1, 2 * t), a_off3 = sw128_off(r1, 2 * t + 1);
    uint32_t c_off = 0;                                   // ring offset of the slot consumed next
    int sa = 0;                                           // weight tile of step i
    int sd = NSTB - 1; uint32_t pd = 1;                   // barrier slot of step i - NSTA and its parity (stepped from i = NSTA - 1 on)
#pragma unroll 1
    for (int i = 0; i < nk; ++i) {
      unsigned char* As = base + (size_t)sa * A_BYTES;
      if (i >= NSTA && alive) alive = tc_wait(tc_smem_u32(step_done + sd), pd, status);
      asm volatile("cp.async.wait_group %0;" ::"n"(WD - 1) : "memory");
      uint4 wv;
      uint32_t sw;
      asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(wv.x), "=r"(wv.y), "=r"(wv.z), "=r"(wv.w) : "r"(wslot0 + c_off) : "memory");
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(sw) : "r"(sslot0 + c_off) : "memory");
      c_off = (c_off + WSLOT == WD * WSLOT) ? 0u : c_off + WSLOT;
      // ---- weights: warp w dequantises n-tile w of the slab (rows 16w + g and 16w + g + 8 of the A tile)
      {
        __half2 s_lo, s_hi;
        split_scales(sw, s_lo, s_hi);
        uint32_t a[4][4];
        dequant8(wv.x, s_lo, s_hi, a[0]);
        dequant8(wv.y, s_lo, s_hi, a[1]);
        dequant8(wv.z, s_lo, s_hi, a[2]);
        dequant8(wv.w, s_lo, s_hi, a[3]);
        // a[j][0] / a[j][2]: features 16t+4j+{0,1} / {2,3} of row g;  a[j][1] / a[j][3]: the same of row g+8
        *reinterpret_cast<uint4*>(As + a_off0) = make_uint4(a[0][0], a[0][2], a[1][0], a[1][2]);
        *reinterpret_cast<uint4*>(As + a_off1) = make_uint4(a[2][0], a[2][2], a[3][0], a[3][2]);
        *reinterpret_cast<uint4*>(As + a_off2) = make_uint4(a[0][1], a[0][3], a[1][1], a[1][3]);
        *reinterpret_cast<uint4*>(As + a_off3) = make_uint4(a[2][1], a[2][3], a[3][1], a[3][3]);
      }
      fetch_w();                                           // refills the slot just read
      // the tensor core reads shared memory through the async proxy: order the writes above before it, then one
      // arrival per warp on the tile's barrier
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc_smem_u32(a_full + sa)) : "memory");
      sa = (sa + 1 == NSTA) ? 0 : sa + 1;
      if (i >= NSTA - 1 && ++sd == NSTB) { sd = 0; pd ^= 1u; }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  // all MMAs done (also when a stage wait gave up earlier: wait, bounded, before touching or freeing anything)
  const bool done = tc_wait(tc_smem_u32(&done_bar), 0u, status);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // ---- accumulator -> fp32 partial sums [split][M][N]: lane = output feature, columns = rows
  if (done && alive && nk > 0 && warp < TC_DEQ_WARPS) {
    const int lane_grp = warp & 3, col_half = warp >> 2;       // warps w and w+4 share the lanes, split the columns
    const int n = slab * TC_BM + lane_grp * 32 + lane;
    float* dst = p.partial + (size_t)split * p.M * p.N;
    for (int c0 = col_half * (NROWS / 2); c0 < (col_half + 1) * (NROWS / 2); c0 += 32) {
      uint32_t v[32];
      const uint32_t taddr = tmem + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)c0;
      asm volatile(
          "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
          "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
          "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
          : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
            "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
            "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
            "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
          : "r"(taddr) : "memory");
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      if (n < p.N) {
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int m = m0 + c0 + j;
          if (m < p.M) dst[(size_t)m * p.N + n] = __uint_as_float(v[j]);
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)NROWS) : "memory");
}

// sum of the K splits (fixed order) plus the LoRA expand term of four consecutive physical columns of row m
__device__ __forceinline__ float4 tc_row_quad(const GemmArgs& p, int ksplit, int m, int c) {
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  const size_t sstride = (size_t)p.M * p.N;
  const float* pp = p.partial + (size_t)m * p.N + c;
  int sp = 0;
  for (; sp + 4 <= ksplit; sp += 4) {                      // four splits' loads in flight; still added in split order
    float4 v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = __ldcg(reinterpret_cast<const float4*>(pp + (size_t)(sp + e) * sstride));
#pragma unroll
    for (int e = 0; e < 4; ++e) { s.x += v[e].x; s.y += v[e].y; s.z += v[e].z; s.w += v[e].w; }
  }
  for (; sp < ksplit; ++sp) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(pp + (size_t)sp * sstride));
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  if (p.lora.adapter_idx != nullptr) {
    const int a = p.lora.adapter_idx[m / p.lora.rows_per_stream];
    if (a >= 0 && a < p.lora.n_slots) {
      int seg, col;
      map_col(p.mode, c, p.seg_n0, p.seg_n1, seg, col);
      const __half* B = p.lora.tabB[(size_t)a * p.lora.tab_stride + p.lora.seg[seg].proj_index];
      if (B != nullptr) {
        const int r = p.lora.rank, ldb = p.lora.seg[seg].n;
        const float* T = p.lora.T + ((size_t)m * p.lora.nseg + seg) * r;
        int j = 0;
        for (; (r & 3) == 0 && j + 4 <= r; j += 4) {            // loads of four rank indices in flight together
          const float4 t4 = *reinterpret_cast<const float4*>(T + j);
          uint2 bv[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) bv[e] = __ldg(reinterpret_cast<const uint2*>(B + (size_t)(j + e) * ldb + col));
          const float tj[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 b01 = __half22float2(u32_as_h2(bv[e].x)), b23 = __half22float2(u32_as_h2(bv[e].y));
            s.x = fmaf(tj[e], b01.x, s.x); s.y = fmaf(tj[e], b01.y, s.y);
            s.z = fmaf(tj[e], b23.x, s.z); s.w = fmaf(tj[e], b23.y, s.w);
          }
        }
        for (; j < r; ++j) {
          const float tj = T[j];
          const uint2 bv = *reinterpret_cast<const uint2*>(B + (size_t)j * ldb + col);
          const float2 b01 = __half22float2(u32_as_h2(bv.x)), b23 = __half22float2(u32_as_h2(bv.y));
          s.x = fmaf(tj, b01.x, s.x); s.y = fmaf(tj, b01.y, s.y);
          s.z = fmaf(tj, b23.x, s.z); s.w = fmaf(tj, b23.y, s.w);
        }
      }
    }
  }
  return s;
}

// One thread per (row, 4 physical columns): split sum, LoRA expand (Eq. 1-4, second factor), projection epilogue.
__global__ void gemm_tc_epilogue_kernel(const GemmArgs p, const int ksplit) {
  const int quads = p.N / 4;
  const long long total = (long long)p.M * quads;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int m = (int)(i / quads), c = (int)(i % quads) * 4;
    if (p.epi == EPI_SWIGLU) {
      if ((c >> 4) & 1) continue;                              // the gate quad's thread also takes the up quad
      const float4 gq = tc_row_quad(p, ksplit, m, c), uq = tc_row_quad(p, ksplit, m, c + 16);
      const float gv[4] = {gq.x, gq.y, gq.z, gq.w}, uv[4] = {uq.x, uq.y, uq.z, uq.w};
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) v[e] = gv[e] / (1.f + __expf(-gv[e])) * uv[e];
      const int f = ((c >> 5) << 4) | (c & 15);
      const __half2 o01 = __floats2half2_rn(v[0], v[1]), o23 = __floats2half2_rn(v[2], v[3]);
      *reinterpret_cast<uint2*>(p.out_f16 + (size_t)m * (p.N / 2) + f) = make_uint2(h2_as_u32(o01), h2_as_u32(o23));
    } else {
      const float4 s = tc_row_quad(p, ksplit, m, c);
      if (p.epi == EPI_F32) {
        *reinterpret_cast<float4*>(p.out_f32 + (size_t)m * p.ldo + c) = s;
      } else {
        float4* xp = reinterpret_cast<float4*>(p.resid + (size_t)m * p.N + c);
        float4 x = *xp;
        x.x += s.x; x.y += s.y; x.z += s.z; x.w += s.w;
        *xp = x;
      }
    }
  }
}

// The same epilogue for passes whose rows come in runs of 16 that share an adapter (rows_per_stream a multiple of
// 16: DS2D trees of 16 or 32 nodes), or that have no adapter at all.  A warp takes 16 rows x 32 physical columns and
// computes the LoRA expand term T B (Eq. 1-4, second factor) with mma.sync m16n8k16: T (fp32) enters as the sum of
// two fp16 values (value and rounding remainder), so the product keeps fp32 accuracy; B is fp16 as stored.  The
// adapter's B values are fetched once per 16 rows instead of once per row.
template <bool SWIGLU>
__global__ void __launch_bounds__(256) gemm_tc_epilogue_mma_kernel(const GemmArgs p, const int ksplit) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int ctiles = (p.N + 31) / 32, rtiles = (p.M + 15) / 16;
  const size_t sstride = (size_t)p.M * p.N;
  for (int wt = blockIdx.x * 8 + (threadIdx.x >> 5); wt < ctiles * rtiles; wt += gridDim.x * 8) {
    const int m0 = (wt / ctiles) * 16, c0 = (wt % ctiles) * 32;
    const int mA = m0 + g, mB = mA + 8;
    const bool okA = mA < p.M, okB = mB < p.M;
    // accumulator fragment of n-tile nt: [0],[1] = row mA, columns c0 + 8 nt + 2t, +1;  [2],[3] = row mB
    float acc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;
    // the adapter of the tile's rows: its loads go out before the split sums need theirs
    int a = -1;
    if (p.lora.adapter_idx != nullptr) a = p.lora.adapter_idx[m0 / p.lora.rows_per_stream];
    auto add_splits = [&](int sp, auto nsp_tag) {              // nsp splits' loads in flight, added in split order
      constexpr int NSP = decltype(nsp_tag)::value;
      float2 va[NSP][4], vb[NSP][4];
#pragma unroll
      for (int u = 0; u < NSP; ++u) {
        const float* pp = p.partial + (size_t)(sp + u) * sstride + c0 + 2 * t;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          const bool cok = c0 + nt * 8 < p.N;
          va[u][nt] = (okA && cok) ? __ldcg(reinterpret_cast<const float2*>(pp + (size_t)mA * p.N + nt * 8)) : make_float2(0.f, 0.f);
          vb[u][nt] = (okB && cok) ? __ldcg(reinterpret_cast<const float2*>(pp + (size_t)mB * p.N + nt * 8)) : make_float2(0.f, 0.f);
        }
      }
#pragma unroll
      for (int u = 0; u < NSP; ++u)
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          acc[nt][0] += va[u][nt].x; acc[nt][1] += va[u][nt].y; acc[nt][2] += vb[u][nt].x; acc[nt][3] += vb[u][nt].y;
        }
    };
    int sp = 0;
    for (; sp + 4 <= ksplit; sp += 4) add_splits(sp, std::integral_constant<int, 4>());
    for (; sp < ksplit; ++sp) add_splits(sp, std::integral_constant<int, 1>());
    if (p.lora.adapter_idx != nullptr) {
      if (a >= 0 && a < p.lora.n_slots) {
        const int r = p.lora.rank;
        int seg_of[4], col_of[4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) map_col(p.mode, min(c0 + nt * 8, p.N - 8), p.seg_n0, p.seg_n1, seg_of[nt], col_of[nt]);
        for (int seg = 0; seg < p.lora.nseg; ++seg) {
          bool any = false;
#pragma unroll
          for (int nt = 0; nt < 4; ++nt) any = any || (seg_of[nt] == seg && c0 + nt * 8 < p.N);
          const __half* B = p.lora.tabB[(size_t)a * p.lora.tab_stride + p.lora.seg[seg].proj_index];
          if (!any || B == nullptr) continue;
          const int ldb = p.lora.seg[seg].n;
          const float* TA = p.lora.T + ((size_t)mA * p.lora.nseg + seg) * r;
          const float* TB = p.lora.T + ((size_t)mB * p.lora.nseg + seg) * r;
          for (int k0 = 0; k0 < r; k0 += 16) {
            // A fragments of T: a0 = (row mA, k 2t, 2t+1), a1 = (row mB, same k), a2 / a3 = the same rows, k + 8
            uint32_t ah[4], al[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float* Tr = (q & 1) ? TB : TA;
              const bool rok = (q & 1) ? okB : okA;
              const int k = k0 + 2 * t + (q >> 1) * 8;
              const float x0 = (rok && k < r) ? Tr[k] : 0.f, x1 = (rok && k + 1 < r) ? Tr[k + 1] : 0.f;
              const __half h0 = __float2half_rn(x0), h1 = __float2half_rn(x1);
              ah[q] = h2_as_u32(__halves2half2(h0, h1));
              al[q] = h2_as_u32(__floats2half2_rn(x0 - __half2float(h0), x1 - __half2float(h1)));
            }
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
              if (seg_of[nt] != seg || c0 + nt * 8 >= p.N) continue;      // uniform over the warp
              // B fragment: b0 = (k 2t, 2t+1; column g), b1 = (k + 8; column g)
              const unsigned short* Bc = reinterpret_cast<const unsigned short*>(B) + col_of[nt] + g;
              const int k = k0 + 2 * t;
              const uint32_t e0 = k < r ? __ldg(Bc + (size_t)k * ldb) : 0u, e1 = k + 1 < r ? __ldg(Bc + (size_t)(k + 1) * ldb) : 0u;
              const uint32_t e2 = k + 8 < r ? __ldg(Bc + (size_t)(k + 8) * ldb) : 0u, e3 = k + 9 < r ? __ldg(Bc + (size_t)(k + 9) * ldb) : 0u;
              const uint32_t b0 = e0 | (e1 << 16), b1 = e2 | (e3 << 16);
              mma_16816(acc[nt], ah, b0, b1);
              mma_16816(acc[nt], al, b0, b1);
            }
          }
        }
      }
    }
    if (SWIGLU) {
      // columns c0 .. c0+15 are a gate tile (n-tiles 0, 1), c0+16 .. c0+31 its up tile (n-tiles 2, 3)
      if (c0 >= p.N) continue;
      const int f0 = (c0 >> 5) << 4;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        float v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) { const float gv = acc[nt][e]; v[e] = gv / (1.f + __expf(-gv)) * acc[nt + 2][e]; }
        const int f = f0 + nt * 8 + 2 * t;
        if (okA) *reinterpret_cast<__half2*>(p.out_f16 + (size_t)mA * (p.N / 2) + f) = __floats2half2_rn(v[0], v[1]);
        if (okB) *reinterpret_cast<__half2*>(p.out_f16 + (size_t)mB * (p.N / 2) + f) = __floats2half2_rn(v[2], v[3]);
      }
    } else {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const int c = c0 + nt * 8 + 2 * t;
        if (c >= p.N) continue;
        if (p.epi == EPI_F32) {
          if (okA) *reinterpret_cast<float2*>(p.out_f32 + (size_t)mA * p.ldo + c) = make_float2(acc[nt][0], acc[nt][1]);
          if (okB) *reinterpret_cast<float2*>(p.out_f32 + (size_t)mB * p.ldo + c) = make_float2(acc[nt][2], acc[nt][3]);
        } else {
          if (okA) {
            float2* xp = reinterpret_cast<float2*>(p.resid + (size_t)mA * p.N + c);
            float2 x = *xp; x.x += acc[nt][0]; x.y += acc[nt][1]; *xp = x;
          }
          if (okB) {
            float2* xp = reinterpret_cast<float2*>(p.resid + (size_t)mB * p.N + c);
            float2 x = *xp; x.x += acc[nt][2]; x.y += acc[nt][3]; *xp = x;
          }
        }
      }
    }
  }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (the library does not link libcuda)
static PFN_cuTensorMapEncodeTiled_v12000 tensor_map_encoder() {
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

// rank-2 fp16 map over the activations h [M][K]: box = 64 features x nrows rows, 128-byte swizzle, zero fill
static cudaError_t encode_act_map(const GemmArgs& a, int nrows, CUtensorMap* map) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = tensor_map_encoder();
  if (enc == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[2] = {(cuuint64_t)a.K, (cuuint64_t)a.M};
  const cuuint64_t strides[1] = {(cuuint64_t)a.K * sizeof(__half)};
  const cuuint32_t box[2] = {(cuuint32_t)TC_BK, (cuuint32_t)nrows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half*>(a.h), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int NROWS>
static cudaError_t tc_launch(const GemmArgs& a, int slabs, int ksplit, int kts_per_split, int* status, cudaStream_t st) {
  const size_t smem = tc_smem_bytes(NROWS);
  dim3 grid(slabs, ksplit, (a.M + NROWS - 1) / NROWS);
  CUtensorMap map;
  const cudaError_t e = encode_act_map(a, NROWS, &map);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = dim3(TC_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, w4_gemm_tc_kernel<NROWS>, a, kts_per_split, status, map);
}

cudaError_t init_gemm_tc() {
  cudaError_t e;
  e = cudaFuncSetAttribute(w4_gemm_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(64));
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(w4_gemm_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(128));
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(w4_gemm_tc_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(256));
}

bool gemm_tc_eligible(const GemmArgs& a) {
  if (a.M < 32 || a.N % 16 || a.K % 64) return false;
  if (reinterpret_cast<uintptr_t>(a.h) % 16 != 0 || tensor_map_encoder() == nullptr) return false;   // TMA needs both
  const int nrows = a.M <= 64 ? 64 : (a.M <= 128 ? 128 : 256);
  const size_t m_blocks = (a.M + nrows - 1) / nrows;
  (void)m_blocks;
  return (size_t)a.M * a.N <= a.partial_capacity;            // room for at least one split
}

// Tensor-core path: partial sums by w4_gemm_tc_kernel, then the epilogue kernel.  `status` may be nullptr.
cudaError_t launch_gemm_tc(const GemmArgs& a, int sm_count, int* status, cudaStream_t st) {
  const int nrows = a.M <= 64 ? 64 : (a.M <= 128 ? 128 : 256);
  const int slabs = (a.N + TC_BM - 1) / TC_BM;
  const int m_blocks = (a.M + nrows - 1) / nrows;
  const int KT = a.K / TILE_K;
  // enough CTAs for two per SM (up to 128 rows two fit), at least four k-tiles per split, partial sums must fit
  int ksplit = (nrows <= 128 ? 2 * sm_count : sm_count) / (slabs * m_blocks);
  if (ksplit < 1) ksplit = 1;
  if (ksplit > KT / 4) ksplit = KT / 4 > 0 ? KT / 4 : 1;
  while (ksplit > 1 && (size_t)ksplit * a.M * a.N > a.partial_capacity) --ksplit;
  const int kts_per_split = (KT + ksplit - 1) / ksplit;
  ksplit = (KT + kts_per_split - 1) / kts_per_split;
  cudaError_t e;
  if (nrows == 64) e = tc_launch<64>(a, slabs, ksplit, kts_per_split, status, st);
  else if (nrows == 128) e = tc_launch<128>(a, slabs, ksplit, kts_per_split, status, st);
  else e = tc_launch<256>(a, slabs, ksplit, kts_per_split, status, st);
  if (e != cudaSuccess) return e;
  const int wtiles = ((a.N + 31) / 32) * ((a.M + 15) / 16);
  if ((a.lora.adapter_idx == nullptr || a.lora.rows_per_stream % 16 == 0) && a.ldo % 2 == 0 && wtiles >= 8 * sm_count) {
    // rows come in runs of 16 with one adapter (or none) and there are enough 16 x 32 tiles to give every SM
    // several warps: the expand term runs on mma.sync (below that size the thread-per-quad kernel hides its
    // latencies better)
    const int blocks = (wtiles + 7) / 8;
    if (a.epi == EPI_SWIGLU) gemm_tc_epilogue_mma_kernel<true><<<blocks, 256, 0, st>>>(a, ksplit);
    else gemm_tc_epilogue_mma_kernel<false><<<blocks, 256, 0, st>>>(a, ksplit);
    return cudaGetLastError();
  }
  const long long total = (long long)a.M * (a.N / 4);
  int blocks = (int)((total + 255) / 256);
  if (blocks > sm_count * 8) blocks = sm_count * 8;
  gemm_tc_epilogue_kernel<<<blocks, 256, 0, st>>>(a, ksplit);
  return cudaGetLastError();
}

}  // namespace mlora
