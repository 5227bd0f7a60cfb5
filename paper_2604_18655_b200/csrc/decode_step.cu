// One decode step -- one new row per stream, at most 8 streams (Sec. 3.4, App. A.1) -- as ONE persistent
// cooperative kernel, one CTA per SM.  Embedding, the four projection groups of every decoder (Sec. 3.1; INT4
// weights, Sec. 3.3; LoRA term of Eq. 1-4 with the adapter picked per row, Sec. 3.2 (c)), the attention over the
// shared prompt segment plus the stream's own segment, lm_head, the row argmax and the suffix-length update are
// phases of the kernel with a grid barrier between them.
//
// Why one kernel: a step moves ~600 MB, about 90 us of HBM time, through 80-odd dependent stages.  Each stage is
// bound by the latency of handing its results to every other SM, not by bandwidth, so everything that does NOT
// depend on the step's activations is taken off that chain:
//   * a producer warp streams, through ONE shared-memory ring and in the order of use, everything immutable the
//     CTA will need in ALL phases: its share of the packed INT4 weights (cp.async.bulk) and, for its output
//     columns, the 16-column slices of the rows' LoRA matrices (tiled TMA copies through tensor maps over the
//     caller's A and B, one copy per row and slice; mbarrier transaction counts).  No activations are staged in
//     shared memory, which leaves most of it to the ring: about one decoder layer is in flight ahead of the math;
//   * the fifteen consumer warps split K: a warp owns the same slice of the input features for every output tile
//     of a batch, so its fp16 input fragments are loaded from L2 into registers once per batch, right behind the
//     barrier, and the weights meet them there (dequantise in registers, mma.sync m16n8k16, fp32);
//   * the LoRA shrink of a projection group is computed by the phase that PRODUCES its input: a CTA multiplies
//     its 16 fresh output columns with the matching column slices of A and adds the partial sums into 64-bit
//     fixed-point accumulators (integer atomics: the order of additions cannot change the result, so the step is
//     bit-reproducible).  The consumer finds the complete T behind the barrier it waits at anyway;
//   * RMSNorm (Sec. 3.1) costs no pass: the producer of a residual slice writes x*gain in fp16 and adds the
//     slice's sum of squares to such an accumulator; the consumer scales its outputs by rsqrt(mean + eps);
//   * the fp32 residual stream never leaves the SM that owns its 16 columns (shared memory for the whole step).
//
// Every wait is bounded (pipe.cuh): on expiry the status word becomes MLORA_ERR_TIMEOUT and the kernel runs its
// data-independent control flow to the end.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <type_traits>

#include "pipe.cuh"

namespace mlora {

constexpr int DS_CWARPS = 15;                      // consumer warps (with the producer warp: 512 threads, 128 registers)
constexpr int DS_CTHREADS = DS_CWARPS * 32;
constexpr int DS_THREADS = DS_CTHREADS + 32;       // + one producer warp
constexpr int DS_STAGE_BYTES = 4480;               // >= CHUNK_KT*512 + 8*32, multiple of 128
constexpr int DS_MAX_STAGES = 48;
constexpr int DS_BT = 6;                           // output tiles whose partial sums are parked together
constexpr int DS_MAX_ITEMS = 6;                    // work items (one k-tile) per warp and tile: K <= 5760
constexpr int DS_ITEM_KT = 1;
constexpr int DS_ITEMS_PER_CHUNK = CHUNK_KT / DS_ITEM_KT;   // = arrivals that free a ring stage
constexpr int DS_RED_BYTES = DS_BT * 16 * 512;
constexpr float DS_FIX = 4294967296.f;             // fixed-point scale of the accumulators (2^32)
constexpr float DS_UNFIX = 1.f / 4294967296.f;
constexpr int DS_MIN_STAGES = 16;

static_assert(DS_STAGE_BYTES >= CHUNK_KT * 512 + 8 * 32, "stage too small for a chunk");
static_assert(DS_STAGE_BYTES % 128 == 0, "TMA destinations are 128-byte aligned");

__device__ __forceinline__ void ds_sync() { asm volatile("bar.sync 1, %0;" ::"n"(DS_CTHREADS) : "memory"); }

// LoRA slices in the ring: a "slot" is one 16-column slice of one row's A or B (rank rows of 32 bytes); a stage holds
// rows_per_stage slots, the slices of a tile's 8 rows take stages_per_set stages
__host__ __device__ inline int ds_slot_bytes(int rank) { return rank * 32; }
__host__ __device__ inline int ds_rows_per_stage(int rank) {
  const int n = rank > 0 ? DS_STAGE_BYTES / ds_slot_bytes(rank) : CHAIN_MAX_ROWS;
  return n > CHAIN_MAX_ROWS ? CHAIN_MAX_ROWS : n;
}
__host__ __device__ inline int ds_stages_per_set(int rank) {
  return (CHAIN_MAX_ROWS + ds_rows_per_stage(rank) - 1) / ds_rows_per_stage(rank);
}

// ----------------------------------------------------------------------------- shared-memory carve-up
struct StepSmem {
  size_t bars, red, ys, xs, ts, ring, total;
};
__host__ __device__ inline StepSmem step_carve(int rank, int own_tiles, int nstages) {
  StepSmem s;
  size_t o = 0;
  s.bars = o; o += 1024;                                              // mbarriers
  s.red = o; o += (size_t)DS_RED_BYTES;                               // parked partial sums; attention partials
  s.ys = o; o += (size_t)DS_BT * CHAIN_MAX_ROWS * TILE_N * 4;         // fresh outputs of the batch (attention: q, k, v)
  s.xs = o; o += (size_t)own_tiles * CHAIN_MAX_ROWS * TILE_N * 4;     // the CTA's slice of the residual stream
  s.ts = o; o += (size_t)CHAIN_MAX_ROWS * 3 * (rank > 0 ? rank : 1) * 4;
  o = (o + 127) / 128 * 128;
  s.ring = o; o += (size_t)nstages * DS_STAGE_BYTES;
  s.total = o;
  return s;
}

int step_plan(int d_model, int d_ffn, int Nq, int Nkv, int hd, int rank, int lora_targets, int sm_count, int* own_tiles) {
  if (hd != 64 || rank > CHAIN_MAX_RANK || sm_count < 1) return 0;
  const int g_heads = Nq / Nkv;
  if (g_heads < 1 || g_heads > 7) return 0;
  for (int K : {d_model, Nq, d_ffn})
    if (K % TILE_K || (K / TILE_K + DS_ITEM_KT - 1) / DS_ITEM_KT > DS_MAX_ITEMS * DS_CWARPS) return 0;
  const int ot = (d_model / TILE_N + sm_count - 1) / sm_count;
  if (ot > 3) return 0;                            // a residual phase's outputs take one pass of the epilogue threads
  // inputs too wide for one pass of three k-tiles per warp: only the down projection, and only one tile per CTA
  const int wide = 3 * DS_CWARPS * TILE_K;
  if (d_model > wide || Nq > wide || (d_ffn > wide && ot > 1)) return 0;
  const int r = (rank > 0 && lora_targets != 0) ? rank : 0;
  if (r % 4) return 0;                             // a row's slice (rank x 32 bytes) is a TMA destination: 128-byte aligned
  const size_t limit = 227 * 1024 - 6144;          // the kernel's static shared memory comes on top
  const size_t base = step_carve(r, ot, 0).total;
  if (base >= limit) return 0;
  int n = (int)((limit - base) / DS_STAGE_BYTES);
  if (n > DS_MAX_STAGES) n = DS_MAX_STAGES;
  // two tiles of the widest input with their slices must fit the ring (see the parity rule in the kernel)
  int maxK = d_model; if (Nq > maxK) maxK = Nq; if (d_ffn > maxK) maxK = d_ffn;
  const int nch = (maxK / TILE_K + CHUNK_KT - 1) / CHUNK_KT;
  if (n < DS_MIN_STAGES || n < 2 * (nch + 4 * ds_stages_per_set(r))) return 0;   // ds_batch_tiles >= 2 for every group
  *own_tiles = ot;
  return n;
}

// what the threads need of a phase beyond its descriptor, worked out once per phase
static_assert(sizeof(StepPhase) % 4 == 0, "a phase descriptor is copied word by word");
struct PhaseS {
  StepPhase ph;
  WLayout L;
  int tpu, n_units, my_units, my_tiles, ipt, gshift, bt;
  unsigned vB, vA;                // bit seg*8+m: row m has an adapter for segment seg of this group / the consuming group
};

__device__ __forceinline__ unsigned long long fix_of(float v) { return (unsigned long long)__float2ll_rn(v * DS_FIX); }
__device__ __forceinline__ float unfix(unsigned long long q) { return __ll2float_rn((long long)q) * DS_UNFIX; }
__device__ __forceinline__ void red_add_u64(unsigned long long* p, unsigned long long v) {
  asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}
// float bits -> unsigned key with the same order
__device__ __forceinline__ uint32_t order_key(float v) {
  const uint32_t u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// tiled TMA copy of one box (16 columns x rank rows) of a LoRA matrix: column x, row 0
__device__ __forceinline__ void tma_slice(uint32_t dst, const void* tmap, int x, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(0), "r"(bar) : "memory");
}
// position `off` stages past (st0, par0) in a ring of n stages (off < n)
__device__ __forceinline__ void ring_at(int st0, uint32_t par0, int off, int n, int& st, uint32_t& par) {
  st = st0 + off;
  par = par0;
  if (st >= n) { st -= n; par ^= 1u; }
}
// tiles per batch of a projection group: the batch's slice stages and weight chunks must fit the ring (a warp may be
// a whole batch ahead of the slowest one, and a wait must never be a ring lap ahead of the fill front: mbarrier
// parities repeat every two laps)
__device__ __forceinline__ int ds_batch_tiles(int nstages, int nchunks, int spr, int nseg, int nnext, int tpu) {
  const int per_tile = nchunks + (nseg > 0 ? spr : 0) + (nnext * spr + tpu - 1) / tpu;
  int bt = nstages / per_tile;
  if (bt > DS_BT) bt = DS_BT;
  if (tpu == 2) bt &= ~1;
  return bt;
}
__device__ __forceinline__ void ds_ldmatrix_x4(uint32_t (&r)[4], const void* smem) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(smem)));
}
__device__ __forceinline__ void ds_ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(smem)));
}
// timeline stamp: the SM's cycle counter (cheap to read); slot 11 of the first and of the last phase also get the
// global nanosecond timer
static __device__ __noinline__ void ds_stamp(const StepArgs& a, int p, int id) {
  if (a.trace != nullptr && threadIdx.x == 0 && (blockIdx.x == 0 || blockIdx.x == gridDim.x - 1)) {
    long long* e = a.trace + ((size_t)(blockIdx.x == 0 ? 0 : 1) * a.n_phases + p) * 12;
    e[id] = clock64();
    if ((p == 0 && id == 0) || (p == a.n_phases - 1 && id == 6)) {
      long long tns;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(tns));
      e[11] = tns;
    }
  }
}

// (functions of their own, to keep the kernel's code small: it is executed once per phase, from a cold instruction cache)
static __device__ __noinline__ uint4 ds_head_piece(const float* head, int c, int hd, const float2* cs) {
  return head_piece_f16(head, c, hd, cs);
}
static __device__ __noinline__ WLayout ds_wlayout(int K, int N, int G) { return make_wlayout(K, N, G); }

// ----------------------------------------------------------------------------- main loop of a projection group
struct GemmLoop {
  unsigned char* ring; uint64_t* full_bar; uint64_t* empty_bar; float4* red;
  const __half* in16;
  int K, KT, nchunks, kc_last, gshift, nstages;
  int st_b; uint32_t par_b;            // ring stage and lap parity of the batch's first chunk
  int nb, it_lo, n_it, M, phase;
  long long* tr;                       // timeline slots of this phase for this thread, or nullptr
};
constexpr int DS_PASS_ITEMS = 3;       // work items whose input fragments a warp holds in registers at a time
// The warp's work items (one k-tile each) of every tile of the batch.  Its slice of the input rows (mma B fragments:
// row g of the lane, features 16t..16t+15 of each k-tile, zero past M) is loaded from L2 into registers first and
// serves every tile of the batch.  A warp with more than DS_PASS_ITEMS items (wide inputs; the batch is then a single
// tile) works in two passes: the second pass's fragments wait, copied asynchronously, in the warp's own slots of the
// parking area, which nothing else uses before the tile is parked.
// `early` runs right behind the issue of those loads (further loads the phase needs: one round trip for all).
template <class Early>
__device__ __forceinline__ void gemm_tiles(const GemmLoop& q, const WaitCtx& wc, Early early) {
  uint4 bfr[DS_PASS_ITEMS][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, t = lane & 3;
  const __half* hrow = q.in16 + (size_t)g * q.K + 16 * t;
  const int n_pass = q.n_it > DS_PASS_ITEMS ? 2 : 1;
  uint4* spare = reinterpret_cast<uint4*>(q.red) + (size_t)warp * 32 + lane;     // + k * 512: the warp's slot of tile k
#pragma unroll
  for (int qi = 0; qi < DS_PASS_ITEMS; ++qi) {
    const int kt = q.it_lo + qi;
    if (qi < q.n_it && kt < q.KT && g < q.M) {
      bfr[qi][0] = __ldcg(reinterpret_cast<const uint4*>(hrow + (size_t)kt * TILE_K));
      bfr[qi][1] = __ldcg(reinterpret_cast<const uint4*>(hrow + (size_t)kt * TILE_K + 8));
    } else {
      bfr[qi][0] = make_uint4(0, 0, 0, 0);
      bfr[qi][1] = make_uint4(0, 0, 0, 0);
    }
  }
  if (n_pass > 1) {
#pragma unroll 1
    for (int qi = DS_PASS_ITEMS; qi < 2 * DS_PASS_ITEMS; ++qi) {
      const int kt = q.it_lo + qi;
      const bool live = qi < q.n_it && kt < q.KT && g < q.M;
      const __half* src = live ? hrow + (size_t)kt * TILE_K : q.in16;
      const uint32_t bytes = live ? 16u : 0u;                             // 0: the destination is filled with zeros
#pragma unroll
      for (int hh = 0; hh < 2; ++hh)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(spare + (size_t)((qi - DS_PASS_ITEMS) * 2 + hh) * 512)),
                     "l"(src + hh * 8), "r"(bytes) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  early();
  int st_t = q.st_b;
  uint32_t par_t = q.par_b;
#pragma unroll 1
  for (int tl = 0; tl < q.nb; ++tl) {
    float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
    int c_cur = -1, st = 0, kc = 0;
    bool ok = false;
    const unsigned char* sb = nullptr;
#pragma unroll 1
    for (int pass = 0; pass < n_pass; ++pass) {
      const int it0 = q.it_lo + pass * DS_PASS_ITEMS, n_here = min(q.n_it - pass * DS_PASS_ITEMS, DS_PASS_ITEMS);
      if (pass == 1) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int qi = 0; qi < DS_PASS_ITEMS; ++qi) {
          bfr[qi][0] = spare[(size_t)(qi * 2) * 512];
          bfr[qi][1] = spare[(size_t)(qi * 2 + 1) * 512];
        }
      }
#pragma unroll
      for (int qi = 0; qi < DS_PASS_ITEMS; ++qi) {
        if (qi < n_here) {
          const int it = it0 + qi;
          const int c = it / DS_ITEMS_PER_CHUNK, itl = it - c * DS_ITEMS_PER_CHUNK;
          if (c != c_cur) {
            c_cur = c;
            st = st_t + c;
            uint32_t par = par_t;
            if (st >= q.nstages) { st -= q.nstages; par ^= 1u; }
            kc = (c == q.nchunks - 1) ? q.kc_last : CHUNK_KT;
            ok = wait_mbar(smem_u32(q.full_bar + st), par, wc, 3, q.phase);
            sb = q.ring + (size_t)st * DS_STAGE_BYTES;
            if (q.tr != nullptr && tl == 0 && pass == 0 && qi == 0) q.tr[8] = clock64();
          }
          if (ok && itl < kc) {
            const uint4 wv = *reinterpret_cast<const uint4*>(sb + itl * 512 + lane * 16);
            const uint32_t sw = *reinterpret_cast<const uint32_t*>(sb + kc * 512 + g * 4 + (itl >> q.gshift) * 32);
            __half2 s_lo, s_hi;
            split_scales(sw, s_lo, s_hi);
            uint32_t af[4];
            dequant8(wv.x, s_lo, s_hi, af);
            mma_16816(acc0, af, bfr[qi][0].x, bfr[qi][0].y);
            dequant8(wv.y, s_lo, s_hi, af);
            mma_16816(acc1, af, bfr[qi][0].z, bfr[qi][0].w);
            dequant8(wv.z, s_lo, s_hi, af);
            mma_16816(acc0, af, bfr[qi][1].x, bfr[qi][1].y);
            dequant8(wv.w, s_lo, s_hi, af);
            mma_16816(acc1, af, bfr[qi][1].z, bfr[qi][1].w);
          }
          __syncwarp();
          // one arrival per item; the last item of a ragged chunk also arrives for the items the chunk lacks
          const int arrivals = (itl == kc - 1) ? DS_ITEMS_PER_CHUNK - kc + 1 : 1;
          if (lane < arrivals) mbar_arrive(smem_u32(q.empty_bar + st));
        }
      }
    }
    if (q.tr != nullptr && tl == 0) {
      // (the accumulators are complete when this value is: it depends on them)
      q.tr[9] = clock64() + (long long)(acc0[0] != acc0[0] ? 1 : 0);
    }
    // park the tile's partial sums: [tile][slot of the warp][lane]
    q.red[(size_t)(tl * 16 + warp) * 32 + lane] =
        make_float4(acc0[0] + acc1[0], acc0[1] + acc1[1], acc0[2] + acc1[2], acc0[3] + acc1[3]);
    st_t += q.nchunks;
    if (st_t >= q.nstages) { st_t -= q.nstages; par_t ^= 1u; }
  }
}

// ----------------------------------------------------------------------------- attention phase
// A CTA takes (stream s, kv head h): the stream's row against the shared prompt segment, the stream's own cached
// rows and the row itself (App. A.1: a stream sees the prefill segment and its own segment only).  K and V
// fragments go from L2 straight into registers: the contraction index of QK^T is permuted so that a lane's
// 16-byte loads are its fragments, the key pairs of the PV fragments are zipped with byte permutes.
struct RingPos { int st; uint32_t par; };
__device__ __forceinline__ void attn_phase(const StepArgs& a, const PhaseS& ps, const int* s_suffix, unsigned char* smem,
                                           uint64_t* full_bar, uint64_t* empty_bar, unsigned char* ring, RingPos& pos,
                                           const WaitCtx& wc, int p) {
  const StepPhase& ph = ps.ph;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int bid = (int)blockIdx.x, G = (int)gridDim.x, M = a.M, r = a.rank, nstages = a.nstages;
  const StepSmem cs = step_carve(r, a.own_tiles, nstages);
  float* redf = reinterpret_cast<float*>(smem + cs.red);
  float* Ys = reinterpret_cast<float*>(smem + cs.ys);
  const int Hkv = a.Hkv, g_heads = a.Hq / Hkv;
  constexpr int HD = 64;
  const float scale_log2 = 1.4426950408889634f * rsqrtf((float)HD);
  __half* Qs = reinterpret_cast<__half*>(Ys);                         // [g_heads][HD], then the new k and v rows
  __half* Kn = Qs + 8 * HD;
  __half* Vn = Kn + HD;
  float* part = redf;                                                 // [warp][head][HD + 2]
  float* outs = redf + DS_CWARPS * g_heads * (HD + 2);                // [g_heads * HD] the unit's output rows
  const int Nqkv = (a.Hq + 2 * Hkv) * HD;
  const int ocols = g_heads * HD;
  const int rps = ds_rows_per_stage(r), slot = ds_slot_bytes(r);
  const int n_ao = (ocols / TILE_N + rps - 1) / rps;                  // ring stages of the o projection's A slices
#pragma unroll 1
  for (int u = bid; u < M * Hkv; u += G) {
    const int s = u / Hkv, h = u - s * Hkv;
    const int S = s_suffix[s];
    const size_t lo = (size_t)ph.layer;
    const __half* pk = a.prefix_k + lo * a.prefix_layer_stride + (size_t)h * a.prefix_head_stride;
    const __half* pv = a.prefix_v + lo * a.prefix_layer_stride + (size_t)h * a.prefix_head_stride;
    const size_t own_off = lo * a.own_layer_stride + (size_t)s * a.own_stream_stride + (size_t)h * a.own_head_stride;
    __half* ok_ = a.own_k + own_off;
    __half* ov_ = a.own_v + own_off;
    const int nP = (a.P + 15) >> 4, nO = (S + 15) >> 4, n_tiles = nP + nO;
    const bool has_ao = (ps.vA >> s) & 1u;                             // the row's adapter has an o projection
    // ---- the row's q heads (rotated), its new k (rotated) and v: fp16 into shared memory, k and v also into the cache
    {
      const float* prow = a.qkv + (size_t)s * Nqkv;
      const float2* csr = a.cs_table + (size_t)(a.P + S) * (HD / 2);
      const int nq = g_heads * (HD / 8);
      if (tid < nq) {
        const int hq = tid / (HD / 8), c = (tid % (HD / 8)) * 8;
        *reinterpret_cast<uint4*>(Qs + hq * HD + c) = ds_head_piece(prow + (size_t)(h * g_heads + hq) * HD, c, HD, csr);
      } else if (tid < nq + HD / 8) {
        const int c = (tid - nq) * 8;
        const uint4 v8 = ds_head_piece(prow + (size_t)(a.Hq + h) * HD, c, HD, csr);
        *reinterpret_cast<uint4*>(Kn + c) = v8;
        *reinterpret_cast<uint4*>(ok_ + (size_t)S * HD + c) = v8;
      } else if (tid < nq + 2 * (HD / 8)) {
        const int c = (tid - nq - HD / 8) * 8;
        const uint4 v8 = ds_head_piece(prow + (size_t)(a.Hq + Hkv + h) * HD, c, HD, nullptr);
        *reinterpret_cast<uint4*>(Vn + c) = v8;
        *reinterpret_cast<uint4*>(ov_ + (size_t)S * HD + c) = v8;
      }
    }
    // ---- the warp's first tile: its loads do not depend on q
    uint4 kf[2][2], vf[4];
    auto load_tile = [&](int ti) {
      const bool own = ti >= nP;
      const int k0 = (own ? ti - nP : ti) << 4;
      const int klast = (own ? S : a.P) - 1;
      const __half* kb = own ? ok_ : pk;
      const __half* vb = own ? ov_ : pv;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int key = min(k0 + nt * 8 + g, klast);                  // rows past the end: a valid row, masked below
        const uint4* src = reinterpret_cast<const uint4*>(kb + (size_t)key * HD + 16 * t);
        kf[nt][0] = ldg_stream(src);
        kf[nt][1] = ldg_stream(src + 1);
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int key = min(k0 + 2 * t + (q & 1) + (q >> 1) * 8, klast);
        vf[q] = ldg_stream(reinterpret_cast<const uint4*>(vb + (size_t)key * HD + 8 * g));
      }
    };
    if (warp < n_tiles) load_tile(warp);
    ds_sync();
    ds_stamp(a, p, 1);
    // ---- q fragments: the lane's 16 features of head g (rows past the group: zero)
    uint32_t qw[8];
    {
      uint4 q0 = make_uint4(0, 0, 0, 0), q1 = q0;
      if (g < g_heads) {
        q0 = *reinterpret_cast<const uint4*>(Qs + g * HD + 16 * t);
        q1 = *reinterpret_cast<const uint4*>(Qs + g * HD + 16 * t + 8);
      }
      qw[0] = q0.x; qw[1] = q0.y; qw[2] = q0.z; qw[3] = q0.w; qw[4] = q1.x; qw[5] = q1.y; qw[6] = q1.z; qw[7] = q1.w;
    }
    // PV runs transposed (O^T = V^T P^T: the 16 rows of an MMA are output features, its 8 columns the heads), so
    // every accumulator register is used: tile i holds feature 8g+2i (registers 0,1) and 8g+2i+1 (2,3) of
    // heads 2t and 2t+1
    float o[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float mrow = -INFINITY, lrow = 0.f;                               // of head g (the lane's row of QK^T)
    const int src_a = (2 * t) * 4 + t, src_b = (2 * t + 1) * 4 + t;   // lanes that hold heads 2t and 2t+1
#pragma unroll 1
    for (int ti = warp; ti < n_tiles; ti += DS_CWARPS) {
      const bool own = ti >= nP;
      const int k0 = (own ? ti - nP : ti) << 4, kend = own ? S : a.P;
      float sc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
        const uint32_t kw[8] = {kf[nt][0].x, kf[nt][0].y, kf[nt][0].z, kf[nt][0].w, kf[nt][1].x, kf[nt][1].y, kf[nt][1].z, kf[nt][1].w};
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
          const uint32_t af[4] = {qw[2 * ks], 0u, qw[2 * ks + 1], 0u};
          mma_16816(sc[nt], af, kw[2 * ks], kw[2 * ks + 1]);
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int key = k0 + nt * 8 + 2 * t + e;
          const float v = key < kend ? sc[nt][e] * scale_log2 : -INFINITY;
          sc[nt][e] = v;
          mx = fmaxf(mx, v);
        }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mnew = fmaxf(mrow, mx);                             // finite: every tile has a valid key
      const float corr = exp2f(mrow - mnew);
      mrow = mnew;
      const float p0 = exp2f(sc[0][0] - mnew), p1 = exp2f(sc[0][1] - mnew);
      const float p2 = exp2f(sc[1][0] - mnew), p3 = exp2f(sc[1][1] - mnew);
      lrow = lrow * corr + (p0 + p1) + (p2 + p3);
      const float corr_a = __shfl_sync(0xffffffffu, corr, src_a), corr_b = __shfl_sync(0xffffffffu, corr, src_b);
      const uint32_t b0v = h2_as_u32(__floats2half2_rn(p0, p1));      // (head g; keys 2t, 2t+1)
      const uint32_t b1v = h2_as_u32(__floats2half2_rn(p2, p3));      // (head g; keys 2t+8, 2t+9)
      const uint32_t va[4] = {vf[0].x, vf[0].y, vf[0].z, vf[0].w}, vb2[4] = {vf[1].x, vf[1].y, vf[1].z, vf[1].w};
      const uint32_t vc[4] = {vf[2].x, vf[2].y, vf[2].z, vf[2].w}, vd[4] = {vf[3].x, vf[3].y, vf[3].z, vf[3].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        o[i][0] *= corr_a; o[i][1] *= corr_b; o[i][2] *= corr_a; o[i][3] *= corr_b;
        // rows g / g+8 of the tile: features 8g+2i / 8g+2i+1; columns of A: keys 2t, 2t+1 and 2t+8, 2t+9
        const uint32_t af[4] = {prmt(va[i], vb2[i], 0x5410u), prmt(va[i], vb2[i], 0x7632u),
                                prmt(vc[i], vd[i], 0x5410u), prmt(vc[i], vd[i], 0x7632u)};
        mma_16816(o[i], af, b0v, b1v);
      }
      if (ti + DS_CWARPS < n_tiles) load_tile(ti + DS_CWARPS);
    }
    // ---- the row itself as one more key, on the warp that would take the next tile
    if (warp == n_tiles % DS_CWARPS) {
      float dot = 0.f;
      const uint4 k0v = *reinterpret_cast<const uint4*>(Kn + 16 * t), k1v = *reinterpret_cast<const uint4*>(Kn + 16 * t + 8);
      const uint32_t kw[8] = {k0v.x, k0v.y, k0v.z, k0v.w, k1v.x, k1v.y, k1v.z, k1v.w};
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float2 qf = __half22float2(u32_as_h2(qw[i])), kk = __half22float2(u32_as_h2(kw[i]));
        dot = fmaf(qf.x, kk.x, dot);
        dot = fmaf(qf.y, kk.y, dot);
      }
      dot += __shfl_xor_sync(0xffffffffu, dot, 1);
      dot += __shfl_xor_sync(0xffffffffu, dot, 2);
      const float v = dot * scale_log2;
      const float mnew = fmaxf(mrow, v);
      const float corr = exp2f(mrow - mnew);
      mrow = mnew;
      const float pn = exp2f(v - mnew);
      lrow = lrow * corr + (t == 0 ? pn : 0.f);
      const float corr_a = __shfl_sync(0xffffffffu, corr, src_a), corr_b = __shfl_sync(0xffffffffu, corr, src_b);
      const float pn_a = __shfl_sync(0xffffffffu, pn, src_a), pn_b = __shfl_sync(0xffffffffu, pn, src_b);
      const uint4 vv = *reinterpret_cast<const uint4*>(Vn + 8 * g);   // features 8g .. 8g+7 of the new v row
      const uint32_t vw[4] = {vv.x, vv.y, vv.z, vv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 v2 = __half22float2(u32_as_h2(vw[i]));           // features 8g+2i, 8g+2i+1
        o[i][0] = o[i][0] * corr_a + pn_a * v2.x;
        o[i][1] = o[i][1] * corr_b + pn_b * v2.x;
        o[i][2] = o[i][2] * corr_a + pn_a * v2.y;
        o[i][3] = o[i][3] * corr_b + pn_b * v2.y;
      }
    }
    lrow += __shfl_xor_sync(0xffffffffu, lrow, 1);
    lrow += __shfl_xor_sync(0xffffffffu, lrow, 2);
    {
      float* pa = part + ((size_t)warp * g_heads + 2 * t) * (HD + 2);       // head 2t, head 2t+1 right behind it
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (2 * t < g_heads) { pa[8 * g + 2 * i] = o[i][0]; pa[8 * g + 2 * i + 1] = o[i][2]; }
        if (2 * t + 1 < g_heads) { pa[(HD + 2) + 8 * g + 2 * i] = o[i][1]; pa[(HD + 2) + 8 * g + 2 * i + 1] = o[i][3]; }
      }
      if (g < g_heads && t == 0) {
        float* pm = part + ((size_t)warp * g_heads + g) * (HD + 2);
        pm[HD] = mrow; pm[HD + 1] = lrow;
      }
    }
    ds_stamp(a, p, 2);
    ds_sync();
    // ---- combine the warps' results (log-sum-exp, warp order fixed) and write the unit's output
    if (tid < ocols) {
      const int hq = tid / HD, d = tid - hq * HD;
      float Mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < DS_CWARPS; ++w) Mx = fmaxf(Mx, part[((size_t)w * g_heads + hq) * (HD + 2) + HD]);
      float num = 0.f, den = 0.f;
#pragma unroll
      for (int w = 0; w < DS_CWARPS; ++w) {
        const float* pw = part + ((size_t)w * g_heads + hq) * (HD + 2);
        const float mw = pw[HD];
        if (mw == -INFINITY) continue;                                // a warp without keys
        const float f = exp2f(mw - Mx);
        num += f * pw[d];
        den += f * pw[HD + 1];
      }
      const __half oh = __float2half_rn(den > 0.f ? num / den : 0.f);
      ph.out16[(size_t)s * (a.Hq * HD) + (size_t)(h * g_heads + hq) * HD + d] = oh;
      outs[tid] = __half2float(oh);
    }
    ds_sync();
    // ---- partial shrink sums of the o projection over this unit's columns: a warp per rank index; the A slices
    // (column block cb of 16 in slot cb of the unit's ring stages, [rank][16]) came through the ring
    if (ph.next_nseg > 0 && a.adapter_idx != nullptr && r > 0) {
      // (every stage is waited for before it is released, also when the row has no adapter and nothing was copied)
#pragma unroll 1
      for (int k = 0; k < n_ao; ++k) {
        int st; uint32_t par;
        ring_at(pos.st, pos.par, k, nstages, st, par);
        wait_mbar(smem_u32(full_bar + st), par, wc, 2, p);
      }
      if (has_ao) {
#pragma unroll 1
        for (int j = warp; j < r; j += DS_CWARPS) {
          float acc = 0.f;
          for (int c = lane; c < ocols; c += 32) {
            const int cb = c >> 4;
            int st; uint32_t par;
            ring_at(pos.st, pos.par, cb / rps, nstages, st, par);
            const __half* sl = reinterpret_cast<const __half*>(ring + (size_t)st * DS_STAGE_BYTES + (size_t)(cb % rps) * slot);
            acc = fmaf(outs[c], __half2float(sl[j * TILE_N + (c & 15)]), acc);
          }
          acc = warp_sum(acc);
          if (lane == 0) red_add_u64(a.tacc + ((size_t)ph.t_out * CHAIN_MAX_ROWS + s) * 3 * r + j, fix_of(acc));
        }
      }
      ds_sync();                                                       // every reader is done with the stages
      if (tid < n_ao * DS_ITEMS_PER_CHUNK) {
        int st; uint32_t par;
        ring_at(pos.st, pos.par, tid / DS_ITEMS_PER_CHUNK, nstages, st, par);
        mbar_arrive(smem_u32(empty_bar + st));
      }
      ring_at(pos.st, pos.par, n_ao, nstages, pos.st, pos.par);
    } else if (u + G < M * Hkv) {
      ds_sync();                                                       // the buffers are reused by the next unit
    }
  }
}

// ----------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(DS_THREADS, 1) decode_step_kernel(const __grid_constant__ StepArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ PhaseS s_ps[2];
  __shared__ float s_scale[CHAIN_MAX_ROWS];
  __shared__ int s_adapter[CHAIN_MAX_ROWS];
  __shared__ int s_suffix[CHAIN_MAX_ROWS];
  __shared__ float s_inv[CHAIN_MAX_ROWS];            // rsqrt(mean square + eps) of the phase's input rows
  __shared__ unsigned long long s_amax[CHAIN_MAX_ROWS];
  __shared__ int s_abort_word;
  __shared__ unsigned long long s_base;

  const int nstages = a.nstages;
  const int r = a.rank;
  const bool lora_on = a.adapter_idx != nullptr && r > 0;
  const StepSmem cs = step_carve(r, a.own_tiles, nstages);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + cs.bars);
  uint64_t* empty_bar = full_bar + DS_MAX_STAGES;
  float4* red = reinterpret_cast<float4*>(smem + cs.red);
  float* redf = reinterpret_cast<float*>(smem + cs.red);
  float* Ys = reinterpret_cast<float*>(smem + cs.ys);
  float* Xs = reinterpret_cast<float*>(smem + cs.xs);
  float* Ts = reinterpret_cast<float*>(smem + cs.ts);
  unsigned char* ring = smem + cs.ring;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int bid = (int)blockIdx.x;
  const int G = (int)gridDim.x;
  const int M = a.M;
  const int rps = ds_rows_per_stage(r), spr = ds_stages_per_set(r), slot = ds_slot_bytes(r);
  WaitCtx wc{a.wait_cycles > 0 ? a.wait_cycles : PIPE_WAIT_CYCLES, &s_abort_word, a.sync, a.status};

  // ---- set-up
  if (tid == 0) {
    for (int s = 0; s < nstages; ++s) {
      mbar_init(smem_u32(full_bar + s), 1);
      mbar_init(smem_u32(empty_bar + s), DS_ITEMS_PER_CHUNK);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort_word = (ld_acquire_u64(a.sync + 2) != 0ull) ? 1 : 0;
    // arrivals of earlier launches are whole multiples of the grid size
    s_base = ld_acquire_u64(a.sync + 0) / (unsigned long long)G * (unsigned long long)G;
  }
  if (tid < CHAIN_MAX_ROWS) {
    int ad = -1;
    float sc = 0.f;
    if (lora_on && tid < M) {
      ad = a.adapter_idx[tid];
      if (ad < 0 || ad >= a.n_slots) ad = -1;
      else sc = a.scale[ad];
    }
    s_adapter[tid] = ad;
    s_scale[tid] = sc;
    s_suffix[tid] = tid < M ? a.suffix_len[tid] : 0;
    s_amax[tid] = 0ull;
  }
  __syncthreads();

  // whether row m has an adapter with both matrices for table entry `proj` (lane seg*8+m asks for segment seg)
  auto row_valid = [&](int m, int proj) -> bool {
    const int ad = s_adapter[m];
    if (!lora_on || ad < 0) return false;
    const size_t e = (size_t)ad * a.tab_stride + proj;
    return a.tabA[e] != nullptr && a.tabB[e] != nullptr;
  };

  // =========================================================================== producer warp
  // The ring schedule, known to the producer and to the consumers alike.  Per projection group, per batch of the CTA's
  // tiles: (1) the weight chunks of the tiles, (2) the LoRA-B slices of the batch's tiles (stages_per_set stages per
  // tile), (3) the LoRA-A slices of the consuming group at the batch's output columns (per unit and segment).  The
  // slices come last because their stages are held until the batch's epilogue is done: the producer, which refills
  // the ring in order, can meanwhile run on through the weight stages that the main loop has freed.
  // Embedding: (3) only.  Attention: the o projection's A slices at the unit's columns.
  if (warp == DS_CWARPS) {
    const uint64_t policy = policy_evict_first();
    int stage = 0;
    uint32_t parity = 1u;                              // a fresh "empty" barrier passes a wait on parity 1
    long long issued = 0;
    bool alive = true;
    // lane 0 waits for the stage to be free; every lane learns the outcome
    auto acquire = [&](int p) -> bool {
      int ok = 1;
      if (lane == 0) ok = wait_mbar(smem_u32(empty_bar + stage), parity, wc, 1, p) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      return ok != 0;
    };
    auto advance = [&]() {
      ++issued;
      if (++stage == nstages) { stage = 0; parity ^= 1u; }
    };
    // the slices of up to 8 rows at column x of the matrices named by (tmaps, proj): lane m copies row m's slice
    auto issue_row_set = [&](int p, const unsigned char* tmaps, int proj, unsigned valid8, int x) -> bool {
#pragma unroll 1
      for (int k = 0; k < spr; ++k) {
        if (!acquire(p)) return false;
        const unsigned here = (valid8 >> (k * rps)) & ((1u << rps) - 1u);
        const uint32_t fb = smem_u32(full_bar + stage);
        if (lane == 0) mbar_expect_tx(fb, (uint32_t)__popc(here) * (uint32_t)slot);
        __syncwarp();
        if (lane < rps && ((here >> lane) & 1u)) {
          const int m = k * rps + lane;
          const size_t e = (size_t)s_adapter[m] * a.tab_stride + proj;
          tma_slice(smem_u32(ring + (size_t)stage * DS_STAGE_BYTES + (size_t)lane * slot), tmaps + e * 128, x, fb);
        }
        advance();
      }
      return true;
    };
#pragma unroll 1
    for (int p = 0; p < a.n_phases && alive; ++p) {
      const StepPhase* ph = a.phases + p;              // immutable: read from global
      const int kind = ph->kind;
      if (kind == SK_FIN) continue;
      const int nseg = lora_on ? ph->lora_nseg : 0, nnext = lora_on ? ph->next_nseg : 0;
      // validity of (segment, row) for this group's B and the consuming group's A: lane seg*8+m
      unsigned vB = 0u, vA = 0u;
      {
        const int seg = lane >> 3, m = lane & 7;
        const bool b = lane < 24 && seg < nseg && m < M && row_valid(m, ph->lora_proj[seg < 3 ? seg : 0]);
        const bool c = lane < 24 && seg < nnext && m < M && row_valid(m, ph->next_proj[seg < 3 ? seg : 0]);
        vB = __ballot_sync(0xffffffffu, b);
        vA = __ballot_sync(0xffffffffu, c);
      }
      if (kind == SK_ATTN) {
#pragma unroll 1
        for (int u = bid; u < M * a.Hkv && alive; u += G) {
          const int s = u / a.Hkv, h = u - s * a.Hkv;
          // the K/V this unit will read: asked for in L2 well ahead of the phase
          if (lane == 0) {
            const size_t lo = (size_t)ph->layer;
            if (a.P > 0) {
              const uint32_t bytes = (uint32_t)a.P * (uint32_t)a.hd * 2u;
              const __half* pk = a.prefix_k + lo * a.prefix_layer_stride + (size_t)h * a.prefix_head_stride;
              const __half* pv = a.prefix_v + lo * a.prefix_layer_stride + (size_t)h * a.prefix_head_stride;
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(pk), "r"(bytes) : "memory");
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(pv), "r"(bytes) : "memory");
            }
            const int S = s_suffix[s];
            if (S > 0) {
              const uint32_t bytes = (uint32_t)S * (uint32_t)a.hd * 2u;
              const size_t off = lo * a.own_layer_stride + (size_t)s * a.own_stream_stride + (size_t)h * a.own_head_stride;
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.own_k + off), "r"(bytes) : "memory");
              asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(a.own_v + off), "r"(bytes) : "memory");
            }
          }
          if (nnext > 0) {
            // the o projection's A slices of the row at the unit's columns: column block cb -> slot cb
            const int ocols = (a.Hq / a.Hkv) * a.hd, nbc = ocols / TILE_N;
            const bool ok_row = (vA >> s) & 1u;
#pragma unroll 1
            for (int c0 = 0; c0 < nbc && alive; c0 += rps) {
              if (!acquire(p)) { alive = false; break; }
              const int here = min(rps, nbc - c0);
              const uint32_t fb = smem_u32(full_bar + stage);
              if (lane == 0) mbar_expect_tx(fb, ok_row ? (uint32_t)here * (uint32_t)slot : 0u);
              __syncwarp();
              if (ok_row && lane < here) {
                const size_t e = (size_t)s_adapter[s] * a.tab_stride + ph->next_proj[0];
                tma_slice(smem_u32(ring + (size_t)stage * DS_STAGE_BYTES + (size_t)lane * slot), a.tmapA + e * 128,
                          h * ocols + (c0 + lane) * TILE_N, fb);
              }
              advance();
            }
          }
        }
        continue;
      }
      if (a.trace != nullptr && lane == 0 && p > 0 && (bid == 0 || bid == G - 1))      // when the producer reached this phase
        a.trace[((size_t)(bid == 0 ? 0 : 1) * a.n_phases + p) * 12 + 11] = clock64();
      int tpu = 1, n_units = ph->N / TILE_N, nchunks = 0, bt = DS_BT;
      WLayout L{};
      if (kind == SK_GEMM) {
        L = ds_wlayout(ph->K, ph->N, ph->G);
        tpu = (ph->mode == MODE_GATEUP) ? 2 : 1;
        n_units = L.NT / tpu;
        nchunks = L.nchunks;
        bt = ds_batch_tiles(nstages, L.nchunks, spr, nseg, ph->epi != EPI_F32 ? nnext : 0, tpu);
      }
      const int my_units = (n_units > bid) ? (n_units - 1 - bid) / G + 1 : 0;
      const int my_tiles = my_units * tpu;
      const bool a_next = nnext > 0 && (kind == SK_EMBED || ph->epi != EPI_F32);
#pragma unroll 1
      for (int b0 = 0; b0 < my_tiles && alive; b0 += bt) {
        const int nb = min(bt, my_tiles - b0);
        // (1) weight chunks of the batch's tiles
#pragma unroll 1
        for (int tl = 0; tl < nb && kind == SK_GEMM && alive; ++tl) {
          const int ti = b0 + tl;
          const int nt = (bid + (ti / tpu) * G) * tpu + (ti % tpu);
          const unsigned char* unit = ph->w + (size_t)nt * L.unit_bytes;
#pragma unroll 1
          for (int c = 0; c < nchunks; ++c) {
            if (!acquire(p)) { alive = false; break; }
            if (lane == 0) {
              const uint32_t bytes = (c == nchunks - 1) ? L.chunk_last : L.chunk_full;
              const uint32_t fb = smem_u32(full_bar + stage);
              mbar_expect_tx(fb, bytes);
              bulk_g2s(smem_u32(ring + (size_t)stage * DS_STAGE_BYTES), unit + (size_t)c * L.chunk_full, bytes, fb, policy);
            }
            advance();
          }
        }
        // (2) LoRA-B slices of the batch's tiles
#pragma unroll 1
        for (int tl = 0; tl < nb && nseg > 0 && alive; ++tl) {
          const int ti = b0 + tl;
          const int nt = (bid + (ti / tpu) * G) * tpu + (ti % tpu);
          int seg = 0, col = 0;
          if (ph->mode == MODE_PLAIN) { seg = 0; col = nt * TILE_N; }
          else if (ph->mode == MODE_QKV) {
            const int c = nt * TILE_N;
            if (c < ph->seg_n0) { seg = 0; col = c; }
            else if (c < ph->seg_n0 + ph->seg_n1) { seg = 1; col = c - ph->seg_n0; }
            else { seg = 2; col = c - ph->seg_n0 - ph->seg_n1; }
          } else { seg = nt & 1; col = (nt >> 1) * TILE_N; }
          const unsigned v8 = seg < nseg ? (vB >> (seg * 8)) & 0xffu : 0u;
          if (!issue_row_set(p, a.tmapB, ph->lora_proj[seg < 3 ? seg : 0], v8, col)) alive = false;
        }
        // (3) LoRA-A slices of the consuming group at the batch's output columns
        if (a_next) {
          const int n_un = nb / tpu;
#pragma unroll 1
          for (int ul = 0; ul < n_un && alive; ++ul) {
            const int col = (bid + (b0 / tpu + ul) * G) * TILE_N;
#pragma unroll 1
            for (int seg = 0; seg < nnext && alive; ++seg)
              if (!issue_row_set(p, a.tmapA, ph->next_proj[seg], (vA >> (seg * 8)) & 0xffu, col)) alive = false;
          }
        }
      }
    }
    if (lane == 0) {
      // no copy may be in flight when the CTA ends (after a wait that gave up the consumers do not take them all):
      // wait (bounded) for the newest fill of every stage
      const long long t0 = clock64();
      const long long inflight = issued < nstages ? issued : nstages;
      for (long long k = 1; k <= inflight; ++k) {
        const long long idx = issued - k;
        const int st = (int)(idx % nstages);
        const uint32_t par = (uint32_t)((idx / nstages) & 1);
        while (!mbar_try_wait(smem_u32(full_bar + st), par)) {
          if (clock64() - t0 > wc.limit) break;
        }
      }
    }
    return;                                             // the consumers use named barriers only
  }

  // =========================================================================== consumer warps
  RingPos pos{0, 0u};                                   // ring stage and lap parity of the CTA's next unread stage
  unsigned long long n_bar = 0;

  // loads phase descriptor p, the rows' adapter validity and the derived values into slot p & 1 (one warp)
  auto load_phase = [&](int p) {
    PhaseS& ps = s_ps[p & 1];
    const int* src = reinterpret_cast<const int*>(a.phases + p);
    int* dst = reinterpret_cast<int*>(&ps.ph);
    for (int i = lane; i < (int)(sizeof(StepPhase) / 4); i += 32) dst[i] = __ldg(src + i);
    __syncwarp();
    {
      const int nseg = lora_on ? ps.ph.lora_nseg : 0, nnext = lora_on ? ps.ph.next_nseg : 0;
      const int seg = lane >> 3, m = lane & 7;
      const bool b = lane < 24 && seg < nseg && m < M && row_valid(m, ps.ph.lora_proj[seg < 3 ? seg : 0]);
      const bool c = lane < 24 && seg < nnext && m < M && row_valid(m, ps.ph.next_proj[seg < 3 ? seg : 0]);
      const unsigned vB = __ballot_sync(0xffffffffu, b), vA = __ballot_sync(0xffffffffu, c);
      if (lane == 0) { ps.vB = vB; ps.vA = vA; }
    }
    if (lane == 0) {
      const StepPhase& ph = ps.ph;
      ps.tpu = 1; ps.n_units = 0; ps.ipt = 0; ps.gshift = 31; ps.bt = DS_BT;
      if (ph.kind == SK_GEMM) {
        ps.L = ds_wlayout(ph.K, ph.N, ph.G);
        ps.tpu = (ph.mode == MODE_GATEUP) ? 2 : 1;
        ps.n_units = ps.L.NT / ps.tpu;
        ps.ipt = (ps.L.KT + DS_ITEM_KT - 1) / DS_ITEM_KT;
        ps.gshift = (ps.L.G >= CHUNK_KT * TILE_K) ? 31 : (31 - __clz(ps.L.G / TILE_K));
        ps.bt = ds_batch_tiles(nstages, ps.L.nchunks, spr, lora_on ? ph.lora_nseg : 0,
                               (lora_on && ph.epi != EPI_F32) ? ph.next_nseg : 0, ps.tpu);
      } else if (ph.kind == SK_EMBED) {
        ps.n_units = ph.N / TILE_N;
      }
      ps.my_units = (ps.n_units > bid) ? (ps.n_units - 1 - bid) / G + 1 : 0;
      ps.my_tiles = ps.my_units * ps.tpu;
    }
  };
  if (warp == 1) load_phase(0);
  ds_sync();

  auto stamp = [&](int p, int id) { ds_stamp(a, p, id); };
  // address of the slice of row m in the row set that starts `off` stages past the batch's first stage
  int sl_base = 0;                                      // stages from the batch's first stage to its first slice stage
  auto slice_ptr = [&](int off, int m) -> const __half* {
    int st; uint32_t par;
    ring_at(pos.st, pos.par, sl_base + off + m / rps, nstages, st, par);
    return reinterpret_cast<const __half*>(ring + (size_t)st * DS_STAGE_BYTES + (size_t)(m % rps) * slot);
  };
  // every thread waits for the n_sl slice stages of the batch (they arrived long ago: one test each)
  auto wait_slices = [&](int n_sl, int p) {
#pragma unroll 1
    for (int k = 0; k < n_sl; ++k) {
      int st; uint32_t par;
      ring_at(pos.st, pos.par, sl_base + k, nstages, st, par);
      wait_mbar(smem_u32(full_bar + st), par, wc, 2, p);
    }
  };
  // after a CTA-wide barrier: the n_sl slice stages are free again
  auto release_slices = [&](int n_sl) {
    if (tid < n_sl * DS_ITEMS_PER_CHUNK) {
      int st; uint32_t par;
      ring_at(pos.st, pos.par, sl_base + tid / DS_ITEMS_PER_CHUNK, nstages, st, par);
      mbar_arrive(smem_u32(empty_bar + st));
    }
  };

  // fresh outputs of residual kind (embedding, o and down projections): new residual value xn of (row m, column
  // c of the CTA's k-th tile) -> residual slice, x*gain for the next projection group, sums of squares
  auto resid_out = [&](const StepPhase& ph, int k, int tl, int m, int c, float xn, float gain, bool valid) {
    // (called by whole warps: the shuffles below need every lane; `valid` is false for rows past M)
    const int col = (bid + k * G) * TILE_N + c;
    float sq = 0.f;
    if (valid) {
      Xs[(k * CHAIN_MAX_ROWS + m) * TILE_N + c] = xn;
      const __half xh = __float2half_rn(xn * gain);
      if (ph.out16 != nullptr) ph.out16[(size_t)m * ph.N + col] = xh;
      Ys[(tl * CHAIN_MAX_ROWS + m) * TILE_N + c] = __half2float(xh);
      if (ph.last && a.hidden_out != nullptr) a.hidden_out[(size_t)m * ph.N + col] = xn;
      sq = xn * xn;
    }
    if (ph.ssq_out >= 0) {
      sq += __shfl_xor_sync(0xffffffffu, sq, 1);        // the 16 columns of (tile, row) sit in one half warp
      sq += __shfl_xor_sync(0xffffffffu, sq, 2);
      sq += __shfl_xor_sync(0xffffffffu, sq, 4);
      sq += __shfl_xor_sync(0xffffffffu, sq, 8);
      if (valid && c == 0) red_add_u64(a.ssq + (size_t)ph.ssq_out * CHAIN_MAX_ROWS + m, fix_of(sq));
    }
  };
  // partial shrink sums of the consuming group over the batch's fresh outputs (Ys, values exact in fp16), on the
  // tensor cores: warp m takes row m; per segment and block of 16 rank indices D[16 j][8 rows] = Aslice[16 j][16 columns]
  // * Y^T[16 columns][8 rows], accumulated over the batch's units; column m of D goes into the fixed-point accumulators.
  // The A slices of (unit, segment) start a_off + (unit * nseg + segment) * spr stages past the batch's first stage.
  auto shrink_partial = [&](const PhaseS& ps, int n_un, int a_off) {
    const int nseg = lora_on ? ps.ph.next_nseg : 0;
    if (nseg == 0 || warp >= M) return;
    const int m = warp, g = lane >> 2, t = lane & 3;
#pragma unroll 1
    for (int seg = 0; seg < nseg; ++seg) {
      if (!((ps.vA >> (seg * 8 + m)) & 1u)) continue;
#pragma unroll 1
      for (int j0 = 0; j0 < r; j0 += 16) {
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
        for (int ul = 0; ul < n_un; ++ul) {
          const unsigned char* sl = reinterpret_cast<const unsigned char*>(slice_ptr(a_off + (ul * nseg + seg) * spr, m));
          uint32_t af[4];
          {
            const int i = lane >> 3;
            const int row = min(j0 + 8 * (i & 1) + (lane & 7), r - 1);     // rows past the rank: a valid row, not used
            ds_ldmatrix_x4(af, sl + (size_t)row * 32 + (i >> 1) * 16);
          }
          const float* yr = Ys + (ul * CHAIN_MAX_ROWS + g) * TILE_N;        // row g of the unit's outputs
          const float2 y0 = *reinterpret_cast<const float2*>(yr + 2 * t), y1 = *reinterpret_cast<const float2*>(yr + 2 * t + 8);
          mma_16816(d, af, h2_as_u32(__floats2half2_rn(y0.x, y0.y)), h2_as_u32(__floats2half2_rn(y1.x, y1.y)));
        }
        if (t == (m >> 1)) {                                               // the lanes that hold column m of D
          unsigned long long* dst = a.tacc + ((size_t)ps.ph.t_out * CHAIN_MAX_ROWS + m) * 3 * r + seg * r;
          if (j0 + g < r) red_add_u64(dst + j0 + g, fix_of(d[m & 1]));
          if (j0 + 8 + g < r) red_add_u64(dst + j0 + 8 + g, fix_of(d[2 + (m & 1)]));
        }
      }
    }
  };

#pragma unroll 1
  for (int p = 0; p < a.n_phases; ++p) {
    const PhaseS& ps = s_ps[p & 1];
    const StepPhase& ph = ps.ph;
    const int kind = ph.kind;
    stamp(p, 0);

    if (kind == SK_EMBED) {
      // ------------------------------------------------------------------- embedding (or hidden-state input)
      const int my_tiles = ps.my_tiles;                                  // <= own_tiles <= 3: one batch
      const int nnext = lora_on ? ph.next_nseg : 0;
      const int n_sl = my_tiles * nnext * spr;
      sl_base = 0;
      {
        const int tl = tid >> 7, m = (tid >> 4) & 7, c = tid & 15;
        if (tl < my_tiles) {
          const int col = (bid + tl * G) * TILE_N + c;
          const bool valid = m < M;
          float xn = 0.f, gain = 1.f;
          if (valid) {
            if (a.tokens != nullptr) {
              int tok = a.tokens[m];
              if (tok < 0 || tok >= a.vocab) { atomicCAS(a.status, 0, MLORA_ERR_ARG); tok = 0; }
              xn = __half2float(__ldg(a.embed + (size_t)tok * ph.N + col));
            } else {
              xn = __half2float(__ldg(a.hidden_in + (size_t)m * ph.N + col));
            }
            if (ph.gain_next != nullptr) gain = __half2float(__ldg(ph.gain_next + col));
          }
          resid_out(ph, tl, tl, m, c, xn, gain, valid);
        }
      }
      wait_slices(n_sl, p);
      ds_sync();
      shrink_partial(ps, my_tiles, 0);
      ds_sync();
      release_slices(n_sl);
      ring_at(pos.st, pos.par, n_sl, nstages, pos.st, pos.par);
    } else if (kind == SK_GEMM) {
      // ------------------------------------------------------------------- one projection group
      const int K = ph.K;
      const WLayout L = ps.L;
      const int nseg = lora_on ? ph.lora_nseg : 0;
      const int nnext = (lora_on && ph.epi != EPI_F32) ? ph.next_nseg : 0;
      const int tpu = ps.tpu, my_tiles = ps.my_tiles, bt = ps.bt, gshift = ps.gshift;
      const int it_lo = (warp * ps.ipt) / DS_CWARPS, it_hi = ((warp + 1) * ps.ipt) / DS_CWARPS;
      const int n_it = it_hi - it_lo;
      // ---- the phase's small inputs: the sums of squares of the rows (tid < M) and, per warp w < M, the accumulated
      // shrink sums of row w.  Their loads are issued behind the input fragments' (see gemm_tiles); the values settle in
      // shared memory later: T (times the adapter's scale; the norm factor is applied to the sum of both terms) in the
      // warp's own part of Ts before its first expand, the norm factors before the epilogue.
      int b0_cur = 0;                                                     // first tile of the running batch
      unsigned long long ssq_raw = 0ull, t_raw[2] = {0ull, 0ull};
      const unsigned long long* t_src = a.tacc + ((size_t)ph.t_in * CHAIN_MAX_ROWS + warp) * 3 * r;
      auto early_loads = [&]() {
        if (b0_cur > 0) return;                                           // first batch only
        if (tid < M && ph.norm_in >= 0) ssq_raw = __ldcg(a.ssq + (size_t)ph.norm_in * CHAIN_MAX_ROWS + tid);
        if (nseg > 0 && warp < M) {
          if (lane < 3 * r) t_raw[0] = __ldcg(t_src + lane);
          if (lane + 32 < 3 * r) t_raw[1] = __ldcg(t_src + lane + 32);
        }
      };
      bool t_settled = false;
      auto settle_t = [&]() {                                             // (whole warp w < M)
        float* Tw = Ts + (size_t)warp * 3 * r;
        const float sc = s_scale[warp];
        if (lane < 3 * r) Tw[lane] = unfix(t_raw[0]) * sc;
        if (lane + 32 < 3 * r) Tw[lane + 32] = unfix(t_raw[1]) * sc;
        for (int i = lane + 64; i < 3 * r; i += 32) Tw[i] = unfix(__ldcg(t_src + i)) * sc;
        __syncwarp();
        t_settled = true;
      };
      // LoRA expand of tile tl for row m = warp (second factor of the low-rank term of Eq. 1-4) on the tensor cores:
      // D[16 columns][8 rows] = Bslice^T[16 columns][rank] * T[rank][8 rows], T zero outside column m.  T enters as fp16
      // value + fp16 remainder.  Column m of D (the lanes and registers that hold it) is parked in the sixteenth slot of
      // the tile's partial sums, beside the fifteen warps' slots: the warps of the 8 rows fill disjoint parts of it.
      auto lora_expand = [&](int tl) {
        if (nseg == 0 || warp >= CHAIN_MAX_ROWS) return;
        const int m = warp;
        const int g = lane >> 2, t = lane & 3;
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        float* slot15 = redf + ((size_t)(tl * 16 + 15) * 32 + lane) * 4;
        const int ti = b0_cur + tl;
        const int nt = (bid + (ti / tpu) * G) * tpu + (ti % tpu);
        int seg, col;
        map_col(ph.mode, nt * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
        if (m >= M || seg >= nseg || !((ps.vB >> (seg * 8 + m)) & 1u)) {
          if (t == (m >> 1)) { slot15[m & 1] = 0.f; slot15[2 + (m & 1)] = 0.f; }
          return;
        }
        if (!t_settled) settle_t();
        int st; uint32_t par;
        ring_at(pos.st, pos.par, sl_base + tl * spr + m / rps, nstages, st, par);
        wait_mbar(smem_u32(full_bar + st), par, wc, 2, p);
        const unsigned char* sl = ring + (size_t)st * DS_STAGE_BYTES + (size_t)(m % rps) * slot;   // [rank][16] fp16
        const float* Tm = Ts + ((size_t)m * 3 + seg) * r;
#pragma unroll 1
        for (int j0 = 0; j0 < r; j0 += 16) {
          // A fragments: (column g | g+8, rank index j0 + 2t.. | j0 + 2t+8..) = transposed 8x8 blocks of the slice
          uint32_t af[4];
          {
            const int i = lane >> 3;
            const int row = min(j0 + 8 * (i >> 1) + (lane & 7), r - 1);   // rows past the rank: a valid row, times zero
            ds_ldmatrix_x4_trans(af, sl + (size_t)row * 32 + (i & 1) * 16);
          }
          float tv[4] = {0.f, 0.f, 0.f, 0.f};
          if (g == m) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int j = j0 + 2 * t + (e & 1) + (e >> 1) * 8;
              if (j < r) tv[e] = Tm[j];
            }
          }
          const __half2 h01 = __floats2half2_rn(tv[0], tv[1]), h23 = __floats2half2_rn(tv[2], tv[3]);
          const float2 f01 = __half22float2(h01), f23 = __half22float2(h23);
          const __half2 l01 = __floats2half2_rn(tv[0] - f01.x, tv[1] - f01.y), l23 = __floats2half2_rn(tv[2] - f23.x, tv[3] - f23.y);
          mma_16816(acc, af, h2_as_u32(h01), h2_as_u32(h23));
          mma_16816(acc, af, h2_as_u32(l01), h2_as_u32(l23));
        }
        if (t == (m >> 1)) { slot15[m & 1] = acc[m & 1]; slot15[2 + (m & 1)] = acc[2 + (m & 1)]; }
      };
      const bool track_max = (ph.epi == EPI_F32 && ph.out_f32 == nullptr);

      // the batches of the CTA's tiles
#pragma unroll 1
      for (int b0 = 0; b0 < my_tiles; b0 += bt) {
        b0_cur = b0;
        const int nb = min(bt, my_tiles - b0);                            // tiles in this batch
        const int n_un = nb / tpu;
        const int nB = nseg > 0 ? nb * spr : 0;                           // slice stages of the batch: B sets, then A sets
        const int nA = nnext > 0 ? n_un * nnext * spr : 0;
        sl_base = nb * L.nchunks;                                         // the weight chunks come first
        // the gain of the RMSNorm that follows, for this thread's output column (used in the epilogue)
        float gpre = 1.f;
        if (ph.epi == EPI_RESID && ph.gain_next != nullptr && (tid >> 7) < nb && ((tid >> 4) & 7) < M)
          gpre = __half2float(__ldg(ph.gain_next + (bid + (b0 + (tid >> 7)) * G) * TILE_N + (tid & 15)));

        // ---- main loop: the warp's items of every tile of the batch; a tile's partial sums are parked at once
        if (b0 == 0) stamp(p, 7);
        {
          const GemmLoop gl{ring, full_bar, empty_bar, red, ph.in16, K, L.KT, L.nchunks, L.kc_last, gshift, nstages, pos.st, pos.par,
                            nb, it_lo, n_it, M, p,
                            (a.trace != nullptr && tid == 0 && b0 == 0 && (bid == 0 || bid == G - 1))
                                ? a.trace + ((size_t)(bid == 0 ? 0 : 1) * a.n_phases + p) * 12 : nullptr};
          gemm_tiles(gl, wc, early_loads);
          if (b0 == 0) stamp(p, 10);
#pragma unroll 1
          for (int tl = 0; tl < nb; ++tl) lora_expand(tl);
        }
        stamp(p, 1);
        if (b0 == 0 && tid < CHAIN_MAX_ROWS)
          s_inv[tid] = (ph.norm_in >= 0 && tid < M) ? rsqrtf(unfix(ssq_raw) / (float)K + a.eps) : 1.f;
        wait_slices(nB + nA, p);
        ds_sync();
        stamp(p, 2);

        // ---- epilogue: one thread per (tile or pair, row, column)
        {
#pragma unroll 1
          for (int o = tid; o < n_un * 128; o += DS_CTHREADS) {           // (whole warps: 128 outputs per unit)
          const int ul = o >> 7, m = (o >> 4) & 7, c = o & 15;            // unit of the batch, row, column
          const bool live = m < M;
          // accumulator layout of m16n8k16: lane (g,t) holds (out g, row 2t), (g, 2t+1), (g+8, 2t), (g+8, 2t+1)
          const int src_lane = (c & 7) * 4 + (m >> 1);
          const int e = (c >> 3) * 2 + (m & 1);
          float yv[2] = {0.f, 0.f};
          if (live) {
            const float inv = s_inv[m];
#pragma unroll
            for (int tu = 0; tu < 2; ++tu) {
              if (tu < tpu) {
                const int tl = ul * tpu + tu;
                float y = 0.f;
#pragma unroll
                for (int w = 0; w < DS_CWARPS; ++w)                       // fixed order
                  y += redf[((size_t)(tl * 16 + w) * 32 + src_lane) * 4 + e];
                if (nseg > 0) y += redf[((size_t)(tl * 16 + 15) * 32 + src_lane) * 4 + e];   // the LoRA expand term
                yv[tu] = y * inv;
              }
            }
          }
          const int k_un = b0 / tpu + ul;                                 // the CTA's unit number
          const int u = bid + k_un * G;                                   // global unit
          if (ph.epi == EPI_F32) {
            if (live) {
              float* out = ph.out_f32 != nullptr ? ph.out_f32 : a.logits;
              if (out != nullptr) __stcg(out + (size_t)m * ph.ldo + u * TILE_N + c, yv[0]);
            }
            if (track_max) {
              // lm_head: the best (logit, lowest index) of the row's 16 columns -> the CTA's row maximum
              unsigned long long best = 0ull;
              if (live) best = ((unsigned long long)order_key(yv[0]) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)(u * TILE_N + c));
#pragma unroll
              for (int sh = 1; sh < 16; sh <<= 1) {
                const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, sh);
                best = other > best ? other : best;
              }
              if (c == 0 && best != 0ull) atomicMax(&s_amax[m], best);
            }
          } else if (ph.epi == EPI_RESID) {
            const float xo = live ? Xs[(k_un * CHAIN_MAX_ROWS + m) * TILE_N + c] : 0.f;
            resid_out(ph, k_un, ul, m, c, xo + yv[0], gpre, live);       // (whole warps: see resid_out)
          } else {                                                        // EPI_SWIGLU: even tile = gate, odd tile = up
            if (live) {
              const float v = yv[0] / (1.f + __expf(-yv[0])) * yv[1];
              const __half vh = __float2half_rn(v);
              ph.out16[(size_t)m * (ph.N / 2) + u * TILE_N + c] = vh;
              Ys[(ul * CHAIN_MAX_ROWS + m) * TILE_N + c] = __half2float(vh);
            }
          }
          }
        }
        stamp(p, 3);
        ds_sync();
        // ---- partial shrink sums of the consuming group over the batch's outputs
        if (nnext > 0) shrink_partial(ps, n_un, nB);
        ds_sync();                                                        // every reader is done with the slices
        release_slices(nB + nA);
        // the ring position after this batch's slices and chunks
        {
          int adv = nB + nA + nb * L.nchunks;
          while (adv >= nstages) { adv -= nstages; pos.par ^= 1u; }
          ring_at(pos.st, pos.par, adv, nstages, pos.st, pos.par);
        }
      }
      if (track_max) {
        // the CTA's best (logit, lowest index) per row -> its slot of the exchange array
        if (tid < CHAIN_MAX_ROWS) __stcg(a.amax + (size_t)bid * CHAIN_MAX_ROWS + tid, s_amax[tid]);
      }
    } else if (kind == SK_ATTN) {
      attn_phase(a, ps, s_suffix, smem, full_bar, empty_bar, ring, pos, wc, p);
    } else {
      // ------------------------------------------------------------------- end of the step
      // greedy tokens from the CTAs' row maxima, suffix lengths advanced, accumulators zeroed for the next launch
      if (bid == 0) {
        if (a.out_next != nullptr && warp < M) {
          unsigned long long best = 0ull;
          for (int c = lane; c < G; c += 32) {
            const unsigned long long v = __ldcg(a.amax + (size_t)c * CHAIN_MAX_ROWS + warp);
            best = v > best ? v : best;
          }
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
          }
          if (lane == 0) a.out_next[warp] = (int32_t)(0xFFFFFFFFu - (uint32_t)(best & 0xFFFFFFFFull));
        }
        if (tid < M) a.suffix_len[tid] = s_suffix[tid] + 1;
      }
      const size_t n_acc = (size_t)a.n_tacc * CHAIN_MAX_ROWS * 3 * (r > 0 ? r : 0);
      for (size_t i = (size_t)bid * DS_CTHREADS + tid; i < n_acc; i += (size_t)G * DS_CTHREADS) a.tacc[i] = 0ull;
      for (size_t i = (size_t)bid * DS_CTHREADS + tid; i < (size_t)a.n_ssq * CHAIN_MAX_ROWS; i += (size_t)G * DS_CTHREADS) a.ssq[i] = 0ull;
    }

    // ---- grid barrier: the next phase reads what every CTA wrote
    stamp(p, 4);
    if (p + 1 < a.n_phases) {
      ++n_bar;
      ds_sync();
      stamp(p, 5);
      if (tid == 0) {
        // the release is cumulative over what the CTA's threads wrote before the named barrier above; the acquire
        // load inside wait_counter orders the next phase's reads after the other CTAs' writes
        red_release_add_u64(a.sync + 0, 1ull);
        // (test hook: with inject_stall the first barrier of the launch waits for one arrival too many)
        wait_counter(a.sync + 0, s_base + n_bar * (unsigned long long)G + ((a.inject_stall && n_bar == 1) ? 1ull : 0ull), wc, 5, p);
      }
      if (warp == 1) load_phase(p + 1);
      ds_sync();
    }
    stamp(p, 6);
  }
}

// ----------------------------------------------------------------------------- host side
cudaError_t init_step() {
  return cudaFuncSetAttribute(decode_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 6144);
}

// cuTensorMapEncodeTiled through the runtime's driver entry point lookup (the library does not link libcuda)
static PFN_cuTensorMapEncodeTiled_v12000 step_map_encoder() {
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

static_assert(sizeof(CUtensorMap) == STEP_TMAP_BYTES, "tensor map size");
// rank-2 fp16 map over a LoRA matrix [rank][width] (row-major): box = 16 columns x rank rows, no swizzle
cudaError_t step_encode_slice_map(const void* base, int width, int rank, void* map_out) {
  PFN_cuTensorMapEncodeTiled_v12000 enc = step_map_encoder();
  if (enc == nullptr) return cudaErrorNotSupported;
  const cuuint64_t dims[2] = {(cuuint64_t)width, (cuuint64_t)rank};
  const cuuint64_t strides[1] = {(cuuint64_t)width * sizeof(__half)};
  const cuuint32_t box[2] = {(cuuint32_t)TILE_N, (cuuint32_t)rank};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult rc = enc(reinterpret_cast<CUtensorMap*>(map_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base),
                          dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return rc == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

cudaError_t launch_step(const StepArgs& a, int sm_count, cudaStream_t st) {
  if (a.M < 1 || a.M > CHAIN_MAX_ROWS || a.nstages < DS_MIN_STAGES || a.nstages > DS_MAX_STAGES) return cudaErrorInvalidValue;
  const size_t smem = step_carve(a.rank, a.own_tiles, a.nstages).total;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)sm_count);
  cfg.blockDim = dim3(DS_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;          // all CTAs resident: the grid barrier needs it
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_step_kernel, a);
}

}  // namespace mlora
