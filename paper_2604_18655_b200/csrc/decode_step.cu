// One decode step -- one new row per stream, at most 8 streams (Sec. 3.4, App. A.1) -- as ONE persistent
// cooperative kernel, one CTA per SM.  Embedding, the four projection groups of every decoder (Sec. 3.1; INT4
// weights, Sec. 3.3; LoRA term of Eq. 1-4 with the adapter picked per row, Sec. 3.2 (c)), the attention over the
// shared prompt segment plus the stream's own segment, lm_head, the row argmax and the suffix-length update are
// phases of the kernel with a grid barrier between them.
//
// Why one kernel: a step moves ~600 MB, about 90 us of HBM time, through 80-odd dependent stages.  Each stage is
// bound by the latency of handing its results to every other SM, not by bandwidth, so everything that does NOT
// depend on the step's activations is taken off that chain:
//   * a producer warp streams the CTA's share of the packed INT4 weights of ALL phases through a shared-memory
//     ring (cp.async.bulk + mbarrier transaction counts).  No activations are staged in shared memory, which
//     leaves most of it to the ring: about one decoder layer is in flight ahead of the math;
//   * the sixteen consumer warps split K: a warp owns the same slice of the input features for every output tile
//     of the phase, so its fp16 input fragments are loaded from L2 into registers once per phase, right behind
//     the barrier, and the weights meet them there (dequantise in registers, mma.sync m16n8k16, fp32);
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
#include "pipe.cuh"

namespace mlora {

constexpr int DS_CWARPS = 16;                      // consumer warps
constexpr int DS_CTHREADS = DS_CWARPS * 32;
constexpr int DS_THREADS = DS_CTHREADS + 32;       // + one producer warp
constexpr int DS_STAGE_BYTES = 4480;               // >= CHUNK_KT*512 + 8*32, multiple of 128
constexpr int DS_MAX_STAGES = 48;
constexpr int DS_BT = 4;                           // output tiles whose partial sums are parked together
constexpr int DS_MAX_ITEMS = 3;                    // work items (two k-tiles) per warp and tile: K <= 6144
constexpr int DS_ITEM_KT = 2;
constexpr int DS_ITEMS_PER_CHUNK = CHUNK_KT / DS_ITEM_KT;
constexpr int DS_RED_BYTES = DS_BT * DS_CWARPS * 512;
constexpr int DS_MAX_TP = 3;                       // shrink outputs per thread (8 rows x 3 segments x rank 64 / 512)
constexpr float DS_FIX = 4294967296.f;             // fixed-point scale of the accumulators (2^32)
constexpr float DS_UNFIX = 1.f / 4294967296.f;
constexpr int DS_MIN_STAGES = 12;

static_assert(DS_STAGE_BYTES >= CHUNK_KT * 512 + 8 * 32, "stage too small for a chunk");

__device__ __forceinline__ void ds_sync() { asm volatile("bar.sync 1, %0;" ::"n"(DS_CTHREADS) : "memory"); }

// ----------------------------------------------------------------------------- shared-memory carve-up
struct StepSmem {
  size_t bars, red, bs, as, ys, xs, ts, ring, total;
};
__host__ __device__ inline StepSmem step_carve(int rank, int own_tiles, int as_bytes, int nstages) {
  StepSmem s;
  size_t o = 0;
  s.bars = o; o += 1024;                                              // mbarriers
  s.red = o; o += (size_t)DS_RED_BYTES;                               // parked partial sums; attention partials
  s.bs = o; o += (size_t)(rank > 0 ? DS_BT * CHAIN_MAX_ROWS * rank * 32 : 0);   // LoRA-B slices [tile][row][j][16]
  s.as = o; o += (size_t)as_bytes;                                    // LoRA-A slices of the consuming group
  s.ys = o; o += (size_t)DS_BT * CHAIN_MAX_ROWS * TILE_N * 4;         // fresh outputs of the batch (attention: q, k, v)
  s.xs = o; o += (size_t)own_tiles * CHAIN_MAX_ROWS * TILE_N * 4;     // the CTA's slice of the residual stream
  s.ts = o; o += (size_t)CHAIN_MAX_ROWS * 3 * (rank > 0 ? rank : 1) * 4;
  o = (o + 127) / 128 * 128;
  s.ring = o; o += (size_t)nstages * DS_STAGE_BYTES;
  s.total = o;
  return s;
}

int step_plan(int d_model, int d_ffn, int Nq, int Nkv, int hd, int rank, int lora_targets, int sm_count, int* own_tiles,
              int* as_bytes) {
  if (hd != 64 || rank > CHAIN_MAX_RANK || sm_count < 1) return 0;
  const int g_heads = Nq / Nkv;
  if (g_heads < 1 || g_heads > 7) return 0;
  for (int K : {d_model, Nq, d_ffn})
    if (K % TILE_K || (K / TILE_K + DS_ITEM_KT - 1) / DS_ITEM_KT > DS_MAX_ITEMS * DS_CWARPS) return 0;
  const int ot = (d_model / TILE_N + sm_count - 1) / sm_count;
  if (ot > DS_BT) return 0;
  const int r = (rank > 0 && lora_targets != 0) ? rank : 0;
  // A slices: of q,k,v / gate,up for the tiles of a residual phase; of down for the pairs of a gate/up batch; of o
  // for the query heads of one attention unit
  size_t ab = (size_t)ot * CHAIN_MAX_ROWS * 3 * r * 32;
  const size_t ab_gu = (size_t)(DS_BT / 2) * CHAIN_MAX_ROWS * r * 32, ab_at = (size_t)r * g_heads * hd * 2;
  if (ab_gu > ab) ab = ab_gu;
  if (ab_at > ab) ab = ab_at;
  ab = (ab + 127) / 128 * 128;
  const size_t limit = 227 * 1024 - 6144;          // the kernel's static shared memory comes on top
  const size_t base = step_carve(r, ot, (int)ab, 0).total;
  if (base >= limit) return 0;
  int n = (int)((limit - base) / DS_STAGE_BYTES);
  if (n > DS_MAX_STAGES) n = DS_MAX_STAGES;
  // one batch of tiles must fit the ring (see the parity rule in the kernel)
  int maxK = d_model; if (Nq > maxK) maxK = Nq; if (d_ffn > maxK) maxK = d_ffn;
  const int nch = (maxK / TILE_K + CHUNK_KT - 1) / CHUNK_KT;
  if (n < DS_MIN_STAGES || n < 2 * nch) return 0;
  *own_tiles = ot;
  *as_bytes = (int)ab;
  return n;
}

// what the threads need of a phase beyond its descriptor, worked out once per phase
static_assert(sizeof(StepPhase) % 4 == 0, "a phase descriptor is copied word by word");
struct PhaseS {
  StepPhase ph;
  WLayout L;
  int tpu, n_units, my_units, my_tiles, ipt, gshift, bt;
  const __half* pB[3][CHAIN_MAX_ROWS];      // this group's LoRA-B per (segment, row); nullptr: the row has none
  const __half* pAn[3][CHAIN_MAX_ROWS];     // the consuming group's LoRA-A
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

// ----------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(DS_THREADS, 1) decode_step_kernel(const StepArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ PhaseS s_ps[2];
  __shared__ float s_scale[CHAIN_MAX_ROWS];
  __shared__ int s_adapter[CHAIN_MAX_ROWS];
  __shared__ int s_suffix[CHAIN_MAX_ROWS];
  __shared__ float s_inv[CHAIN_MAX_ROWS];            // rsqrt(mean square + eps) of the phase's input rows
  __shared__ float s_fac[CHAIN_MAX_ROWS];            // factor of the shrink sums: adapter scale (x s_inv)
  __shared__ unsigned long long s_amax[CHAIN_MAX_ROWS];
  __shared__ int s_abort_word;
  __shared__ unsigned long long s_base;

  const int nstages = a.nstages;
  const int r = a.rank;
  const bool lora_on = a.adapter_idx != nullptr && r > 0;
  const StepSmem cs = step_carve(r, a.own_tiles, a.as_bytes, nstages);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + cs.bars);
  uint64_t* empty_bar = full_bar + DS_MAX_STAGES;
  float4* red = reinterpret_cast<float4*>(smem + cs.red);
  float* redf = reinterpret_cast<float*>(smem + cs.red);
  __half* Bs = reinterpret_cast<__half*>(smem + cs.bs);
  __half* As = reinterpret_cast<__half*>(smem + cs.as);
  float* Ys = reinterpret_cast<float*>(smem + cs.ys);
  float* Xs = reinterpret_cast<float*>(smem + cs.xs);
  float* Ts = reinterpret_cast<float*>(smem + cs.ts);
  unsigned char* ring = smem + cs.ring;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int bid = (int)blockIdx.x;
  const int G = (int)gridDim.x;
  const int M = a.M;
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

  // =========================================================================== producer warp
  if (warp == DS_CWARPS) {
    const uint64_t policy = policy_evict_first();
    int stage = 0;
    uint32_t parity = 1u;                              // a fresh "empty" barrier passes a wait on parity 1
    long long issued = 0;
    bool alive = true;
    for (int p = 0; p < a.n_phases && alive; ++p) {
      const StepPhase* ph = a.phases + p;              // immutable: read from global
      const int kind = ph->kind;
      if (kind == SK_ATTN) {
        // the K/V this CTA's unit will read: asked for in L2 well ahead of the phase
        if (lane == 0) {
          for (int u = bid; u < M * a.Hkv; u += G) {
            const int s = u / a.Hkv, h = u - s * a.Hkv;
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
        }
        continue;
      }
      if (kind != SK_GEMM) continue;
      const unsigned char* wbase = ph->w;
      const WLayout L = make_wlayout(ph->K, ph->N, ph->G);
      const int tpu = (ph->mode == MODE_GATEUP) ? 2 : 1;
      const int n_units = L.NT / tpu;
      for (int u = bid; u < n_units && alive; u += G) {
        for (int tu = 0; tu < tpu && alive; ++tu) {
          const unsigned char* unit = wbase + (size_t)(u * tpu + tu) * L.unit_bytes;
          for (int c = 0; c < L.nchunks; ++c) {
            int ok = 1;
            if (lane == 0) ok = wait_mbar(smem_u32(empty_bar + stage), parity, wc, 1, p) ? 1 : 0;
            ok = __shfl_sync(0xffffffffu, ok, 0);
            if (!ok) { alive = false; break; }
            if (lane == 0) {
              const uint32_t bytes = (c == L.nchunks - 1) ? L.chunk_last : L.chunk_full;
              const uint32_t fb = smem_u32(full_bar + stage);
              mbar_expect_tx(fb, bytes);
              bulk_g2s(smem_u32(ring + (size_t)stage * DS_STAGE_BYTES), unit + (size_t)c * L.chunk_full, bytes, fb, policy);
            }
            ++issued;
            if (++stage == nstages) { stage = 0; parity ^= 1u; }
          }
        }
      }
    }
    if (!alive && lane == 0) {
      // abort: the copies already issued still land; wait (bounded) for the stages that may be in flight
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
  const int g = lane >> 2, t = lane & 3;
  int pos_st = 0;                                       // ring stage and lap parity of the CTA's next unread chunk
  uint32_t pos_par = 0u;
  unsigned long long n_bar = 0;

  // loads phase descriptor p, the rows' adapter pointers and the derived values into slot p & 1 (one warp)
  auto load_phase = [&](int p) {
    PhaseS& ps = s_ps[p & 1];
    const int* src = reinterpret_cast<const int*>(a.phases + p);
    int* dst = reinterpret_cast<int*>(&ps.ph);
    for (int i = lane; i < (int)(sizeof(StepPhase) / 4); i += 32) dst[i] = __ldg(src + i);
    __syncwarp();
    if (lane < 3 * CHAIN_MAX_ROWS) {
      const int seg = lane / CHAIN_MAX_ROWS, m = lane % CHAIN_MAX_ROWS;
      const int ad = s_adapter[m];
      const __half *pb = nullptr, *pa = nullptr;
      if (lora_on && ad >= 0) {
        if (seg < ps.ph.lora_nseg) {
          const size_t e = (size_t)ad * a.tab_stride + ps.ph.lora_proj[seg];
          pb = a.tabB[e];
          if (pb == nullptr || a.tabA[e] == nullptr) pb = nullptr;
        }
        if (seg < ps.ph.next_nseg) {
          const size_t e = (size_t)ad * a.tab_stride + ps.ph.next_proj[seg];
          pa = a.tabA[e];
          if (pa == nullptr || a.tabB[e] == nullptr) pa = nullptr;
        }
      }
      ps.pB[seg][m] = pb;
      ps.pAn[seg][m] = pa;
    }
    if (lane == 0) {
      const StepPhase& ph = ps.ph;
      ps.tpu = 1; ps.n_units = 0; ps.ipt = 0; ps.gshift = 31; ps.bt = DS_BT;
      if (ph.kind == SK_GEMM) {
        ps.L = make_wlayout(ph.K, ph.N, ph.G);
        ps.tpu = (ph.mode == MODE_GATEUP) ? 2 : 1;
        ps.n_units = ps.L.NT / ps.tpu;
        ps.ipt = (ps.L.KT + DS_ITEM_KT - 1) / DS_ITEM_KT;
        ps.gshift = (ps.L.G >= CHUNK_KT * TILE_K) ? 31 : (31 - __clz(ps.L.G / TILE_K));
        // a batch of tiles must fit the ring: a warp may be a whole batch ahead of the slowest one, and a wait
        // must never be a ring lap ahead of the fill front (mbarrier parities repeat every two laps)
        int bt = nstages / ps.L.nchunks;
        if (bt > DS_BT) bt = DS_BT;
        if (ps.tpu == 2) bt &= ~1;
        ps.bt = bt;
      } else if (ph.kind == SK_EMBED) {
        ps.n_units = ph.N / TILE_N;
      }
      ps.my_units = (ps.n_units > bid) ? (ps.n_units - 1 - bid) / G + 1 : 0;
      ps.my_tiles = ps.my_units * ps.tpu;
    }
  };
  if (warp == 1) load_phase(0);
  ds_sync();

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
  // LoRA-A slices of the consuming group at the columns of the batch's units -> As[unit][row][seg*r + j][16]
  // (cols_unit0: logical column of unit 0's first output, unit stride in columns, units in the batch)
  auto issue_a_next = [&](const PhaseS& ps, int col0, int col_stride, int n_un) {
    const int nseg = ps.ph.next_nseg;
    if (!lora_on || nseg == 0) return;
    const int per_row = nseg * r * 2;                                   // 16-byte pieces per (unit, row)
    const int total = n_un * M * per_row;
    for (int idx = tid; idx < total; idx += DS_CTHREADS) {
      const int ul = idx / (M * per_row);
      const int rem = idx - ul * (M * per_row);
      const int m = rem / per_row;
      const int x = rem - m * per_row, sj = x >> 1, h16 = x & 1;
      const int seg = sj / r, j = sj - seg * r;
      const __half* A = ps.pAn[seg][m];
      if (A != nullptr)
        cp_async16_ca(As + ((size_t)(ul * CHAIN_MAX_ROWS + m) * (nseg * r) + sj) * 16 + h16 * 8,
                      A + (size_t)j * ps.ph.next_ld + col0 + ul * col_stride + h16 * 8);
    }
  };
  // partial shrink sums of the consuming group over the batch's fresh outputs (Ys), kept per thread across batches
  auto shrink_partial = [&](const PhaseS& ps, int n_un, float (&tp)[DS_MAX_TP]) {
    const int nseg = ps.ph.next_nseg;
    if (!lora_on || nseg == 0) return;
    const int per_row = nseg * r;
#pragma unroll
    for (int q = 0; q < DS_MAX_TP; ++q) {
      const int o = tid + q * DS_CTHREADS;
      if (o >= M * per_row) break;
      const int m = o / per_row, sj = o - m * per_row;
      if (ps.pAn[sj / r][m] == nullptr) continue;
      float acc = 0.f;
      for (int ul = 0; ul < n_un; ++ul) {
        const uint4* ap = reinterpret_cast<const uint4*>(As + ((size_t)(ul * CHAIN_MAX_ROWS + m) * per_row + sj) * 16);
        const float4* yp = reinterpret_cast<const float4*>(Ys + (ul * CHAIN_MAX_ROWS + m) * TILE_N);
        const uint4 a0 = ap[0], a1 = ap[1];
        const float4 y0 = yp[0], y1 = yp[1], y2 = yp[2], y3 = yp[3];
        const float2 f0 = __half22float2(u32_as_h2(a0.x)), f1 = __half22float2(u32_as_h2(a0.y));
        const float2 f2 = __half22float2(u32_as_h2(a0.z)), f3 = __half22float2(u32_as_h2(a0.w));
        const float2 f4 = __half22float2(u32_as_h2(a1.x)), f5 = __half22float2(u32_as_h2(a1.y));
        const float2 f6 = __half22float2(u32_as_h2(a1.z)), f7 = __half22float2(u32_as_h2(a1.w));
        acc += y0.x * f0.x + y0.y * f0.y + y0.z * f1.x + y0.w * f1.y + y1.x * f2.x + y1.y * f2.y + y1.z * f3.x + y1.w * f3.y +
               y2.x * f4.x + y2.y * f4.y + y2.z * f5.x + y2.w * f5.y + y3.x * f6.x + y3.y * f6.y + y3.z * f7.x + y3.w * f7.y;
      }
      tp[q] += acc;
    }
  };
  auto shrink_commit = [&](const PhaseS& ps, const float (&tp)[DS_MAX_TP]) {
    const int nseg = ps.ph.next_nseg;
    if (!lora_on || nseg == 0 || ps.my_units == 0) return;
    const int per_row = nseg * r;
#pragma unroll
    for (int q = 0; q < DS_MAX_TP; ++q) {
      const int o = tid + q * DS_CTHREADS;
      if (o >= M * per_row) break;
      const int m = o / per_row, sj = o - m * per_row;
      if (ps.pAn[sj / r][m] == nullptr) continue;
      red_add_u64(a.tacc + ((size_t)ps.ph.t_out * CHAIN_MAX_ROWS + m) * 3 * r + sj, fix_of(tp[q]));
    }
  };

  for (int p = 0; p < a.n_phases; ++p) {
    const PhaseS& ps = s_ps[p & 1];
    const StepPhase& ph = ps.ph;
    const int kind = ph.kind;

    if (kind == SK_EMBED) {
      // ------------------------------------------------------------------- embedding (or hidden-state input)
      float tp[DS_MAX_TP] = {0.f, 0.f, 0.f};
      const int my_tiles = ps.my_tiles;                                  // <= own_tiles <= DS_BT: one batch
      issue_a_next(ps, bid * TILE_N, G * TILE_N, my_tiles);
      asm volatile("cp.async.commit_group;" ::: "memory");
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
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      ds_sync();
      shrink_partial(ps, my_tiles, tp);
      shrink_commit(ps, tp);
    } else if (kind == SK_GEMM) {
      // ------------------------------------------------------------------- one projection group
      const int K = ph.K;
      const WLayout L = ps.L;
      const int nseg = lora_on ? ph.lora_nseg : 0;
      const int tpu = ps.tpu, my_tiles = ps.my_tiles, bt = ps.bt, gshift = ps.gshift;
      const int it_lo = (warp * ps.ipt) / DS_CWARPS, it_hi = ((warp + 1) * ps.ipt) / DS_CWARPS;
      const int n_it = it_hi - it_lo;
      // ---- 1. the warp's slice of the input rows -> registers (mma B fragments; row g of the lane, zero past M)
      uint4 bfr[DS_MAX_ITEMS][DS_ITEM_KT][2];
      {
        const __half* hrow = ph.in16 + (size_t)g * K + 16 * t;
#pragma unroll
        for (int qi = 0; qi < DS_MAX_ITEMS; ++qi)
#pragma unroll
          for (int q = 0; q < DS_ITEM_KT; ++q) {
            const int kt = (it_lo + qi) * DS_ITEM_KT + q;
            if (qi < n_it && kt < L.KT && g < M && my_tiles > 0) {
              bfr[qi][q][0] = __ldcg(reinterpret_cast<const uint4*>(hrow + (size_t)kt * TILE_K));
              bfr[qi][q][1] = __ldcg(reinterpret_cast<const uint4*>(hrow + (size_t)kt * TILE_K + 8));
            } else {
              bfr[qi][q][0] = make_uint4(0, 0, 0, 0);
              bfr[qi][q][1] = make_uint4(0, 0, 0, 0);
            }
          }
      }
      // ---- 2. the norm factor of the rows and the accumulated shrink sums of this group
      if (tid < CHAIN_MAX_ROWS) {
        float inv = 1.f;
        if (ph.norm_in >= 0 && tid < M)
          inv = rsqrtf(unfix(__ldcg(a.ssq + (size_t)ph.norm_in * CHAIN_MAX_ROWS + tid)) / (float)K + a.eps);
        s_inv[tid] = inv;
        s_fac[tid] = s_scale[tid] * inv;
      }
      if (nseg > 0)
        for (int i = tid; i < M * 3 * r; i += DS_CTHREADS) {
          const int seg = (i / r) % 3;
          Ts[i] = seg < nseg ? unfix(__ldcg(a.tacc + (size_t)ph.t_in * CHAIN_MAX_ROWS * 3 * r + i)) : 0.f;
        }
      float tp[DS_MAX_TP] = {0.f, 0.f, 0.f};
      unsigned long long best = 0ull;                                     // lm_head: the thread's best (logit, index)
      const bool track_max = (ph.epi == EPI_F32 && ph.out_f32 == nullptr);

      for (int b0 = 0; b0 < my_tiles; b0 += bt) {
        const int nb = min(bt, my_tiles - b0);                            // tiles in this batch
        // ---- 3. LoRA-B slices of the batch's tiles and LoRA-A slices of the consuming group (immutable)
        if (nseg > 0) {
          const int r2 = r * 2;
          for (int idx = tid; idx < nb * M * r2; idx += DS_CTHREADS) {
            const int tl = idx / (M * r2);
            const int rem = idx - tl * (M * r2);
            const int m = rem / r2, x = rem - m * r2, j = x >> 1, h16 = x & 1;
            const int ti = b0 + tl;
            const int nt = (bid + (ti / tpu) * G) * tpu + (ti % tpu);
            int seg, col;
            map_col(ph.mode, nt * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
            if (seg >= nseg) continue;
            const __half* B = ps.pB[seg][m];
            if (B != nullptr)
              cp_async16_ca(Bs + (((size_t)tl * CHAIN_MAX_ROWS + m) * r + j) * 16 + h16 * 8,
                            B + (size_t)j * ph.lora_n[seg] + col + h16 * 8);
          }
        }
        if (ph.epi == EPI_RESID) issue_a_next(ps, (bid + b0 * G) * TILE_N, G * TILE_N, nb);
        else if (ph.epi == EPI_SWIGLU) issue_a_next(ps, (bid + (b0 / 2) * G) * TILE_N, G * TILE_N, nb / 2);
        asm volatile("cp.async.commit_group;" ::: "memory");

        // the gain of the RMSNorm that follows, for this thread's output column (used in the epilogue)
        float gpre = 1.f;
        if (ph.epi == EPI_RESID && ph.gain_next != nullptr && (tid >> 7) < nb && ((tid >> 4) & 7) < M)
          gpre = __half2float(__ldg(ph.gain_next + (bid + (b0 + (tid >> 7)) * G) * TILE_N + (tid & 15)));

        // ---- 4. main loop: the warp's items of every tile of the batch
        float acc[DS_BT][4];
#pragma unroll
        for (int tl = 0; tl < DS_BT; ++tl) {
          acc[tl][0] = acc[tl][1] = acc[tl][2] = acc[tl][3] = 0.f;
          if (tl < nb && n_it > 0) {
            float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
            // stage and lap parity of the tile's first chunk, stepped (no division in the loop)
            int st_t = pos_st + (b0 + tl) * L.nchunks;
            uint32_t par_t = pos_par;
            while (st_t >= nstages) { st_t -= nstages; par_t ^= 1u; }
            int c_cur = -1, st = 0, kc = 0;
            bool ok = false;
            const unsigned char* sb = nullptr;
            const unsigned char* ssc = nullptr;
#pragma unroll
            for (int qi = 0; qi < DS_MAX_ITEMS; ++qi) {
              if (qi < n_it) {
                const int it = it_lo + qi;
                const int c = it / DS_ITEMS_PER_CHUNK, itl = it - c * DS_ITEMS_PER_CHUNK;
                if (c != c_cur) {
                  c_cur = c;
                  st = st_t + c;
                  uint32_t par = par_t;
                  if (st >= nstages) { st -= nstages; par ^= 1u; }
                  kc = (c == L.nchunks - 1) ? L.kc_last : CHUNK_KT;
                  ok = wait_mbar(smem_u32(full_bar + st), par, wc, 3, p);
                  sb = ring + (size_t)st * DS_STAGE_BYTES;
                  ssc = sb + kc * 512 + g * 4;
                }
                const int ktl = itl * DS_ITEM_KT;
                if (ok) {
#pragma unroll
                  for (int q = 0; q < DS_ITEM_KT; ++q) {
                    if (ktl + q < kc) {
                      const uint4 wv = *reinterpret_cast<const uint4*>(sb + (ktl + q) * 512 + lane * 16);
                      const uint32_t sw = *reinterpret_cast<const uint32_t*>(ssc + ((ktl + q) >> gshift) * 32);
                      __half2 s_lo, s_hi;
                      split_scales(sw, s_lo, s_hi);
                      uint32_t af[4][4];
                      dequant8(wv.x, s_lo, s_hi, af[0]);
                      dequant8(wv.y, s_lo, s_hi, af[1]);
                      dequant8(wv.z, s_lo, s_hi, af[2]);
                      dequant8(wv.w, s_lo, s_hi, af[3]);
                      const uint4 b01 = bfr[qi][q][0], b23 = bfr[qi][q][1];
                      mma_16816(acc0, af[0], b01.x, b01.y);
                      mma_16816(acc1, af[1], b01.z, b01.w);
                      mma_16816(acc0, af[2], b23.x, b23.y);
                      mma_16816(acc1, af[3], b23.z, b23.w);
                    }
                  }
                }
                __syncwarp();
                // one arrival per item; the last item of a ragged chunk also arrives for the items the chunk lacks
                const int items_here = (kc + DS_ITEM_KT - 1) / DS_ITEM_KT;
                const int arrivals = (itl == items_here - 1) ? DS_ITEMS_PER_CHUNK - items_here + 1 : 1;
                if (lane < arrivals) mbar_arrive(smem_u32(empty_bar + st));
              }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[tl][e] = acc0[e] + acc1[e];
          }
        }
        // ---- 5. park the partial sums: [tile][warp][lane]
#pragma unroll
        for (int tl = 0; tl < DS_BT; ++tl)
          if (tl < nb) red[(size_t)(tl * DS_CWARPS + warp) * 32 + lane] = make_float4(acc[tl][0], acc[tl][1], acc[tl][2], acc[tl][3]);
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        ds_sync();

        // ---- 6. epilogue: one thread per (tile or pair, row, column)
        {
          const int ul = tid >> 7, m = (tid >> 4) & 7, c = tid & 15;      // unit of the batch, row, column
          const int n_ul = nb / tpu;
          const bool live = ul < n_ul && m < M;
          // accumulator layout of m16n8k16: lane (g,t) holds (out g, row 2t), (g, 2t+1), (g+8, 2t), (g+8, 2t+1)
          const int src_lane = (c & 7) * 4 + (m >> 1);
          const int e = (c >> 3) * 2 + (m & 1);
          float yv[2] = {0.f, 0.f};
          if (live) {
            const float inv = s_inv[m], fac = s_fac[m];
#pragma unroll
            for (int tu = 0; tu < 2; ++tu) {
              if (tu < tpu) {
                const int tl = ul * tpu + tu;
                float y = 0.f;
#pragma unroll
                for (int w = 0; w < DS_CWARPS; ++w)                       // fixed order
                  y += redf[((size_t)(tl * DS_CWARPS + w) * 32 + src_lane) * 4 + e];
                y *= inv;
                if (nseg > 0) {
                  const int ti = b0 + tl;
                  const int nt = (bid + (ti / tpu) * G) * tpu + (ti % tpu);
                  int seg, col;
                  map_col(ph.mode, nt * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
                  if (seg < nseg && ps.pB[seg][m] != nullptr) {
                    // LoRA expand (second factor of the low-rank term of Eq. 1-4)
                    const float* Tm = Ts + ((size_t)m * 3 + seg) * r;
                    const __half* bp = Bs + (((size_t)tl * CHAIN_MAX_ROWS + m) * r) * 16 + c;
                    float s0 = 0.f, s1 = 0.f;
                    for (int j = 0; j < r; j += 2) {
                      s0 = fmaf(Tm[j], __half2float(bp[(size_t)j * 16]), s0);
                      if (j + 1 < r) s1 = fmaf(Tm[j + 1], __half2float(bp[(size_t)(j + 1) * 16]), s1);
                    }
                    y += fac * (s0 + s1);
                  }
                }
                yv[tu] = y;
              }
            }
          }
          const int k_un = b0 / tpu + ul;                                 // the CTA's unit number
          const int u = bid + k_un * G;                                   // global unit
          if (ph.epi == EPI_F32) {
            if (live) {
              const int col = u * TILE_N + c;
              float* out = ph.out_f32 != nullptr ? ph.out_f32 : a.logits;
              if (out != nullptr) __stcg(out + (size_t)m * ph.ldo + col, yv[0]);
              if (track_max) {
                const unsigned long long key = ((unsigned long long)order_key(yv[0]) << 32) | (unsigned long long)(0xFFFFFFFFu - (uint32_t)col);
                best = key > best ? key : best;
              }
            }
          } else if (ph.epi == EPI_RESID) {
            if (ul < n_ul) {                                              // whole warps: see resid_out
              const float xo = live ? Xs[(k_un * CHAIN_MAX_ROWS + m) * TILE_N + c] : 0.f;
              resid_out(ph, k_un, ul, m, c, xo + yv[0], gpre, live);
            }
          } else {                                                        // EPI_SWIGLU: even tile = gate, odd tile = up
            if (live) {
              const float v = yv[0] / (1.f + __expf(-yv[0])) * yv[1];
              const __half vh = __float2half_rn(v);
              ph.out16[(size_t)m * (ph.N / 2) + u * TILE_N + c] = vh;
              Ys[(ul * CHAIN_MAX_ROWS + m) * TILE_N + c] = __half2float(vh);
            }
          }
        }
        ds_sync();
        // ---- 7. partial shrink sums of the consuming group over the batch's outputs
        if (ph.epi != EPI_F32) {
          shrink_partial(ps, nb / tpu, tp);
          if (b0 + bt < my_tiles) ds_sync();                              // the slices are about to be overwritten
        }
      }
      shrink_commit(ps, tp);
      if (track_max) {
        // the CTA's best (logit, lowest index) per row -> its slot of the exchange array
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
          const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        if ((tid & 15) == 0 && best != 0ull) atomicMax(&s_amax[(tid >> 4) & 7], best);
        ds_sync();
        if (tid < CHAIN_MAX_ROWS) __stcg(a.amax + (size_t)bid * CHAIN_MAX_ROWS + tid, s_amax[tid]);
      }
      // the ring position after this phase's chunks
      {
        int st = pos_st + my_tiles * L.nchunks;
        while (st >= nstages) { st -= nstages; pos_par ^= 1u; }
        pos_st = st;
      }
    } else if (kind == SK_ATTN) {
      // ------------------------------------------------------------------- attention of one layer
      // A CTA takes (stream s, kv head h): the stream's row against the shared prompt segment, the stream's own
      // cached rows and the row itself (App. A.1: a stream sees the prefill segment and its own segment only).
      // K and V fragments go from L2 straight into registers: the contraction index of QK^T is permuted so that a
      // lane's 16-byte loads are its fragments, the key pairs of the PV fragments are zipped with byte permutes.
      const int Hkv = a.Hkv, g_heads = a.Hq / Hkv;
      constexpr int HD = 64;
      const float scale_log2 = 1.4426950408889634f * rsqrtf((float)HD);
      __half* Qs = reinterpret_cast<__half*>(Ys);                         // [g_heads][HD], then the new k and v rows
      __half* Kn = Qs + 8 * HD;
      __half* Vn = Kn + HD;
      float* part = redf;                                                 // [warp][head][HD + 2]
      float* outs = redf + DS_CWARPS * g_heads * (HD + 2);                // [g_heads * HD] the unit's output rows
      const int Nqkv = (a.Hq + 2 * Hkv) * HD;
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
        // ---- LoRA-A slices of the o projection at this unit's columns: As[j][g_heads * HD]
        const int ocols = g_heads * HD;
        const __half* Ao = (lora_on && ph.next_nseg > 0) ? ps.pAn[0][s] : nullptr;
        if (Ao != nullptr) {
          const int ppr = ocols / 8;
          for (int idx = tid; idx < r * ppr; idx += DS_CTHREADS) {
            const int j = idx / ppr, x = idx - j * ppr;
            cp_async16_ca(As + (size_t)j * ocols + x * 8, Ao + (size_t)j * ph.next_ld + h * ocols + x * 8);
          }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // ---- the row's q heads (rotated), its new k (rotated) and v: fp16 into shared memory, k and v also into the cache
        {
          const float* prow = a.qkv + (size_t)s * Nqkv;
          const float2* csr = a.cs_table + (size_t)(a.P + S) * (HD / 2);
          const int nq = g_heads * (HD / 8);
          if (tid < nq) {
            const int hq = tid / (HD / 8), c = (tid % (HD / 8)) * 8;
            *reinterpret_cast<uint4*>(Qs + hq * HD + c) = head_piece_f16(prow + (size_t)(h * g_heads + hq) * HD, c, HD, csr);
          } else if (tid < nq + HD / 8) {
            const int c = (tid - nq) * 8;
            const uint4 v8 = head_piece_f16(prow + (size_t)(a.Hq + h) * HD, c, HD, csr);
            *reinterpret_cast<uint4*>(Kn + c) = v8;
            *reinterpret_cast<uint4*>(ok_ + (size_t)S * HD + c) = v8;
          } else if (tid < nq + 2 * (HD / 8)) {
            const int c = (tid - nq - HD / 8) * 8;
            const uint4 v8 = head_piece_f16(prow + (size_t)(a.Hq + Hkv + h) * HD, c, HD, nullptr);
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
        float o[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
        float mrow = -INFINITY, lrow = 0.f;
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
          const uint32_t pf[4] = {h2_as_u32(__floats2half2_rn(p0, p1)), 0u, h2_as_u32(__floats2half2_rn(p2, p3)), 0u};
          const uint32_t va[4] = {vf[0].x, vf[0].y, vf[0].z, vf[0].w}, vb2[4] = {vf[1].x, vf[1].y, vf[1].z, vf[1].w};
          const uint32_t vc[4] = {vf[2].x, vf[2].y, vf[2].z, vf[2].w}, vd[4] = {vf[3].x, vf[3].y, vf[3].z, vf[3].w};
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            o[i][0] *= corr; o[i][1] *= corr;
            const uint32_t sel = (i & 1) ? 0x7632u : 0x5410u;
            const uint32_t b0v = prmt(va[i >> 1], vb2[i >> 1], sel);       // (key 2t, key 2t+1) of column 8g + i
            const uint32_t b1v = prmt(vc[i >> 1], vd[i >> 1], sel);       // (key 2t+8, key 2t+9)
            mma_16816(o[i], pf, b0v, b1v);
          }
          if (ti + DS_CWARPS < n_tiles) load_tile(ti + DS_CWARPS);
        }
        // ---- the row itself as one more key, on the warp that would take the next tile
        if (warp == (n_tiles & (DS_CWARPS - 1))) {
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
          const uint4 v0v = *reinterpret_cast<const uint4*>(Vn + 16 * t), v1v = *reinterpret_cast<const uint4*>(Vn + 16 * t + 8);
          const uint32_t vw[8] = {v0v.x, v0v.y, v0v.z, v0v.w, v1v.x, v1v.y, v1v.z, v1v.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            // the lane's output columns are 16t + i (o[i][0]) and 16t + 8 + i (o[i][1])
            const float2 lo2 = __half22float2(u32_as_h2(vw[i >> 1])), hi2 = __half22float2(u32_as_h2(vw[4 + (i >> 1)]));
            o[i][0] = o[i][0] * corr + pn * ((i & 1) ? lo2.y : lo2.x);
            o[i][1] = o[i][1] * corr + pn * ((i & 1) ? hi2.y : hi2.x);
          }
        }
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 1);
        lrow += __shfl_xor_sync(0xffffffffu, lrow, 2);
        if (g < g_heads) {
          float* po = part + ((size_t)warp * g_heads + g) * (HD + 2);
#pragma unroll
          for (int i = 0; i < 8; ++i) { po[16 * t + i] = o[i][0]; po[16 * t + 8 + i] = o[i][1]; }
          if (t == 0) { po[HD] = mrow; po[HD + 1] = lrow; }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
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
        // ---- partial shrink sums of the o projection over this unit's columns: a warp per rank index
        if (Ao != nullptr) {
          for (int j = warp; j < r; j += DS_CWARPS) {
            float acc = 0.f;
            for (int c = lane; c < ocols; c += 32) acc = fmaf(outs[c], __half2float(As[(size_t)j * ocols + c]), acc);
            acc = warp_sum(acc);
            if (lane == 0) red_add_u64(a.tacc + ((size_t)ph.t_out * CHAIN_MAX_ROWS + s) * 3 * r + j, fix_of(acc));
          }
        }
        if (u + G < M * Hkv) ds_sync();                                   // the buffers are reused by the next unit
      }
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
    if (p + 1 < a.n_phases) {
      ++n_bar;
      ds_sync();
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
  }
}

// ----------------------------------------------------------------------------- host side
cudaError_t init_step() {
  return cudaFuncSetAttribute(decode_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 6144);
}

cudaError_t launch_step(const StepArgs& a, int sm_count, cudaStream_t st) {
  if (a.M < 1 || a.M > CHAIN_MAX_ROWS || a.nstages < DS_MIN_STAGES || a.nstages > DS_MAX_STAGES) return cudaErrorInvalidValue;
  const int r = (a.adapter_idx != nullptr) ? a.rank : a.rank;            // the carve-up is fixed per context
  const size_t smem = step_carve(r, a.own_tiles, a.as_bytes, a.nstages).total;
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
