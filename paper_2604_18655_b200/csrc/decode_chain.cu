// Persistent projection chain for decode-sized batches (at most 8 rows): a range of fused projection groups
// of the decoder (Sec. 3.1; LoRA term of Eq. 1-4 with the adapter picked per row, Sec. 3.2 (c); INT4 weights,
// Sec. 3.3) runs inside ONE cooperative kernel, one CTA per SM, with a grid barrier between groups.
//
// Why: at these sizes a projection moves a few MB -- about a microsecond of HBM time -- so a kernel per
// projection is bound by launch and ramp-up latency.  Here a producer warp streams the CTA's share of the
// packed INT4 weights (and of the LoRA-A rows) of ALL phases through a shared-memory ring with bulk
// asynchronous copies (cp.async.bulk + mbarrier transaction counts).  They do not depend on activations, so
// the ring keeps filling while the consumer warps sit in a grid barrier or in a prologue: HBM never idles
// across phase boundaries.  Sixteen consumer warps (four per scheduler, to hide latency) work in teams: a team
// takes one n-tile (or gate/up pair) at a time, its warps split K, dequantise in registers and multiply on the
// tensor cores (mma.sync m16n8k16: weights are the 16-wide operand, the rows the 8-wide one), add their
// partial sums through shared memory in a fixed order and run the epilogue (LoRA expand, residual add, SwiGLU,
// fp32 store) on their own, behind a named barrier of the team.
//
// The LoRA shrink T = (alpha/r) h A^T is spread over all CTAs at the start of a phase; a counter tells every
// CTA when all of T is in global memory; the expand happens in the epilogue from 32-byte slices of B that the
// team fetched with cp.async before the phase's prologue.
//
// Every wait (mbarrier, grid barrier, shrink counter) is bounded by a clock limit.  When one runs out the CTA
// raises a global abort flag and the status word MLORA_ERR_TIMEOUT and records which wait it was; from then on
// every wait returns at once and the kernel runs its (data-independent) control flow to the end, so no CTA is
// left in a barrier.
#include "pipe.cuh"

namespace mlora {

constexpr int CH_CWARPS = 16;                      // consumer warps
constexpr int CH_CTHREADS = CH_CWARPS * 32;
constexpr int CH_THREADS = CH_CTHREADS + 32;       // + one producer warp
constexpr int CH_STAGE_BYTES = 4480;               // >= CHUNK_KT*512 + 8*32, multiple of 128
constexpr int CH_MAX_STAGES = 40;
constexpr int CH_MAX_ITEMS = 16;                   // shrink items per CTA per phase
constexpr int CH_ITEM_KT = 2;                      // k-tiles per GEMM work item
constexpr int CH_ITEMS_PER_CHUNK = CHUNK_KT / CH_ITEM_KT;   // = arrivals that free a ring stage
constexpr int CH_A_PIECE = 2048;                   // halves of a LoRA-A row per ring stage
constexpr int CH_RED_BYTES = 2 * CH_CWARPS * 512;  // partial sums: one slot per consumer warp and tile of a pair
constexpr int CH_BS_BYTES = 24 * 1024;             // LoRA-B slices of the teams' units: [team][tile][row][j][16] fp16
constexpr int CH_MAX_TEAMS = 8;

static_assert(CH_STAGE_BYTES >= CHUNK_KT * 512 + 8 * 32, "stage too small for a chunk");
static_assert(CH_STAGE_BYTES >= CH_A_PIECE * 2, "stage too small for an A piece");

__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(CH_CTHREADS) : "memory"); }

// ----------------------------------------------------------------------------- shared-memory carve-up
struct ChainSmem {
  size_t bars, red, bs, ts, hs, ring, total;
};
__host__ __device__ inline ChainSmem chain_carve(int kmax, int rank, int nstages) {
  ChainSmem s;
  size_t o = 0;
  s.bars = o; o += 1024;                                                   // mbarriers
  s.red = o; o += (size_t)CH_RED_BYTES;                                    // partial sums [tile of pair][warp][lane]
  s.bs = o; o += (size_t)(rank > 0 ? CH_BS_BYTES : 0);                     // LoRA-B slices
  s.ts = o; o += (size_t)CHAIN_MAX_ROWS * 3 * (rank > 0 ? rank : 1) * 4;   // T of the phase
  o = (o + 127) / 128 * 128;
  s.hs = o; o += (size_t)CHAIN_MAX_ROWS * (kmax + 8) * 2;                  // activations fp16 [8][K+8]
  o = (o + 127) / 128 * 128;
  s.ring = o; o += (size_t)nstages * CH_STAGE_BYTES;
  s.total = o;
  return s;
}

// A consumer may never wait a whole ring lap ahead of the fill front (mbarrier parities repeat every two laps):
// one unit's chunks, and the A rows of a CTA's shrink items, must fit the ring.
bool chain_phase_fits(int K, int mode, int nseg, int rank, int nstages, int sm_count) {
  const WLayout L = make_wlayout(K, TILE_N, TILE_K);
  const int tpu = (mode == MODE_GATEUP) ? 2 : 1;
  if (tpu * L.nchunks > nstages) return false;
  if (nseg > 0 && rank > 0) {
    const int items = (CHAIN_MAX_ROWS * nseg * rank + sm_count - 1) / sm_count;
    const int np = (K + CH_A_PIECE - 1) / CH_A_PIECE;
    if (items > CH_MAX_ITEMS || items * np > nstages || np > 8) return false;   // 2 np partial sums per item fit 16 slots
    if (CH_BS_BYTES / (tpu * CHAIN_MAX_ROWS * rank * 32) < 1) return false;     // one unit's B slices must fit
  }
  return true;
}

size_t chain_smem_bytes(int kmax, int rank, int nstages) { return chain_carve(kmax, rank, nstages).total; }

int chain_pick_stages(int kmax, int rank) {
  if (rank > CHAIN_MAX_RANK || kmax % TILE_K) return 0;
  const size_t limit = 227 * 1024 - 3584;        // static shared memory of the kernel comes on top
  const size_t base = chain_carve(kmax, rank, 0).total;
  if (base >= limit) return 0;
  int n = (int)((limit - base) / CH_STAGE_BYTES);
  if (n > CH_MAX_STAGES) n = CH_MAX_STAGES;
  return n >= 8 ? n : 0;
}

// what every consumer thread needs of a phase beyond its descriptor; worked out once per phase by one thread (the
// divisions in it would otherwise sit at the head of every thread's phase, ahead of its first loads)
static_assert(sizeof(ChainPhase) == 128, "a phase descriptor is loaded as one word per lane");
struct PhaseDerived {
  WLayout L;
  int tpu, n_units, ipt, gshift, my_units, teams, n_my_items, shr_warps, gemm_warps;
  int n_valid;                       // the CTA's shrink items whose row has an adapter, in item order
  int item_i[CH_MAX_ITEMS];          // their index (row, segment, rank index) = position in T
  int item_sm[CH_MAX_ITEMS];         // their segment | row << 8
};

// ----------------------------------------------------------------------------- the ring schedule
// Everything immutable and bulky that a CTA needs flows through the ring in one fixed order, known to the
// producer and to the consumers alike.  Per phase:
//   1. for each shrink item of the CTA (row m, segment, rank index j) whose row has an adapter: the row j of
//      A in pieces of CH_A_PIECE halves, one stage per piece;
//   2. for each unit of the CTA, per tile, the weight chunks.
struct Ring {
  int stage;
  uint32_t parity;
  int nstages;
  __device__ __forceinline__ void advance() { if (++stage == nstages) { stage = 0; parity ^= 1; } }
};

// RMSNorm (Sec. 3.1) of up to 8 rows by all consumer threads: thread `tid` owns the float4 columns
// tid + i*CH_CTHREADS (i < NVR) of EVERY row, so the gain is loaded once per thread and the rows stay in
// registers between the sum of squares and the scaling.  The rows were written by other CTAs: read through L2.
template <int NVR>
__device__ __forceinline__ void norm_rows(const float* __restrict__ x, const __half* __restrict__ gain, int K, int M,
                                          float eps, __half* hs, int hs_stride, float* s_ssw, float* s_inv, int tid) {
  const int warp = tid >> 5, lane = tid & 31;
  const int nvec = K >> 2;
  float4 xv[NVR][CHAIN_MAX_ROWS];
  uint2 gv[NVR];
  float ss[CHAIN_MAX_ROWS];
#pragma unroll
  for (int m = 0; m < CHAIN_MAX_ROWS; ++m) ss[m] = 0.f;
#pragma unroll
  for (int i = 0; i < NVR; ++i) {
    const int v = tid + i * CH_CTHREADS;
    const bool in = v < nvec;
    gv[i] = in ? __ldg(reinterpret_cast<const uint2*>(gain) + v) : make_uint2(0, 0);
#pragma unroll
    for (int m = 0; m < CHAIN_MAX_ROWS; ++m)
      xv[i][m] = (in && m < M) ? __ldcg(reinterpret_cast<const float4*>(x + (size_t)m * K) + v) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int i = 0; i < NVR; ++i)
#pragma unroll
    for (int m = 0; m < CHAIN_MAX_ROWS; ++m)
      ss[m] += xv[i][m].x * xv[i][m].x + xv[i][m].y * xv[i][m].y + xv[i][m].z * xv[i][m].z + xv[i][m].w * xv[i][m].w;
#pragma unroll
  for (int m = 0; m < CHAIN_MAX_ROWS; ++m) {
    ss[m] = warp_sum(ss[m]);
    if (lane == 0) s_ssw[warp * CHAIN_MAX_ROWS + m] = ss[m];
  }
  consumer_sync();
  if (tid < CHAIN_MAX_ROWS) {
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < CH_CWARPS; ++w) tot += s_ssw[w * CHAIN_MAX_ROWS + tid];
    s_inv[tid] = rsqrtf(tot / (float)K + eps);
  }
  consumer_sync();
#pragma unroll
  for (int i = 0; i < NVR; ++i) {
    const int v = tid + i * CH_CTHREADS;
    if (v < nvec) {
      const float2 g01 = __half22float2(u32_as_h2(gv[i].x)), g23 = __half22float2(u32_as_h2(gv[i].y));
#pragma unroll
      for (int m = 0; m < CHAIN_MAX_ROWS; ++m) {
        if (m < M) {
          const float inv = s_inv[m];
          const __half2 o01 = __floats2half2_rn(xv[i][m].x * inv * g01.x, xv[i][m].y * inv * g01.y);
          const __half2 o23 = __floats2half2_rn(xv[i][m].z * inv * g23.x, xv[i][m].w * inv * g23.y);
          *reinterpret_cast<uint2*>(hs + (size_t)m * hs_stride + 4 * v) = make_uint2(h2_as_u32(o01), h2_as_u32(o23));
        }
      }
    }
  }
}

// ----------------------------------------------------------------------------- the kernel
__global__ void __launch_bounds__(CH_THREADS, 1) decode_chain_kernel(const ChainArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ ChainPhase s_ph[2];
  __shared__ PhaseDerived s_pd[2];
  __shared__ const __half* s_pA[2][3][CHAIN_MAX_ROWS];
  __shared__ const __half* s_pB[2][3][CHAIN_MAX_ROWS];
  __shared__ float s_scale[CHAIN_MAX_ROWS];
  __shared__ int s_adapter[CHAIN_MAX_ROWS];
  __shared__ int s_abort_word;
  __shared__ volatile unsigned s_t_ready;             // LoRA phases of this launch whose T is in shared memory
  __shared__ unsigned long long s_base[2];
  __shared__ float s_shr_part[CH_MAX_ITEMS][16];      // shrink: partial sums of an item's half pieces
  __shared__ float s_ssw[CH_CWARPS * CHAIN_MAX_ROWS];  // RMSNorm: per-warp sums of squares of every row
  __shared__ float s_inv[CHAIN_MAX_ROWS];

  const int nstages = a.nstages;
  const ChainSmem cs = chain_carve(a.kmax, a.rank, nstages);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + cs.bars);
  uint64_t* empty_bar = full_bar + CH_MAX_STAGES;
  float4* red = reinterpret_cast<float4*>(smem + cs.red);
  __half* Bs = reinterpret_cast<__half*>(smem + cs.bs);
  float* Ts = reinterpret_cast<float*>(smem + cs.ts);
  __half* hs = reinterpret_cast<__half*>(smem + cs.hs);
  unsigned char* ring = smem + cs.ring;

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const unsigned G = gridDim.x;
  const int M = a.M;
  const int r = a.rank;
  const int r2_shift = (r > 0 && (r & (r - 1)) == 0) ? 32 - __clz(r) : -1;   // log2(2 r) for power-of-two ranks
  const bool lora_on = a.adapter_idx != nullptr && a.rank > 0;
  WaitCtx wc{a.wait_cycles > 0 ? a.wait_cycles : PIPE_WAIT_CYCLES, &s_abort_word, a.sync, a.status};

  // ---- set-up: barriers, first phase descriptor, adapters of the rows, counter bases
  if (tid == 0) {
    for (int s = 0; s < nstages; ++s) {
      mbar_init(smem_u32(full_bar + s), 1);
      mbar_init(smem_u32(empty_bar + s), CH_ITEMS_PER_CHUNK);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_abort_word = (ld_acquire_u64(a.sync + 2) != 0ull) ? 1 : 0;
    s_t_ready = 0u;
    // arrivals of earlier launches are whole multiples of the grid size; arrivals of this launch that are
    // already counted are fewer than one grid
    s_base[0] = ld_acquire_u64(a.sync + 0) / G * G;
    s_base[1] = ld_acquire_u64(a.sync + 1) / G * G;
  }
  if (tid < CHAIN_MAX_ROWS) {
    int ad = -1;
    float sc = 0.f;
    if (lora_on && tid < M) {
      ad = a.adapter_idx[tid / a.rows_per_stream];
      if (ad < 0 || ad >= a.n_slots) ad = -1;
      else sc = a.scale[ad];
    }
    s_adapter[tid] = ad;
    s_scale[tid] = sc;
  }
  __syncthreads();

  // loads phase descriptor p and the rows' adapter pointers into slot (p - p0) & 1 (one warp)
  auto prep_phase = [&](int p) {
    const int slot = (p - a.p0) & 1;
    const int* src = reinterpret_cast<const int*>(a.phases + p);
    int* dst = reinterpret_cast<int*>(&s_ph[slot]);
    for (int i = lane; i < (int)(sizeof(ChainPhase) / 4); i += 32) dst[i] = __ldg(src + i);
    __syncwarp();
    if (lane < 3 * CHAIN_MAX_ROWS) {
      const int seg = lane / CHAIN_MAX_ROWS, m = lane % CHAIN_MAX_ROWS;
      const __half *pa = nullptr, *pb = nullptr;
      const int ad = s_adapter[m];
      if (lora_on && seg < s_ph[slot].lora_nseg && ad >= 0) {
        const size_t e = (size_t)ad * a.tab_stride + s_ph[slot].lora_proj[seg];
        pa = a.tabA[e];
        pb = a.tabB[e];
        if (pa == nullptr || pb == nullptr) { pa = nullptr; pb = nullptr; }
      }
      s_pA[slot][seg][m] = pa;
      s_pB[slot][seg][m] = pb;
    }
  };
  // the phase's derived values, by one thread, once its descriptor is in shared memory
  auto derive_phase = [&](int p) {
    const int slot = (p - a.p0) & 1;
    {
      const ChainPhase& ph = s_ph[slot];
      PhaseDerived& d = s_pd[slot];
      d.L = make_wlayout(ph.K, ph.N, ph.G);
      const int nseg = lora_on ? ph.lora_nseg : 0;
      d.tpu = (ph.mode == MODE_GATEUP) ? 2 : 1;
      d.n_units = d.L.NT / d.tpu;
      d.ipt = (d.L.KT + CH_ITEM_KT - 1) / CH_ITEM_KT;                 // items per tile
      d.gshift = (d.L.G >= CHUNK_KT * TILE_K) ? 31 : (31 - __clz(d.L.G / TILE_K));   // k-tile -> scale group of its chunk
      // teams: as many units in flight as the CTA has, as the ring can hold at once (a wait must never be a whole
      // lap ahead of the fill front: mbarrier parities repeat every two laps) and as the B buffer has room for
      d.my_units = (d.n_units > (int)blockIdx.x) ? (d.n_units - 1 - (int)blockIdx.x) / (int)G + 1 : 0;
      int teams = d.my_units < CH_MAX_TEAMS ? d.my_units : CH_MAX_TEAMS;
      if (teams > nstages / (d.tpu * d.L.nchunks)) teams = nstages / (d.tpu * d.L.nchunks);
      if (nseg > 0 && teams > CH_BS_BYTES / (d.tpu * CHAIN_MAX_ROWS * r * 32)) teams = CH_BS_BYTES / (d.tpu * CHAIN_MAX_ROWS * r * 32);
      if (teams < 1) teams = 1;
      // LoRA phases: the CTA's shrink items (row, segment, rank index) run on the last shr_warps warps, off the
      // critical path of the GEMM teams, which share the other warps
      d.n_my_items = 0;
      if (nseg > 0) {
        const int n_items = M * nseg * r;
        d.n_my_items = (n_items > (int)blockIdx.x) ? (n_items - 1 - (int)blockIdx.x) / (int)G + 1 : 0;
        if (d.n_my_items > CH_MAX_ITEMS) d.n_my_items = CH_MAX_ITEMS;
      }
      d.n_valid = 0;
      for (int k = 0; k < d.n_my_items; ++k) {
        const int i = blockIdx.x + k * (int)G;
        const int seg = (i / r) % nseg, m = i / (r * nseg);
        if (s_pA[slot][seg][m] == nullptr) continue;
        d.item_i[d.n_valid] = i;
        d.item_sm[d.n_valid] = seg | (m << 8);
        ++d.n_valid;
      }
      // one shrink warp per half piece of 1024 features, four at most for tile pairs
      {
        const int n_half = d.n_valid * 2 * ((ph.K + CH_A_PIECE - 1) / CH_A_PIECE);
        // (eight where a unit is a single tile: there the wait for T, not the GEMM, ends the phase)
        const int cap = d.tpu == 1 ? 8 : 4;
        d.shr_warps = nseg > 0 ? (n_half < cap ? (n_half > 0 ? n_half : 1) : cap) : 0;
      }
      d.gemm_warps = CH_CWARPS - d.shr_warps;
      if (teams > d.gemm_warps) teams = d.gemm_warps;
      d.teams = teams;
    }
  };
  if (warp == 0) {
    prep_phase(a.p0);
    __syncwarp();
    if (lane == 0) derive_phase(a.p0);
  }
  __syncthreads();

  // =========================================================================== producer warp
  if (warp == CH_CWARPS) {
    const uint64_t policy = policy_evict_first();
    Ring rg{0, 1u, nstages};                         // a fresh "empty" barrier passes a wait on parity 1
    long long issued = 0;
    bool alive = true;
    int cur_phase = a.p0;
    // lane 0 waits for the stage to be free; every lane learns the outcome
    auto acquire = [&]() -> bool {
      int ok = 1;
      if (lane == 0) ok = wait_mbar(smem_u32(empty_bar + rg.stage), rg.parity, wc, 1, cur_phase) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      return ok != 0;
    };
    for (int p = a.p0; p < a.p1 && alive; ++p) {
      cur_phase = p;
      if (p == a.p1 - 1) {
        // last phase of the launch: what the next kernel reads first (its K/V) is asked for in L2 now, in 4 KB
        // pieces dealt over the CTAs and lanes
#pragma unroll 1
        for (int d = 0; d < 4; ++d) {
          const ChainPrefetch f = a.pf[d];
          if (f.base == nullptr || f.inner == 0u) continue;
          const unsigned ppo = (f.inner + 4095u) / 4096u, total = f.n_outer * ppo;
          for (unsigned i = blockIdx.x * 32u + lane; i < total; i += G * 32u) {
            const unsigned o = i / ppo, off = (i - o * ppo) * 4096u;
            const unsigned bytes = min(4096u, f.inner - off);
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(f.base + (size_t)o * f.outer_stride + off), "r"(bytes) : "memory");
          }
        }
      }
      const ChainPhase* ph = a.phases + p;           // immutable: read the descriptor from global
      const unsigned char* wbase = ph->w;
      const int mode = ph->mode, K = ph->K;
      const WLayout L = make_wlayout(K, ph->N, ph->G);
      const int nseg = lora_on ? ph->lora_nseg : 0;
      // LoRA-A matrices of the rows for this phase: lane (seg, m)
      const __half* myA = nullptr;
      if (nseg > 0 && lane < 3 * CHAIN_MAX_ROWS) {
        const int seg = lane / CHAIN_MAX_ROWS, m = lane % CHAIN_MAX_ROWS;
        const int ad = s_adapter[m];
        if (seg < nseg && ad >= 0) {
          const size_t e = (size_t)ad * a.tab_stride + ph->lora_proj[seg];
          myA = a.tabA[e];
          if (myA == nullptr || a.tabB[e] == nullptr) myA = nullptr;
        }
      }
      // ---- 1. rows of A for the CTA's shrink items
      if (nseg > 0) {
        const int n_items = M * nseg * r;
        int my = 0;
        for (int i = blockIdx.x; i < n_items && my < CH_MAX_ITEMS && alive; i += G, ++my) {
          const int j = i % r, seg = (i / r) % nseg, m = i / (r * nseg);
          const __half* A = reinterpret_cast<const __half*>(
              __shfl_sync(0xffffffffu, (unsigned long long)myA, seg * CHAIN_MAX_ROWS + m));
          if (A == nullptr) continue;
          for (int k0 = 0; k0 < K; k0 += CH_A_PIECE) {
            if (!acquire()) { alive = false; break; }
            if (lane == 0) {
              const uint32_t bytes = (uint32_t)min(CH_A_PIECE, K - k0) * 2;
              const uint32_t fb = smem_u32(full_bar + rg.stage);
              mbar_expect_tx(fb, bytes);
              bulk_g2s(smem_u32(ring + (size_t)rg.stage * CH_STAGE_BYTES), A + (size_t)j * K + k0, bytes, fb, policy);
            }
            ++issued;
            rg.advance();
          }
        }
      }
      // ---- 2. units: weight chunks
      const int tpu = (mode == MODE_GATEUP) ? 2 : 1;
      const int n_units = L.NT / tpu;
      for (int u = blockIdx.x; u < n_units && alive; u += G) {
        for (int tu = 0; tu < tpu && alive; ++tu) {
          const unsigned char* unit = wbase + (size_t)(u * tpu + tu) * L.unit_bytes;
          for (int c = 0; c < L.nchunks; ++c) {
            if (!acquire()) { alive = false; break; }
            if (lane == 0) {
              const uint32_t bytes = (c == L.nchunks - 1) ? L.chunk_last : L.chunk_full;
              const uint32_t fb = smem_u32(full_bar + rg.stage);
              mbar_expect_tx(fb, bytes);
              bulk_g2s(smem_u32(ring + (size_t)rg.stage * CH_STAGE_BYTES), unit + (size_t)c * L.chunk_full, bytes, fb, policy);
            }
            ++issued;
            rg.advance();
          }
        }
      }
    }
    if (!alive && lane == 0) {
      // abort: the copies already issued still land; wait (bounded) for the stages that may be in flight
      const long long t0 = clock64();
      const long long inflight = issued < nstages ? issued : nstages;
      for (long long k = 1; k <= inflight; ++k) {
        const long long idx = issued - k;            // k-th last stage filled
        const int st = (int)(idx % nstages);
        const uint32_t par = (uint32_t)((idx / nstages) & 1);
        while (!mbar_try_wait(smem_u32(full_bar + st), par)) {
          if (clock64() - t0 > wc.limit) break;
        }
      }
    }
    return;                                           // consumers use named barriers; nothing below is for this warp
  }

  // =========================================================================== consumer warps
  // The CTA's stages of a phase form one list (see "the ring schedule"); a consumer finds a stage by its
  // running count since the start of the launch.
  //   shrink item k   -> warp k % 16 reads all pieces of the row and frees each stage on its own
  //   weight chunks   -> warps work in teams, formed anew for every round of units: in a round team tm takes the
  //                      CTA's next unit number tm; inside a unit
  //                      every tile's k-tiles are cut into items of CH_ITEM_KT k-tiles and each member warp owns a
  //                      contiguous run of them, keeps their partial sums in registers and parks them in its own
  //                      slot; the team adds the slots in member order (fixed summation order) and runs the
  //                      epilogue.  A stage is free again after CH_ITEMS_PER_CHUNK arrivals, one per item.
  const int g = lane >> 2, t = lane & 3;
  int pos = 0;                                        // stages of this CTA consumed (or skipped) so far
  unsigned long long n_bar = 0;                       // barriers passed in this launch
  unsigned n_shr = 0;                                 // LoRA phases passed in this launch
  float* redf = reinterpret_cast<float*>(red);
  for (int p = a.p0; p < a.p1; ++p) {
    const int slot = (p - a.p0) & 1;
    const ChainPhase& ph = s_ph[slot];
    const int K = ph.K;
    const int hs_stride = K + 8;
    const PhaseDerived& pd = s_pd[slot];
    const WLayout L = pd.L;
    const int nseg = lora_on ? ph.lora_nseg : 0;
    const int tpu = pd.tpu, ipt = pd.ipt, gshift = pd.gshift, my_units = pd.my_units, teams = pd.teams;
    const int shr_warps = pd.shr_warps, gemm_warps = pd.gemm_warps;
    // the teams are formed anew for every round of units: the last round may have fewer units than teams, and
    // then all GEMM warps share what is left
    int teams_r = 0, wpt = 1, tm = 0, member = 0, team_threads = 32, tt = 0;
    bool in_team = false;
    __half* Bs_team = Bs;
    auto form_teams = [&](int units_left) {
      teams_r = units_left < teams ? units_left : teams;
      if (teams_r < 1) teams_r = 1;
      wpt = gemm_warps / teams_r;                                     // warps per team
      tm = warp / wpt;
      member = warp - tm * wpt;
      in_team = tm < teams_r;
      team_threads = wpt * 32;
      tt = member * 32 + lane;
      Bs_team = Bs + (size_t)tm * tpu * CHAIN_MAX_ROWS * r * 16;
    };
    form_teams(my_units);
    const int shr_id = warp - gemm_warps;                             // >= 0: this warp is shrink warp shr_id
    auto team_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(2 + tm), "r"(team_threads) : "memory"); };
    // LoRA-B slices of unit u -> Bs_team[tile][m][j][16]; immutable, so no need to wait for activations
    auto issue_b = [&](int u) {
      const int r2 = r * 2;                                            // 16-byte pieces per row of a tile
      for (int tu = 0; tu < tpu; ++tu) {
        int seg, col;
        map_col(ph.mode, (u * tpu + tu) * TILE_N, ph.seg_n0, ph.seg_n1, seg, col);
        if (seg >= nseg) continue;
        const int ldb = ph.lora_n[seg];
        for (int idx = tt; idx < M * r2; idx += team_threads) {
          const int m = r2_shift >= 0 ? idx >> r2_shift : idx / r2;
          const int x = idx - m * r2, j = x >> 1, h16 = x & 1;
          const __half* B = s_pB[slot][seg][m];
          if (B != nullptr)
            cp_async16_ca(Bs_team + (((size_t)tu * CHAIN_MAX_ROWS + m) * r + j) * 16 + h16 * 8,
                          B + (size_t)j * ldb + col + h16 * 8);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };
    if (nseg > 0 && in_team && tm < my_units) issue_b(blockIdx.x + tm * (int)G);

    // ---- 1. activations of the phase -> shared memory, fp16 [8][K+8]
    if (ph.in_kind == IN_NORM) {
      const int nvec = K >> 2;
      if (nvec <= CH_CTHREADS) norm_rows<1>(ph.x_f32, ph.gain, K, M, a.eps, hs, hs_stride, s_ssw, s_inv, tid);
      else if (nvec <= 2 * CH_CTHREADS) norm_rows<2>(ph.x_f32, ph.gain, K, M, a.eps, hs, hs_stride, s_ssw, s_inv, tid);
      else {
        // wide rows: two passes, warps 2m and 2m+1 own the halves of row m
        const int m = warp >> 1, hf = warp & 1;
        const int kh = K / 2;
        const float* x = ph.x_f32 + (size_t)m * K + hf * kh;
        const __half* gp = ph.gain + hf * kh;
        float ss = 0.f;
        if (m < M) {
          for (int k = lane * 4; k < kh; k += 128) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(x + k));
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          }
          ss = warp_sum(ss);
        }
        if (lane == 0) s_ssw[warp] = ss;
        consumer_sync();
        if (m < M) {
          const float inv = rsqrtf((s_ssw[2 * m] + s_ssw[2 * m + 1]) / (float)K + a.eps);
          __half* dst = hs + (size_t)m * hs_stride + hf * kh;
          for (int k = lane * 4; k < kh; k += 128) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(x + k));
            const uint2 gw = __ldg(reinterpret_cast<const uint2*>(gp + k));
            const float2 g01 = __half22float2(u32_as_h2(gw.x)), g23 = __half22float2(u32_as_h2(gw.y));
            const __half2 o01 = __floats2half2_rn(v.x * inv * g01.x, v.y * inv * g01.y);
            const __half2 o23 = __floats2half2_rn(v.z * inv * g23.x, v.w * inv * g23.y);
            *reinterpret_cast<uint2*>(dst + k) = make_uint2(h2_as_u32(o01), h2_as_u32(o23));
          }
        }
      }
    } else {
      const int vec_per_row = K / 8;
      const __half* h_in = ph.h_in != nullptr ? ph.h_in : a.h_in;
      for (int i = tid; i < M * vec_per_row; i += CH_CTHREADS) {
        const int m = i / vec_per_row, k = (i % vec_per_row) * 8;
        *reinterpret_cast<uint4*>(hs + (size_t)m * hs_stride + k) =
            __ldcg(reinterpret_cast<const uint4*>(h_in + (size_t)m * K + k));
      }
    }
    consumer_sync();

    // ---- 2. next phase's descriptor and adapter pointers (immutable) while this phase runs: warp 0 issues the
    // loads here and stores what they return further down, so neither round trip holds anything up
    const bool prep_next = warp == 0 && p + 1 < a.p1;
    const int nslot = slot ^ 1;
    int prep_word = 0;
    const __half *prep_pa = nullptr, *prep_pb = nullptr;
    if (prep_next) prep_word = __ldg(reinterpret_cast<const int*>(a.phases + p + 1) + lane);

    // ---- 3. LoRA shrink (first factor of the low-rank term of Eq. 1-4): items (row, segment, rank index)
    // are dealt round-robin to the CTAs; item k of the CTA belongs to shrink warp k % shr_warps
    if (nseg > 0) {
      const int np = (K + CH_A_PIECE - 1) / CH_A_PIECE;
      // The items with an adapter were listed when the phase was set up; only the shrink warps walk them.  An item
      // (one rank index of one row: a dot product over K) is cut into half pieces of 1024 features that are dealt
      // to the shrink warps, so that a long row (K = 5632: six halves) does not sit on one warp; the partial sums
      // are added in order by the first shrink warp, which also tells the grid that the CTA's share of T is written.
      if (shr_id >= 0) {
        const int hp = 2 * np;                                            // half pieces per item
        const int n_half = pd.n_valid * hp;
        const int st0 = pos_stage(pos, nstages);
        const uint32_t par0 = pos_parity(pos, nstages);
        int kk = 0, hq = shr_id;                                          // item and half piece of unit un, stepped
        for (int un = shr_id; un < n_half; un += shr_warps, hq += shr_warps) {
          while (hq >= hp) { hq -= hp; ++kk; }
          const int q = hq >> 1, hf = hq & 1;
          const int m = pd.item_sm[kk] >> 8;
          // the CTA's A pieces of a phase fit the ring (checked on the host): at most one wrap from the first
          int st = st0 + kk * np + q;
          uint32_t par = par0;
          if (st >= nstages) { st -= nstages; par ^= 1u; }
          const bool ok = wait_mbar(smem_u32(full_bar + st), par, wc, 2, p);
          const int k0 = q * CH_A_PIECE + hf * (CH_A_PIECE / 2);
          const unsigned char* sb = ring + (size_t)st * CH_STAGE_BYTES + hf * CH_A_PIECE;   // bytes: half a piece
          const __half* hrow = hs + (size_t)m * hs_stride + k0;
          float acc4[4] = {0.f, 0.f, 0.f, 0.f};
          if (ok) {
#pragma unroll
            for (int v = 0; v < CH_A_PIECE / 512; ++v) {
              const int off = v * 256 + lane * 8;                         // halves inside the half piece
              if (k0 + off < K) {
                const uint4 av = *reinterpret_cast<const uint4*>(sb + off * 2);
                const uint4 hv = *reinterpret_cast<const uint4*>(hrow + off);
                const uint32_t aw[4] = {av.x, av.y, av.z, av.w};
                const uint32_t hw[4] = {hv.x, hv.y, hv.z, hv.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float2 af = __half22float2(u32_as_h2(aw[e])), hf2 = __half22float2(u32_as_h2(hw[e]));
                  acc4[e] = fmaf(af.x, hf2.x, acc4[e]);
                  acc4[e] = fmaf(af.y, hf2.y, acc4[e]);
                }
              }
            }
          }
          __syncwarp();
          if (lane < CH_ITEMS_PER_CHUNK / 2) mbar_arrive(smem_u32(empty_bar + st));   // the two halves free the stage
          const float acc = warp_sum((acc4[0] + acc4[1]) + (acc4[2] + acc4[3]));
          if (lane == 0) s_shr_part[kk][hq] = acc;
        }
        asm volatile("bar.sync 11, %0;" ::"r"(shr_warps * 32) : "memory");
        if (shr_id == 0) {
          if (lane < pd.n_valid) {
            float tot = 0.f;
            for (int hq = 0; hq < hp; ++hq) tot += s_shr_part[lane][hq];
            __stcg(a.T + pd.item_i[lane], tot * s_scale[pd.item_sm[lane] >> 8]);
          }
          // the warp barrier orders the lanes' stores before lane 0's release, which is cumulative over them
          __syncwarp();
          if (lane == 0) red_release_add_u64(a.sync + 1, 1ull);
          // This warp has nothing else to do in the phase: it watches for the other CTAs' shares and brings all of
          // T into shared memory as soon as it is complete, so that the GEMM teams, when their main loop ends, find
          // it there instead of paying a counter poll and a load round trip each.
          if (lane == 0) wait_counter(a.sync + 1, s_base[1] + (unsigned long long)(n_shr + 1u) * G, wc, 4, p);
          __syncwarp();
          for (int i = lane; i < M * nseg * r; i += 32) Ts[i] = __ldcg(a.T + i);
          __threadfence_block();
          __syncwarp();
          if (lane == 0) s_t_ready = n_shr + 1u;
        }
      }
      pos += np * pd.n_valid;
      ++n_shr;
    }
    if (prep_next) {
      reinterpret_cast<int*>(&s_ph[nslot])[lane] = prep_word;
      __syncwarp();
      if (lane < 3 * CHAIN_MAX_ROWS) {
        const int seg = lane / CHAIN_MAX_ROWS, m = lane % CHAIN_MAX_ROWS;
        const int ad = s_adapter[m];
        if (lora_on && seg < s_ph[nslot].lora_nseg && ad >= 0) {
          const size_t e = (size_t)ad * a.tab_stride + s_ph[nslot].lora_proj[seg];
          prep_pa = a.tabA[e];
          prep_pb = a.tabB[e];
        }
      }
    }

    // ---- 4. the CTA's units: one n-tile (or a gate/up pair of n-tiles), all of K
    bool t_loaded = false;
    for (int k0 = 0; k0 < my_units && warp < gemm_warps; k0 += teams_r) {
      if (k0 > 0) {
        // next round: every GEMM warp is done with the last one (partial sums, B slices and T are settled)
        asm volatile("bar.sync 10, %0;" ::"r"(gemm_warps * 32) : "memory");
        form_teams(my_units - k0);
        t_loaded = true;
      }
      if (in_team) {
        const int it_lo = (member * ipt) / wpt, it_hi = ((member + 1) * ipt) / wpt;   // this warp's items of a tile
        const int k = k0 + tm;
        const int u = blockIdx.x + k * (int)G;
        if (nseg > 0 && k0 > 0) issue_b(u);                               // the first round's went out before the prologue
        const int ubase = pos + k * tpu * L.nchunks;                      // first stage of the unit
        for (int tu = 0; tu < tpu; ++tu) {
          float acc0[4] = {0.f, 0.f, 0.f, 0.f}, acc1[4] = {0.f, 0.f, 0.f, 0.f};
          // the warp's items it_lo .. it_hi-1 lie in consecutive chunks; stage and parity of a chunk are stepped,
          // not divided out again (the loop is a serial chain per warp: every instruction in it counts)
          int c = it_lo / CH_ITEMS_PER_CHUNK;
          int st = 0;
          uint32_t par = 0;
          if (it_lo < it_hi) {
            const int P0 = ubase + tu * L.nchunks + c;
            st = pos_stage(P0, nstages);
            par = pos_parity(P0, nstages);
          }
          const __half* hrow = hs + (size_t)g * hs_stride + 16 * t;
          for (int it = it_lo; it < it_hi; ++c) {
            const int kc = (c == L.nchunks - 1) ? L.kc_last : CHUNK_KT;
            const int items_here = (kc + CH_ITEM_KT - 1) / CH_ITEM_KT;
            const int it_end = min(it_hi, (c + 1) * CH_ITEMS_PER_CHUNK);
            const bool ok = wait_mbar(smem_u32(full_bar + st), par, wc, 3, p);
            const unsigned char* sb = ring + (size_t)st * CH_STAGE_BYTES;
            const unsigned char* ssc = sb + kc * 512 + g * 4;
            const uint32_t ebar = smem_u32(empty_bar + st);
            for (; it < it_end; ++it) {
              const int itl = it - c * CH_ITEMS_PER_CHUNK;                // item inside its chunk
              const int ktl = itl * CH_ITEM_KT;                           // its first k-tile inside the chunk
              if (ok) {
                const __half* hbase = hrow + (size_t)(c * CHUNK_KT + ktl) * TILE_K;
#pragma unroll
                for (int q = 0; q < CH_ITEM_KT; ++q) {
                  if (ktl + q < kc) {
                    const uint4 wv = *reinterpret_cast<const uint4*>(sb + (ktl + q) * 512 + lane * 16);
                    const uint32_t sw = *reinterpret_cast<const uint32_t*>(ssc + ((ktl + q) >> gshift) * 32);
                    const uint4 b01 = *reinterpret_cast<const uint4*>(hbase + q * TILE_K);
                    const uint4 b23 = *reinterpret_cast<const uint4*>(hbase + q * TILE_K + 8);
                    __half2 s_lo, s_hi;
                    split_scales(sw, s_lo, s_hi);
                    uint32_t af[4][4];
                    dequant8(wv.x, s_lo, s_hi, af[0]);
                    dequant8(wv.y, s_lo, s_hi, af[1]);
                    dequant8(wv.z, s_lo, s_hi, af[2]);
                    dequant8(wv.w, s_lo, s_hi, af[3]);
                    mma_16816(acc0, af[0], b01.x, b01.y);
                    mma_16816(acc1, af[1], b01.z, b01.w);
                    mma_16816(acc0, af[2], b23.x, b23.y);
                    mma_16816(acc1, af[3], b23.z, b23.w);
                  }
                }
              }
              __syncwarp();
              // one arrival per item; the last item of a ragged chunk also arrives for the items the chunk lacks
              const int arrivals = (itl == items_here - 1) ? CH_ITEMS_PER_CHUNK - items_here + 1 : 1;
              if (lane < arrivals) mbar_arrive(ebar);
            }
            if (++st == nstages) { st = 0; par ^= 1u; }
          }
          red[(size_t)(tu * CH_CWARPS + warp) * 32 + lane] =
              make_float4(acc0[0] + acc1[0], acc0[1] + acc1[1], acc0[2] + acc1[2], acc0[3] + acc1[3]);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        team_sync();
        if (nseg > 0 && !t_loaded) {
          // all of T must be in shared memory before the first expand: the first shrink warp puts it there
          if (tt == 0) {
            const long long t0 = clock64();
            for (int it = 0; s_t_ready < n_shr; ++it) {
              if ((it & 255) == 255) {
                if (*wc.s_abort) break;
                if (clock64() - t0 > wc.limit) { raise_abort(wc, 4, p); break; }
              }
            }
          }
          team_sync();
          t_loaded = true;
        }
        // ---- epilogue of the unit: one thread per (row, column)
        for (int o = tt; o < CHAIN_MAX_ROWS * TILE_N; o += team_threads) {
          const int m = o >> 4, col16 = o & 15;
          if (m >= M) continue;
          // accumulator layout of m16n8k16: lane (g,t) holds (out g, row 2t), (g, 2t+1), (g+8, 2t), (g+8, 2t+1)
          const int src_lane = (col16 & 7) * 4 + (m >> 1);
          const int e = (col16 >> 3) * 2 + (m & 1);
          float yv[2] = {0.f, 0.f};
          int colv[2] = {0, 0};
#pragma unroll
          for (int tu = 0; tu < 2; ++tu) {
            if (tu < tpu) {
              const int nt = u * tpu + tu;
              float y = 0.f;
              for (int j = 0; j < wpt; ++j)                               // fixed order: member 0, 1, ...
                y += redf[((size_t)(tu * CH_CWARPS + tm * wpt + j) * 32 + src_lane) * 4 + e];
              int seg, col;
              map_col(ph.mode, nt * TILE_N + col16, ph.seg_n0, ph.seg_n1, seg, col);
              if (nseg > 0 && seg < nseg && s_pB[slot][seg][m] != nullptr) {
                // LoRA expand (second factor of the low-rank term of Eq. 1-4)
                const float* Tm = Ts + ((size_t)m * nseg + seg) * r;
                const __half* bp = Bs_team + (((size_t)tu * CHAIN_MAX_ROWS + m) * r) * 16 + col16;
                float s0 = 0.f, s1 = 0.f;
                for (int j = 0; j < r; j += 2) {
                  s0 = fmaf(Tm[j], __half2float(bp[(size_t)j * 16]), s0);
                  if (j + 1 < r) s1 = fmaf(Tm[j + 1], __half2float(bp[(size_t)(j + 1) * 16]), s1);
                }
                y += s0 + s1;
              }
              yv[tu] = y;
              colv[tu] = col;
            }
          }
          const int nt0 = u * tpu;
          if (ph.epi == EPI_F32) {
            float* out = ph.out_f32 != nullptr ? ph.out_f32 : a.logits;
            __stcg(out + (size_t)m * ph.ldo + nt0 * TILE_N + col16, yv[0]);
          } else if (ph.epi == EPI_RESID) {
            float* xp = ph.resid + (size_t)m * ph.N + nt0 * TILE_N + col16;
            __stcg(xp, __ldcg(xp) + yv[0]);
          } else {                                     // EPI_SWIGLU: even tile = gate, odd tile = up
            const float v = yv[0] / (1.f + __expf(-yv[0])) * yv[1];
            ph.out_f16[(size_t)m * (ph.N / 2) + colv[1]] = __float2half_rn(v);
          }
        }
        team_sync();                                   // the team's partial sums and B slices may be rewritten
      }
    }
    pos += my_units * tpu * L.nchunks;
    if (prep_next && lane < 3 * CHAIN_MAX_ROWS) {
      if (prep_pa == nullptr || prep_pb == nullptr) { prep_pa = nullptr; prep_pb = nullptr; }
      s_pA[nslot][lane / CHAIN_MAX_ROWS][lane % CHAIN_MAX_ROWS] = prep_pa;
      s_pB[nslot][lane / CHAIN_MAX_ROWS][lane % CHAIN_MAX_ROWS] = prep_pb;
    }

    // ---- 5. grid barrier: the next phase reads what every CTA wrote
    if (p + 1 < a.p1) {
      ++n_bar;
      consumer_sync();
      if (tid == 0) {
        // the release is cumulative over what the CTA's threads wrote before the named barrier above; the
        // acquire load inside wait_counter orders the next phase's reads after the other CTAs' writes
        red_release_add_u64(a.sync + 0, 1ull);
        // (test hook: with inject_stall the first barrier of the launch waits for one arrival too many)
        wait_counter(a.sync + 0, s_base[0] + n_bar * G + ((a.inject_stall && n_bar == 1) ? 1ull : 0ull), wc, 5, p);
      }
      // while thread 0 waits for the other CTAs: the next phase's derived values (its descriptor was loaded
      // before the barrier above)
      if (tid == 32) derive_phase(p + 1);
      consumer_sync();
    }
  }
}


// ----------------------------------------------------------------------------- host side
cudaError_t init_chain() {
  return cudaFuncSetAttribute(decode_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 3584);
}

cudaError_t launch_chain(const ChainArgs& a, int sm_count, cudaStream_t st) {
  if (a.M < 1 || a.M > CHAIN_MAX_ROWS || a.nstages < 2 || a.nstages > CH_MAX_STAGES) return cudaErrorInvalidValue;
  const size_t smem = chain_smem_bytes(a.kmax, a.rank, a.nstages);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)sm_count);
  cfg.blockDim = dim3(CH_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;          // all CTAs resident: the grid barrier needs it
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_chain_kernel, a);
}

}  // namespace mlora
