// Shared device helpers and the kernel-launch interface between the translation units.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mlora {

// ----------------------------------------------------------------------------- layout constants
// Private weight layout ("fragment-major, chunked"): the [K][N] INT4 matrix is cut into tiles of 16 output
// features x 64 input features.  A tile is 32 lanes x 16 bytes: lane (g = lane/4, t = lane%4) owns the
// 16 consecutive input features k0+16t .. k0+16t+15 of output features n0+g and n0+g+8, so that one
// 128-bit load per lane feeds four m16n8k16 tensor-core steps (the weights are the 16-wide operand).
// Word j (0..3) of the lane's uint4 holds input features k0+16t+4j+{0,1,2,3}:
//   nibble 0/4: feature +0/+1 of row g      nibble 1/5: feature +0/+1 of row g+8
//   nibble 2/6: feature +2/+3 of row g      nibble 3/7: feature +2/+3 of row g+8
// The tiles of one n-tile (16 output features, all of K) form one contiguous "unit", cut into chunks of
// CHUNK_KT k-tiles.  A chunk is self-contained -- its weight tiles followed by the scales of the groups it
// covers (32 bytes per group: entry g packs the fp16 scale of row n0+g (low) and n0+g+8 (high)) -- so that
// one bulk copy brings everything a CTA needs for 512 input features of 16 outputs:
//   unit  = [chunk 0][chunk 1]...            chunk = [kc tiles x 512 B][groups x 32 B]
// Chunks start on group boundaries: G divides 512 or is a multiple of 512.
constexpr int TILE_N = 16;
constexpr int TILE_K = 64;
constexpr int CHUNK_KT = 8;                    // k-tiles per chunk (512 input features)

struct WLayout {
  int K, N, G, KT, NT, nchunks, kc_last, gpc, g_last;
  uint32_t chunk_full, chunk_last;             // bytes
  size_t unit_bytes;
};
// log2 of a power of two (group sizes below a chunk's 512 inputs are 64, 128 or 256: wlayout_group_ok)
__host__ __device__ inline int wl_log2(int v) {
#ifdef __CUDA_ARCH__
  return 31 - __clz(v);
#else
  int s = 0;
  while ((1 << (s + 1)) <= v) ++s;
  return s;
#endif
}
__host__ __device__ inline WLayout make_wlayout(int K, int N, int G) {
  WLayout L;
  L.K = K; L.N = N; L.G = G;
  L.KT = K / TILE_K; L.NT = N / TILE_N;
  L.nchunks = (L.KT + CHUNK_KT - 1) / CHUNK_KT;
  L.kc_last = L.KT - (L.nchunks - 1) * CHUNK_KT;
  const int ck = CHUNK_KT * TILE_K;
  // (G < ck: a power of two, so the divisions are shifts -- these run at the start of every kernel)
  L.gpc = G >= ck ? 1 : ck >> wl_log2(G);
  L.g_last = G >= ck ? 1 : (L.kc_last * TILE_K + G - 1) >> wl_log2(G);
  L.chunk_full = CHUNK_KT * 512 + L.gpc * 32;
  L.chunk_last = L.kc_last * 512 + L.g_last * 32;
  L.unit_bytes = (size_t)(L.nchunks - 1) * L.chunk_full + L.chunk_last;
  return L;
}
__host__ __device__ inline bool wlayout_group_ok(int G) {
  const int ck = CHUNK_KT * TILE_K;
  return G > 0 && G % TILE_K == 0 && (ck % G == 0 || G % ck == 0);
}
// byte offset, inside a unit, of k-tile kt's weights and of the scale entry of its group
__host__ __device__ inline size_t wl_tile_off(const WLayout& L, int kt) {
  return (size_t)(kt / CHUNK_KT) * L.chunk_full + (size_t)(kt % CHUNK_KT) * 512;
}
__host__ __device__ inline size_t wl_scale_off(const WLayout& L, int kt) {
  const int c = kt / CHUNK_KT;
  const int kc = (c == L.nchunks - 1) ? L.kc_last : CHUNK_KT;
  const int gi = (L.G >= CHUNK_KT * TILE_K) ? 0 : ((kt % CHUNK_KT) * TILE_K) >> wl_log2(L.G);
  return (size_t)c * L.chunk_full + (size_t)kc * 512 + (size_t)gi * 32;
}

// GEMM CTA shape
constexpr int GEMM_WARPS = 4;
constexpr int GEMM_THREADS = GEMM_WARPS * 32;
constexpr int GEMM_NB = GEMM_WARPS * TILE_N;   // output features per CTA
constexpr int GEMM_PF = 8;                     // weight tiles in flight per lane
constexpr int GEMM_MAX_MT = 16;                // m-tiles of 8 rows per CTA (128 rows)

enum GemmMode { MODE_PLAIN = 0, MODE_QKV = 1, MODE_GATEUP = 2 };
enum GemmEpi { EPI_F32 = 0, EPI_RESID = 1, EPI_SWIGLU = 2 };

struct LoraSeg {
  int proj_index;   // index into the adapter pointer tables (layer*7 + proj), or the plain table index 0
  int n;            // logical output width of the segment
};

struct LoraArgs {
  const int32_t* adapter_idx;     // dev: adapter of stream (row / rows_per_stream); nullptr => no LoRA
  int rows_per_stream;
  const __half* const* tabA;      // dev [n_slots][tab_stride]
  const __half* const* tabB;
  const float* scale;             // dev [n_slots]
  int tab_stride;
  int n_slots;
  int rank;
  int nseg;
  LoraSeg seg[3];
  float* T;                       // dev fp32 [M][nseg][rank], already multiplied by the adapter scale
};

struct GemmArgs {
  const unsigned char* w;         // packed weights (chunked fragment-major layout)
  int K, N, G;                    // N = physical (fused) width
  const __half* h;                // [M][K]
  int M;
  int mode, epi;
  int seg_n0, seg_n1;             // MODE_QKV: widths of the first two segments
  float* out_f32; int ldo;        // EPI_F32
  float* resid;                   // EPI_RESID: [M][N] in place
  __half* out_f16;                // EPI_SWIGLU: [M][N/2]
  float* partial;                 // split-K scratch [ksplit][M][N]
  size_t partial_capacity;        // floats
  unsigned* counters;             // zeroed, >= n_blocks * m_blocks entries
  LoraArgs lora;
};

struct ShrinkArgs {
  const float* x_f32;             // NORM mode: residual stream [M][K]
  const __half* gain;             // NORM mode: RMSNorm gain
  float eps;
  const __half* h_in;             // PLAIN mode: fp16 input [M][K]
  __half* h_out;                  // NORM mode: normalised fp16 rows written here
  int M, K;
  LoraArgs lora;                  // adapter_idx == nullptr: only the norm is done
};

struct AttnArgs {
  const __half* q;                // [rows][Hq][hd]
  const __half* prefix_k; const __half* prefix_v; size_t prefix_head_stride; int P;
  const __half* own_k; const __half* own_v; size_t own_stream_stride, own_head_stride;
  const int32_t* suffix_len;      // dev [n]
  int suffix_bound;               // host upper bound on suffix_len
  const unsigned long long* anc;  // dev [n][T] ancestor-or-self bit masks
  int causal;                     // the pass's rows form a chain (prefill): row t sees new rows 0..t, anc is not read
  int n, T, Hq, Hkv, hd;
  __half* out;                    // [rows][Hq][hd]
  float* part_o; float* part_ml;  // scratch
  int n_prefix_chunks, prefix_chunk; // keys per prefix chunk (multiple of 64)
  int n_own_chunks, own_chunk;
  // fused mode (qkv_f32 != nullptr): q and the pass's new k rows are rotated here (RoPE, Sec. 3.1) and the new K/V
  // rows are written to the own segment by the CTA that owns their chunk; q is not read
  const float* qkv_f32;           // [rows][(Hq + 2 Hkv) * hd] fp32 projections
  const float2* cs_table;         // cos/sin of pos * theta^(-2i/hd): [pos][hd/2]
  int pos_base;                   // position of a row = pos_base + suffix_len[s] + depth[row]
  const int32_t* depth;           // dev [rows]
  int stream_mode;                // set by attn_plan: the streaming kernel for one row per stream over a long prefix
  int* status;                    // dev status word for bounded waits that run out (may be null)
  // single-kernel decode attention only: partial LoRA shrink of the o projection over the (kv head, stream)'s output
  // features, added to 64-bit fixed-point sums (o_tacc == nullptr: not wanted)
  unsigned long long* o_tacc;     // [8 rows][3][o_rank] of the o projection's group
  const __half* const* o_tabA;    // adapter A pointers [slot][o_tab_stride]
  const int32_t* o_adapter_idx;   // dev [n]
  int o_proj_index, o_rank, o_tab_stride, o_n_slots;
  long long* trace0;              // timeline of a traced step (nullptr otherwise): this launch's 12 slots
  int o_direct;                   // o_tabA is indexed by stream (looked up once per call): o_adapter_idx is not read
  int pdl;                        // launch the single-kernel decode attention with programmatic stream serialisation
};

// ----------------------------------------------------------------------------- persistent projection chain
// A "phase" is one fused projection group of the decoder (q,k,v | o | gate,up | down | lm_head) over at most
// 8 rows.  The chain kernel runs a range of phases back to back with a grid barrier between them.
enum ChainIn { IN_NORM = 0, IN_F16 = 1 };
struct ChainPhase {
  const unsigned char* w;         // packed weights
  int K, N, G;                    // N = physical (fused) width
  int mode, epi, in_kind;
  int seg_n0, seg_n1;             // MODE_QKV: widths of the first two segments
  const float* x_f32;             // IN_NORM: residual stream [M][K]
  const __half* gain;             // IN_NORM: RMSNorm gain [K]
  const __half* h_in;             // IN_F16: [M][K]
  float* out_f32; int ldo;        // EPI_F32 (nullptr: the call's logits destination)
  float* resid;                   // EPI_RESID: [M][N] in place
  __half* out_f16;                // EPI_SWIGLU: [M][N/2]
  int lora_nseg;                  // 0: no LoRA on this group
  int lora_proj[3];               // index into the adapter pointer tables per segment
  int lora_n[3];                  // logical output width per segment
};
// a strided region of global memory that the kernel launched next will read (the next attention's K/V): the chain
// kernel asks for it in L2 while its last phase runs
struct ChainPrefetch {
  const unsigned char* base;      // nullptr: nothing
  unsigned n_outer, outer_stride, inner;   // n_outer runs of `inner` bytes, `outer_stride` bytes apart (multiples of 16)
};
struct ChainArgs {
  const ChainPhase* phases;       // dev
  int p0, p1;                     // phase range [p0, p1)
  int M;
  float eps;
  float* logits;                  // destination of a phase whose out_f32 is nullptr
  const __half* h_in;             // input of an IN_F16 phase whose h_in is nullptr
  const int32_t* adapter_idx;     // dev; nullptr: base weights only
  int rows_per_stream;
  const __half* const* tabA;
  const __half* const* tabB;
  const float* scale;
  int tab_stride, n_slots, rank;
  float* T;                       // dev fp32 [M][3][rank] scratch
  unsigned long long* sync;       // dev [4]: grid-barrier arrivals, shrink arrivals, abort flag, spare
  int* status;                    // dev status word
  long long wait_cycles;          // clock limit of every wait (0: the default, about two seconds)
  int inject_stall;               // test hook: the launch's first grid barrier waits for an arrival nobody makes
  int nstages;                    // ring stages
  int kmax;                       // largest K of the phases in range (sizes the activation buffer)
  ChainPrefetch pf[4];
};
constexpr int CHAIN_MAX_ROWS = 8;
constexpr int CHAIN_MAX_RANK = 64;
cudaError_t init_chain();
// shared memory the chain kernel needs for the given largest K and rank with `nstages` ring stages; 0 if it cannot fit
size_t chain_smem_bytes(int kmax, int rank, int nstages);
int chain_pick_stages(int kmax, int rank);      // most stages that fit (0: not eligible)
// whether one projection group (K inputs, nseg LoRA segments) can run in the chain kernel with that many stages
bool chain_phase_fits(int K, int mode, int nseg, int rank, int nstages, int sm_count);
cudaError_t launch_chain(const ChainArgs& a, int sm_count, cudaStream_t st);

// ----------------------------------------------------------------------------- whole decode step in one kernel
// One decode step (one row per stream, at most 8 rows) as ONE persistent cooperative kernel: embedding, every
// projection group, the attention of every layer, lm_head, row argmax and the suffix-length update are phases
// separated by grid barriers.
enum StepKind { SK_EMBED = 0, SK_GEMM = 1, SK_ATTN = 2, SK_FIN = 3 };
constexpr unsigned long long LEAN_PF_MAX_BYTES = 16ull << 20;   // at most this much of the next group's weights is asked for in L2
struct StepPhase {
  int kind, layer;
  const unsigned char* w;         // SK_GEMM: packed weights
  int K, N, G;                    // N = physical (fused) width; SK_EMBED: N = d_model
  int mode, epi;
  int seg_n0, seg_n1;             // MODE_QKV: widths of the first two segments
  const __half* in16;             // SK_GEMM: input rows fp16 [8][K]
  int norm_in;                    // index of the sums of squares that normalise the input rows (-1: used as they are)
  int ldo;
  float* out_f32;                 // EPI_F32 (nullptr: the call's logits destination)
  __half* out16;                  // EPI_SWIGLU: [8][N/2]; EPI_RESID / SK_EMBED: x * gain_next [8][N]; SK_ATTN: [8][Hq*hd]
  const __half* gain_next;        // EPI_RESID / SK_EMBED: gain of the RMSNorm that follows (nullptr: none)
  int ssq_out;                    // where the sums of squares of the new residual rows are accumulated (-1: nowhere)
  int lora_nseg;                  // 0: no LoRA on this group
  int lora_proj[3];               // index into the adapter pointer tables per segment
  int lora_n[3];                  // logical output width per segment
  int t_in;                       // index of this group's accumulated shrink sums
  int next_nseg;                  // LoRA segments of the group that consumes this phase's outputs (0: none)
  int next_proj[3];
  int next_ld;                    // row length of their A matrices (= that group's K)
  int t_out;                      // where the partial shrink sums over this phase's outputs are accumulated
  int last;                       // the residual rows this phase writes are the call's hidden-state output
  int pad_;
  const unsigned char* pf_w;      // kernel-per-projection path: packed weights of the projection group that runs next,
  unsigned long long pf_bytes;    // asked for in L2 by this phase's CTAs (a share each); 0: nothing
};
struct StepArgs {
  const StepPhase* phases;        // dev
  int n_phases;
  int M;                          // rows = streams
  float eps;
  const int32_t* tokens;          // dev [M] (nullptr: hidden-state input)
  const __half* embed; int vocab;
  const __half* hidden_in;        // dev fp16 [M][d_model]
  const int32_t* adapter_idx;     // dev [M]; nullptr: base weights only
  const __half* const* tabA;
  const __half* const* tabB;
  const float* scale;
  int tab_stride, n_slots, rank;
  const unsigned char* tmapA;     // dev [n_slots][tab_stride] tensor maps (STEP_TMAP_BYTES each) over the A / B matrices:
  const unsigned char* tmapB;     // boxes of 16 columns x rank rows
  // attention
  int Hq, Hkv, hd, P;
  const float* qkv;               // fp32 [8][(Hq + 2 Hkv) hd]: q,k,v projections of the layer
  const __half* prefix_k; const __half* prefix_v; size_t prefix_layer_stride, prefix_head_stride;
  __half* own_k; __half* own_v; size_t own_layer_stride, own_stream_stride, own_head_stride;
  int32_t* suffix_len;            // dev [M]: read at the start, advanced by one at the end
  const float2* cs_table;
  // outputs
  float* logits;                  // dev fp32 [M][vocab] or nullptr
  int32_t* out_next;              // dev [M] greedy tokens (vocab > 0)
  float* hidden_out;              // dev fp32 [M][d_model] (vocab == 0)
  unsigned long long* amax;       // dev [grid][8]: per-CTA row maxima of the logits
  // accumulators (64-bit fixed point, zero at launch; the kernel leaves them zero)
  unsigned long long* tacc;       // [n_tacc][8][3][rank]
  unsigned long long* ssq;        // [n_ssq][8]
  int n_tacc, n_ssq;
  unsigned long long* sync;       // dev [4]: grid-barrier arrivals, spare, abort flag, where the first wait gave up
  int* status;
  long long wait_cycles;
  int inject_stall;
  int nstages, own_tiles;
  long long* trace;               // dev [2][n_phases][12] nanosecond stamps of the first and the last CTA, or nullptr
};
cudaError_t init_step();
// ring stages the step kernel gets for this model on this device (0: the kernel cannot run it)
int step_plan(int d_model, int d_ffn, int Nq, int Nkv, int hd, int rank, int lora_targets, int sm_count, int* own_tiles);
constexpr int STEP_TMAP_BYTES = 128;
// tensor map (STEP_TMAP_BYTES, host memory) over one LoRA matrix fp16 [rank][width] for the step kernel's slice copies
cudaError_t step_encode_slice_map(const void* base, int width, int rank, void* map_out);
cudaError_t launch_step(const StepArgs& a, int sm_count, cudaStream_t st);

// ----------------------------------------------------------------------------- launchers
cudaError_t init_gemm();        // opt-in shared-memory sizes; call once per process before the first launch
cudaError_t init_shrink();
cudaError_t init_attention();
// repack: logical n-tile nt of the canonical [K][N] matrix goes to physical unit dst_tile_off + nt*dst_tile_stride
cudaError_t launch_repack(const uint8_t* qweight, const __half* scales, int K, int N, int G, unsigned char* w,
                          int dst_tile_off, int dst_tile_stride, cudaStream_t st);
cudaError_t launch_dequant(const unsigned char* w, int K, int N, int G, int tile_off, int tile_stride,
                           __half* out, cudaStream_t st);
int gemm_pick_split(int K, int N, int M, size_t partial_capacity);
cudaError_t launch_gemm(const GemmArgs& a, cudaStream_t st);
// tcgen05 path for passes with 32 rows or more: partial sums on the tensor cores, then an epilogue kernel
cudaError_t init_gemm_tc();
bool gemm_tc_eligible(const GemmArgs& a);
cudaError_t launch_gemm_tc(const GemmArgs& a, int sm_count, int* status, cudaStream_t st);
cudaError_t launch_shrink(const ShrinkArgs& a, cudaStream_t st);
cudaError_t launch_embed(const int32_t* tokens, const __half* embed, const __half* hidden_in, float* X, int M,
                         int d, int vocab, int* status, cudaStream_t st, const __half* forecast = nullptr,
                         int n_forecast = 0);
cudaError_t launch_draft(const float* logits, int V, int n, int R, int m, int wmax, const int32_t* widths,
                         const int32_t* level, const int32_t* rank, const int32_t* forecast_of, const int32_t* acc_len,
                         const int32_t* acc_idx, const int32_t* next, int32_t* cand, int32_t* out_tokens, int* status,
                         cudaStream_t st);
cudaError_t launch_tree_prep(const int32_t* parent, int n, int T, unsigned long long* anc, int32_t* depth,
                             int* status, cudaStream_t st);
void attn_plan(AttnArgs& a, int sm_count);
size_t attn_workspace_floats(const AttnArgs& a);
bool attn_decode_o_slice_fits(int hd, int g_heads, int rank);
bool attn_single_pass(const AttnArgs& a);          // one kernel does the whole softmax: no merge launch follows
cudaError_t launch_attention(const AttnArgs& a, cudaStream_t st);
cudaError_t launch_attention_merge(const AttnArgs& a, cudaStream_t st);
cudaError_t launch_argmax(const float* logits, int M, int V, int32_t* out, cudaStream_t st);
cudaError_t launch_topn(const float* logits, int V, int n, int32_t* out, cudaStream_t st);
cudaError_t launch_accept(const int32_t* tokens, const int32_t* parent, const int32_t* argmax, int n, int T,
                          int32_t* acc_len, int32_t* acc_idx, int32_t* next, cudaStream_t st);
cudaError_t launch_compact(__half* own_k, __half* own_v, size_t layer_stride, size_t stream_stride,
                           size_t head_stride, int L, int n, int Hkv, int hd, const int32_t* suffix_len,
                           const int32_t* acc_len, const int32_t* acc_idx, int T, cudaStream_t st);
cudaError_t launch_advance(int32_t* suffix_len, const int32_t* acc_len, int n, int fixed, cudaStream_t st);
// ---- decode step as one small kernel per projection group (decode_lean.cu)
struct LeanArgs {
  int M;
  float eps;
  const int32_t* adapter_idx;     // dev [M] or nullptr
  const __half* const* tabA;
  const __half* const* tabB;
  const float* scale;
  int tab_stride, n_slots, rank;
  float* X;                       // residual stream fp32 [M][d_model]
  float* logits;                  // destination of a phase whose out_f32 is null
  unsigned long long* tacc;       // [n_tacc][8][3][rank]
  unsigned long long* ssq;        // [n_ssq][8]
  long long* trace0;              // timeline of a traced step (nullptr otherwise): 12 slots of this launch for its first CTA
  long long* trace1;              // ... and for its last CTA
  int rank_log2;                  // log2(rank) when the rank is a power of two, else -1 (index arithmetic by shifts)
  int rows_direct;                // tabA / tabB / scale are indexed by ROW (looked up once per call): adapter_idx is not read
  int late_wait;                  // the kernel ahead produces only T: wait for it after the main loop, not before
  unsigned long long* amax;       // [8]: row maxima of the lm_head as (ordered value, complemented column) keys, zero at
                                  // the start of a step; non-null = no logits are written, the greedy tokens come from here
};
inline int lean_rank_log2(int r) {                     // LeanArgs::rank_log2
  if (r <= 0 || (r & (r - 1)) != 0) return -1;
  int s = 0;
  while ((1 << s) < r) ++s;
  return s;
}
cudaError_t launch_lean_rowptr(const int32_t* adapter_idx, const __half* const* tabA, const __half* const* tabB, const float* scale,
                               int n_slots, int tab_stride, int M, const __half** rowA, const __half** rowB, float* rowscale,
                               cudaStream_t st);
cudaError_t launch_lean_finish(const unsigned long long* amax, int32_t* out_next, int32_t* suffix_len, int n, cudaStream_t st);
cudaError_t init_lean();
bool lean_shapes_ok(int d_model, int d_ffn, int Nq, int Nkv, int rank);
cudaError_t launch_lean_embed(const LeanArgs& a, const StepPhase& ph, const int32_t* tokens, const __half* embed, int vocab,
                              const __half* hidden_in, int* status, cudaStream_t st);
cudaError_t launch_lean_gemm(const LeanArgs& a, const StepPhase& ph, cudaStream_t st);
cudaError_t launch_quant_act(const __half* x, long long count, float scale, signed char* out, cudaStream_t st);
bool w4a8_shape_ok(int M, int K, int N);
cudaError_t launch_w4a8(const unsigned char* w, const __half* ws, const signed char* x, float x_scale, int M, int K, int N,
                        float* y, cudaStream_t st);
cudaError_t launch_copy_rows_f32(const float* src, float* dst, size_t count, cudaStream_t st);

// ----------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ldg_nc_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// Eight INT4 weights -> four fp16x2 registers in m16n8k16 A-fragment order.  Each stored nibble u = q + 8
// is placed into the mantissa of 1024.0 (giving 1024+u, or 1024+16u for the nibbles one hex digit up),
// q = u - 8 is recovered exactly by one subtract / fused multiply-add, and the dequantised weight is the
// single correctly-rounded fp16 product q * scale.
__device__ __forceinline__ void dequant8(uint32_t w, __half2 s_lo, __half2 s_hi, uint32_t (&a)[4]) {
  const uint32_t MAGIC = 0x64006400u;                       // (1024.0, 1024.0)
  const __half2 k1032 = u32_as_h2(0x64086408u);             // 1032.0
  const __half2 k16th = u32_as_h2(0x2C002C00u);             // 1/16
  const __half2 km72 = u32_as_h2(0xD480D480u);              // -72.0
  const uint32_t w8 = w >> 8;
  const __half2 x0 = u32_as_h2((w & 0x000F000Fu) | MAGIC);
  const __half2 x1 = u32_as_h2((w & 0x00F000F0u) | MAGIC);
  const __half2 x2 = u32_as_h2((w8 & 0x000F000Fu) | MAGIC);
  const __half2 x3 = u32_as_h2((w8 & 0x00F000F0u) | MAGIC);
  a[0] = h2_as_u32(__hmul2(__hsub2(x0, k1032), s_lo));
  a[1] = h2_as_u32(__hmul2(__hfma2(x1, k16th, km72), s_hi));
  a[2] = h2_as_u32(__hmul2(__hsub2(x2, k1032), s_lo));
  a[3] = h2_as_u32(__hmul2(__hfma2(x3, k16th, km72), s_hi));
}
__device__ __forceinline__ void split_scales(uint32_t sw, __half2& s_lo, __half2& s_hi) {
  s_lo = u32_as_h2(__byte_perm(sw, sw, 0x1010));
  s_hi = u32_as_h2(__byte_perm(sw, sw, 0x3232));
}
// physical column of a fused projection -> (segment, logical column)
__device__ __forceinline__ void map_col(int mode, int c, int n0, int n1, int& seg, int& col) {
  if (mode == MODE_PLAIN) { seg = 0; col = c; }
  else if (mode == MODE_QKV) {
    if (c < n0) { seg = 0; col = c; }
    else if (c < n0 + n1) { seg = 1; col = c - n0; }
    else { seg = 2; col = c - n0 - n1; }
  } else {                         // gate/up interleaved by 16-column tiles
    const int tile = c >> 4;
    seg = tile & 1;
    col = ((tile >> 1) << 4) | (c & 15);
  }
}
// eight consecutive elements c..c+7 of one head of a projection row, rotated (pairs (i, i + hd/2), Sec. 3.1) or not.
// All loads are issued before the first use; the row was written by another kernel or CTA: read through L2.
__device__ __forceinline__ uint4 head_piece_f16(const float* __restrict__ head, int c, int hd, const float2* __restrict__ cs) {
  const float4 x0 = __ldcg(reinterpret_cast<const float4*>(head + c));
  const float4 x1 = __ldcg(reinterpret_cast<const float4*>(head + c + 4));
  float v[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
  if (cs != nullptr) {
    const int half = hd >> 1;
    const bool lo = c < half;                          // a piece never straddles the middle: c and hd/2 are multiples of 8
    const int pc = lo ? c + half : c - half;           // the partner piece
    const float4 y0 = __ldcg(reinterpret_cast<const float4*>(head + pc));
    const float4 y1 = __ldcg(reinterpret_cast<const float4*>(head + pc + 4));
    const float4* t4 = reinterpret_cast<const float4*>(cs + (lo ? c : pc));
    const float4 t0 = __ldg(t4), t1 = __ldg(t4 + 1), t2 = __ldg(t4 + 2), t3 = __ldg(t4 + 3);
    const float y[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
    const float co[8] = {t0.x, t0.z, t1.x, t1.z, t2.x, t2.z, t3.x, t3.z};
    const float si[8] = {t0.y, t0.w, t1.y, t1.w, t2.y, t2.w, t3.y, t3.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = lo ? v[i] * co[i] - y[i] * si[i] : v[i] * co[i] + y[i] * si[i];
  }
  __half2 o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) o[i] = __halves2half2(__float2half_rn(v[2 * i]), __float2half_rn(v[2 * i + 1]));
  return make_uint4(h2_as_u32(o[0]), h2_as_u32(o[1]), h2_as_u32(o[2]), h2_as_u32(o[3]));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
#endif

}  // namespace mlora
