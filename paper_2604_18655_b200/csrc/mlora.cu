// Host side of the C ABI: context, weight repacking, the launch sequence of one decode / verify pass,
// CUDA-graph replay of steps, per-family event timing.  Every step of the path runs in the kernels of
// this library; there is no CPU or library fallback.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_map>
#include <vector>

#include "../../include/mlora.h"
#include "common.cuh"

using namespace mlora;

namespace {

thread_local std::string g_last_error;

struct PackedWeight {
  unsigned char* data = nullptr;   // chunked fragment-major layout: nibbles and scales interleaved per chunk
  int K = 0, N = 0, G = 0;         // N = physical width (all fused segments)
};

cudaError_t alloc_packed(PackedWeight& w, int K, int N, int G) {
  w.K = K; w.N = N; w.G = G;
  const WLayout L = make_wlayout(K, N, G);
  return cudaMalloc(&w.data, (size_t)L.NT * L.unit_bytes);
}
void free_packed(PackedWeight& w) {
  if (w.data) cudaFree(w.data);
  w.data = nullptr;
}

constexpr int PREFILL_ROWS = 1024;                 // rows of one causal prefill pass
constexpr int MAX_FORECAST = 8, MAX_DRAFT_WIDTH = 32;

struct GraphKey {
  int kind, n, T, prefix_chunk, n_prefix_chunks, own_chunk, n_own_chunks, flags, suffix_bound, pad_;
  const void* p[12];
  bool operator==(const GraphKey& o) const { return std::memcmp(this, &o, sizeof(GraphKey)) == 0; }
};
struct GraphKeyHash {
  size_t operator()(const GraphKey& k) const {
    const unsigned char* b = reinterpret_cast<const unsigned char*>(&k);
    size_t h = 1469598103934665603ull;
    for (size_t i = 0; i < sizeof(GraphKey); ++i) { h ^= b[i]; h *= 1099511628211ull; }
    return h;
  }
};
struct GraphEntry { cudaGraphExec_t exec; int nodes; };

}  // namespace

struct mlora_weight {
  PackedWeight w;
  cudaStream_t stream;
  int device = 0;                  // the device the packed weights live on
  ChainPhase* phase = nullptr;     // dev: descriptor of this projection for the persistent kernel
  int sm_count = 0;
};

struct mlora_ctx {
  mlora_model_desc d;
  cudaStream_t stream = nullptr;
  int sm_count = 148;
  int L = 0, Nq = 0, Nkv = 0, Nqkv = 0, cap = 0, Mmax = 0;
  std::vector<PackedWeight> w_qkv, w_o, w_gateup, w_down;
  PackedWeight w_lm;
  std::vector<const __half*> rms_attn, rms_ffn;
  // KV caches
  __half *prefix_k = nullptr, *prefix_v = nullptr;   // [L][Hkv][max_prefix][hd]
  __half *own_k = nullptr, *own_v = nullptr;         // [L][n][Hkv][cap][hd]
  size_t prefix_layer_stride = 0, prefix_head_stride = 0;
  size_t own_layer_stride = 0, own_stream_stride = 0, own_head_stride = 0;
  // scratch
  float *X = nullptr, *qkv = nullptr, *logits = nullptr, *T = nullptr, *partial = nullptr, *att_ws = nullptr;
  __half *h = nullptr, *attn16 = nullptr, *act16 = nullptr;
  size_t partial_floats = 0, att_ws_floats = 0;
  unsigned* counters = nullptr;
  unsigned long long* anc = nullptr;
  int32_t *depth = nullptr, *argmax = nullptr, *suffix_len = nullptr, *zero_len = nullptr, *chain_parent = nullptr,
          *root_parent = nullptr;
  int* status = nullptr;
  float2* cs_table = nullptr;
  // adapters
  const __half** tabA = nullptr;
  const __half** tabB = nullptr;
  float* ad_scale = nullptr;
  const __half** stageA = nullptr;   // pinned host staging [max_adapters][L*7]
  const __half** stageB = nullptr;
  float* stage_scale = nullptr;
  // host state
  int P = 0;
  bool prefilled = false;
  int suffix_bound = 0;
  int32_t* snap = nullptr;           // pinned copy of suffix_len
  cudaEvent_t snap_event = nullptr;
  bool snap_pending = false;
  int snap_inc = 0;
  int dbg_skip_compact = 0, dbg_no_graph = 0, dbg_no_chain = 0, dbg_no_tc = 0, dbg_inject_stall = 0;
  int step_mode = 0;                 // decode steps: 0 = the library's choice, 1 = per-layer kernels, 2 = the single-kernel step
  int32_t* host_io = nullptr;        // dev [3][max_streams]: adapter_idx, tokens, next of the host-buffer step
  const __half* forecast = nullptr;  // caller-owned dev fp16 [n_forecast][d_model] (DS2D forecast embeddings)
  int n_forecast = 0;
  int32_t* draft_cand = nullptr;     // dev [max_streams][MAX_FORECAST][MAX_DRAFT_WIDTH]: candidates of a drafting round
  int32_t* gen_tokens = nullptr;     // dev [k][n]: the tokens of a host-buffer generation (grown on demand)
  size_t gen_capacity = 0;
  // persistent projection chain (rows <= 8)
  ChainPhase* phases = nullptr;      // dev [4*L (+1)]: qkv, o, gate/up, down per layer; then lm_head
  int n_phases = 0;
  unsigned long long* chain_sync = nullptr;   // dev [4]
  int chain_stages = 0, chain_kmax = 0;
  // whole decode step in one kernel (one row per stream, rows <= 8)
  std::vector<StepPhase> step_phases_host;
  size_t step_acc_bytes = 0;         // step_tacc and step_ssq, contiguous
  bool lean_ok = false;              // the per-projection decode kernels take this model's shapes
  const __half** step_rowA = nullptr;   // dev [8][L*7]: the rows' adapter matrices, looked up once per call (lean path)
  const __half** step_rowB = nullptr;
  float* step_rowscale = nullptr;    // dev [8]
  StepPhase* step_phases = nullptr;  // dev [5*L + 3]: embed; qkv, attention, o, gate/up, down per layer; lm_head; end
  int n_step_phases = 0, step_stages = 0, step_own_tiles = 0;
  unsigned char *tmapA = nullptr, *tmapB = nullptr;           // dev [max_adapters][L*7] tensor maps over the adapters' matrices
  unsigned char *stage_tmA = nullptr, *stage_tmB = nullptr;   // pinned host staging of the same
  __half *xg_attn = nullptr, *xg_ffn = nullptr;     // residual rows times the gain of the next RMSNorm, fp16 [8][d_model]
  unsigned long long *step_tacc = nullptr, *step_ssq = nullptr, *step_amax = nullptr;
  long long* step_trace = nullptr;   // dev [2][n_step_phases][8]
  int dbg_trace = 0;
  int n_tacc = 0, n_ssq = 0;
  // graphs
  std::unordered_map<GraphKey, GraphEntry, GraphKeyHash> graphs;
  bool capturing = false;
  // profiling
  bool profiling = false;
  struct Ev { cudaEvent_t a, b; int fam, count; bool open; };   // one interval per run of consecutive launches of a family
  std::vector<Ev> evs;
  std::vector<cudaEvent_t> ev_pool;
  int64_t launches = 0;
  int captured_nodes = 0;
};

namespace {

int fail(int code, const std::string& msg) {
  g_last_error = msg;
  return code;
}
#define CK(call)                                                                                   \
  do {                                                                                             \
    cudaError_t e__ = (call);                                                                      \
    if (e__ != cudaSuccess)                                                                        \
      return fail(MLORA_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__));            \
  } while (0)

// ends the open profiling interval, if any
void prof_close(mlora_ctx* c) {
  if (!c->evs.empty() && c->evs.back().open) {
    cudaEventRecord(c->evs.back().b, c->stream);
    c->evs.back().open = false;
  }
}

// wraps one kernel launch: counts it and, when profiling, keeps it inside an event pair.  Consecutive launches of one
// family share a pair, so that what they overlap among themselves (programmatic launches) stays overlapped.
template <class F>
cudaError_t run(mlora_ctx* c, int fam, F&& f) {
  if (c->capturing) c->captured_nodes++;
  else c->launches++;
  if (!c->profiling) return f();
  if (c->evs.empty() || !c->evs.back().open || c->evs.back().fam != fam) {
    prof_close(c);
    mlora_ctx::Ev ev;
    for (cudaEvent_t* e : {&ev.a, &ev.b}) {
      if (!c->ev_pool.empty()) { *e = c->ev_pool.back(); c->ev_pool.pop_back(); }
      else { cudaError_t r = cudaEventCreate(e); if (r != cudaSuccess) return r; }
    }
    ev.fam = fam; ev.count = 0; ev.open = true;
    cudaEventRecord(ev.a, c->stream);
    c->evs.push_back(ev);
  }
  c->evs.back().count++;
  return f();
}

struct PassIO {
  int n = 0, T = 1;
  const int32_t* tokens = nullptr;
  const __half* hidden_in = nullptr;
  const int32_t* adapter_idx = nullptr;   // nullptr: base weights for every row
  const int32_t* parent = nullptr;        // dev [n][T]
  bool prefill = false;
  int pos_base = 0;                        // length of the shared segment the rows attend to
  const int32_t* suffix_len = nullptr;
  int suffix_bound = 0;
  float* logits = nullptr;                 // [M][vocab] destination, nullptr: skip lm_head
  int32_t* fused_next = nullptr;           // decode passes that want no logits: greedy tokens straight from the lm_head,
                                           // suffix lengths advanced (set by forward when its path did both)
  bool fused_done = false;
  bool last_row_logits = false;            // prefill: only the pass's last row goes through the final norm and lm_head
                                           // (io.logits receives that one row)
  bool rows_resolved = false;              // the rows' adapter pointers were looked up earlier in this call (same adapter_idx)
  AttnArgs plan;                           // chunking, filled by plan_pass
};

LoraArgs lora_args(mlora_ctx* c, const PassIO& io, int l, int nseg, const int* projs, const int* widths) {
  LoraArgs la{};
  int mask = 0;
  for (int i = 0; i < nseg; ++i) mask |= (1 << projs[i]);
  if (io.adapter_idx == nullptr || !(c->d.lora_targets & mask) || c->d.lora_rank <= 0) return la;
  la.adapter_idx = io.adapter_idx;
  la.rows_per_stream = io.T;
  la.tabA = c->tabA;
  la.tabB = c->tabB;
  la.scale = c->ad_scale;
  la.tab_stride = c->L * 7;
  la.n_slots = c->d.max_adapters;
  la.rank = c->d.lora_rank;
  la.nseg = nseg;
  for (int i = 0; i < nseg; ++i) { la.seg[i].proj_index = l * 7 + projs[i]; la.seg[i].n = widths[i]; }
  la.T = c->T;
  return la;
}

void plan_pass(mlora_ctx* c, PassIO& io) {
  AttnArgs& a = io.plan;
  a = AttnArgs{};
  a.P = io.pos_base;
  a.n = io.n; a.T = io.T; a.Hq = c->d.n_q_heads; a.Hkv = c->d.n_kv_heads; a.hd = c->d.head_dim;
  a.suffix_bound = (io.suffix_bound + 63) / 64 * 64;   // coarse, so the launch shape changes rarely
  attn_plan(a, c->sm_count);
}

// where a pass writes the K/V of its rows
void kv_destination(mlora_ctx* c, const PassIO& io, int l, __half*& kd, __half*& vd, size_t& sstride, size_t& hstride) {
  const int hd = c->d.head_dim;
  if (io.prefill) {
    kd = c->prefix_k + (size_t)l * c->prefix_layer_stride + (size_t)io.pos_base * hd;
    vd = c->prefix_v + (size_t)l * c->prefix_layer_stride + (size_t)io.pos_base * hd;
    sstride = 0; hstride = c->prefix_head_stride;
  } else {
    kd = c->own_k + (size_t)l * c->own_layer_stride;
    vd = c->own_v + (size_t)l * c->own_layer_stride;
    sstride = c->own_stream_stride; hstride = c->own_head_stride;
  }
}

int launch_attention_block(mlora_ctx* c, const PassIO& io, int l) {
  cudaStream_t st = c->stream;
  __half *kd, *vd;
  size_t sstride, hstride;
  kv_destination(c, io, l, kd, vd, sstride, hstride);
  AttnArgs a = io.plan;
  // q and the new k rows are rotated on load, the new K/V rows appended by the attention kernel itself
  a.qkv_f32 = c->qkv; a.cs_table = c->cs_table; a.pos_base = io.pos_base; a.depth = c->depth;
  a.prefix_k = c->prefix_k + (size_t)l * c->prefix_layer_stride;
  a.prefix_v = c->prefix_v + (size_t)l * c->prefix_layer_stride;
  a.prefix_head_stride = c->prefix_head_stride;
  a.own_k = kd; a.own_v = vd; a.own_stream_stride = sstride; a.own_head_stride = hstride;
  a.suffix_len = io.suffix_len; a.anc = c->anc; a.causal = io.prefill ? 1 : 0;
  a.out = c->attn16; a.status = c->status;
  if (attn_workspace_floats(a) > c->att_ws_floats) return fail(MLORA_ERR_CAPACITY, "attention scratch too small");
  a.part_o = c->att_ws;
  a.part_ml = c->att_ws + (attn_workspace_floats(a) / (a.hd + 2)) * a.hd;
  CK(run(c, MLORA_PROF_ATTN, [&] { return launch_attention(a, st); }));
  if (!attn_single_pass(a)) CK(run(c, MLORA_PROF_ATTN_MERGE, [&] { return launch_attention_merge(a, st); }));
  return MLORA_OK;
}

bool chain_eligible(const mlora_ctx* c, const PassIO& io) {
  return c->chain_stages > 0 && !c->dbg_no_chain && !io.prefill && io.n * io.T <= CHAIN_MAX_ROWS;
}

// a decode step (one row per stream) that the single-kernel path can take
bool step_eligible(const mlora_ctx* c, int n, int T) {
  // (the library's own choice is the per-layer path: at the 1B / 8-stream shapes it is the faster of the two)
  return c->step_stages > 0 && !c->dbg_no_chain && c->step_mode == 2 && T == 1 && n <= CHAIN_MAX_ROWS;
}

// one decode step as one persistent kernel: embedding to greedy token (or hidden state), suffix lengths advanced
int forward_step(mlora_ctx* c, int n, const int32_t* adapter_idx, const int32_t* tokens, const __half* hidden,
                 int32_t* out_next, float* out_logits, float* hidden_out) {
  const mlora_model_desc& d = c->d;
  StepArgs a{};
  a.phases = c->step_phases; a.n_phases = c->n_step_phases; a.M = n; a.eps = d.rms_eps;
  a.tokens = tokens; a.embed = (const __half*)d.embed; a.vocab = d.vocab; a.hidden_in = hidden;
  if (adapter_idx != nullptr && d.lora_rank > 0 && d.max_adapters > 0 && d.lora_targets != 0) {
    a.adapter_idx = adapter_idx; a.tabA = c->tabA; a.tabB = c->tabB; a.scale = c->ad_scale;
    a.tab_stride = c->L * 7; a.n_slots = d.max_adapters;
    a.tmapA = c->tmapA; a.tmapB = c->tmapB;
  }
  a.rank = (d.max_adapters > 0 && d.lora_targets != 0) ? d.lora_rank : 0;
  a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.hd = d.head_dim; a.P = c->P;
  a.qkv = c->qkv;
  a.prefix_k = c->prefix_k; a.prefix_v = c->prefix_v;
  a.prefix_layer_stride = c->prefix_layer_stride; a.prefix_head_stride = c->prefix_head_stride;
  a.own_k = c->own_k; a.own_v = c->own_v;
  a.own_layer_stride = c->own_layer_stride; a.own_stream_stride = c->own_stream_stride; a.own_head_stride = c->own_head_stride;
  a.suffix_len = c->suffix_len; a.cs_table = c->cs_table;
  a.logits = out_logits; a.out_next = out_next; a.hidden_out = hidden_out; a.amax = c->step_amax;
  a.tacc = c->step_tacc; a.ssq = c->step_ssq; a.n_tacc = c->n_tacc; a.n_ssq = c->n_ssq;
  a.sync = c->chain_sync; a.status = c->status;
  if (c->dbg_inject_stall) {                           // one pass only: short waits, one barrier that cannot complete
    a.wait_cycles = 200000000ll;                       // ~0.1 s
    a.inject_stall = 1;
    c->dbg_inject_stall = 0;
  }
  a.nstages = c->step_stages; a.own_tiles = c->step_own_tiles;
  a.trace = c->dbg_trace ? c->step_trace : nullptr;
  CK(run(c, MLORA_PROF_GEMM, [&] { return launch_step(a, c->sm_count, c->stream); }));
  return MLORA_OK;
}

// decode-sized pass: the projections of a layer run as one persistent kernel between the attention blocks
int forward_chain(mlora_ctx* c, const PassIO& io) {
  const mlora_model_desc& d = c->d;
  cudaStream_t st = c->stream;
  const int M = io.n * io.T;
  CK(run(c, MLORA_PROF_MISC, [&] { return launch_embed(io.tokens, (const __half*)d.embed, io.hidden_in, c->X, M, d.d_model, d.vocab, c->status, st, c->forecast, c->n_forecast); }));
  CK(run(c, MLORA_PROF_MISC, [&] { return launch_tree_prep(io.parent, io.n, io.T, c->anc, c->depth, c->status, st); }));
  ChainArgs a{};
  a.phases = c->phases;
  a.M = M; a.eps = d.rms_eps; a.logits = io.logits;
  if (io.adapter_idx != nullptr && d.lora_rank > 0 && d.max_adapters > 0 && d.lora_targets != 0) {
    a.adapter_idx = io.adapter_idx; a.rows_per_stream = io.T;
    a.tabA = c->tabA; a.tabB = c->tabB; a.scale = c->ad_scale;
    a.tab_stride = c->L * 7; a.n_slots = d.max_adapters;
  }
  a.rank = d.lora_rank;
  a.T = c->T; a.sync = c->chain_sync; a.status = c->status;
  a.nstages = c->chain_stages; a.kmax = c->chain_kmax;
  if (c->dbg_inject_stall) {                           // one pass only: short waits, one barrier that cannot complete
    a.wait_cycles = 200000000ll;                       // ~0.1 s
    a.inject_stall = 1;
    c->dbg_inject_stall = 0;
  }
  const int last = 4 * c->L + ((d.vocab > 0 && io.logits != nullptr) ? 1 : 0);
  // the K/V that the attention of layer l reads: prefetched into L2 by the chain launch before it
  auto kv_prefetch = [&](int l) {
    for (int i = 0; i < 4; ++i) a.pf[i] = ChainPrefetch{};
    if (l >= c->L) return;
    const unsigned hd2 = (unsigned)d.head_dim * 2u;
    if (io.pos_base > 0) {
      a.pf[0] = ChainPrefetch{(const unsigned char*)(c->prefix_k + (size_t)l * c->prefix_layer_stride), (unsigned)d.n_kv_heads,
                              (unsigned)(c->prefix_head_stride * 2), (unsigned)io.pos_base * hd2};
      a.pf[1] = a.pf[0];
      a.pf[1].base = (const unsigned char*)(c->prefix_v + (size_t)l * c->prefix_layer_stride);
    }
    // (the same coarse bound on the suffix lengths as the attention's launch shape, so frozen graphs stay valid)
    const size_t own_rows = std::min<size_t>((size_t)(io.suffix_bound + 63) / 64 * 64, c->own_head_stride / (size_t)d.head_dim);
    if (own_rows > 0 && c->own_stream_stride == c->own_head_stride * (size_t)d.n_kv_heads) {
      a.pf[2] = ChainPrefetch{(const unsigned char*)(c->own_k + (size_t)l * c->own_layer_stride), (unsigned)(io.n * d.n_kv_heads),
                              (unsigned)(c->own_head_stride * 2), (unsigned)own_rows * hd2};
      a.pf[3] = a.pf[2];
      a.pf[3].base = (const unsigned char*)(c->own_v + (size_t)l * c->own_layer_stride);
    }
  };
  a.p0 = 0; a.p1 = 1;
  kv_prefetch(0);
  CK(run(c, MLORA_PROF_GEMM, [&] { return launch_chain(a, c->sm_count, st); }));
  for (int l = 0; l < c->L; ++l) {
    int rc = launch_attention_block(c, io, l);
    if (rc != MLORA_OK) return rc;
    a.p0 = 4 * l + 1;
    a.p1 = (l + 1 < c->L) ? 4 * l + 5 : last;
    kv_prefetch(l + 1);
    CK(run(c, MLORA_PROF_GEMM, [&] { return launch_chain(a, c->sm_count, st); }));
  }
  return MLORA_OK;
}

// one projection of a pass with more than 8 rows: tensor-core path from 32 rows up, split-K mma.sync below
cudaError_t launch_projection(mlora_ctx* c, const GemmArgs& g, cudaStream_t st) {
  if (!c->dbg_no_tc && gemm_tc_eligible(g)) return launch_gemm_tc(g, c->sm_count, c->status, st);
  return launch_gemm(g, st);
}

// the launch sequence of one pass over M = n*T rows (Sec. 3.1 decoder, Eq. 1-4 projections)
// decode-sized pass as one small kernel per projection group (decode_lean.cu), attention between them
bool lean_eligible(const mlora_ctx* c, const PassIO& io) {
  // (the library's own choice where it applies: the fastest of the three decode paths at the measured shapes)
  return (c->step_mode == 3 || c->step_mode == 0) && !c->dbg_no_chain && c->lean_ok && c->step_phases != nullptr && !io.prefill && io.T == 1 &&
         io.n <= CHAIN_MAX_ROWS && io.parent == c->root_parent && attn_single_pass(io.plan);
}

int forward_lean(mlora_ctx* c, PassIO& io) {
  const mlora_model_desc& d = c->d;
  cudaStream_t st = c->stream;
  CK(cudaMemsetAsync(c->step_tacc, 0, c->step_acc_bytes, st));   // the step's accumulators (a memset node, not a kernel)
  LeanArgs a{};
  a.M = io.n; a.eps = d.rms_eps;
  const bool lora = io.adapter_idx != nullptr && d.lora_rank > 0 && d.max_adapters > 0 && d.lora_targets != 0;
  if (lora) {
    // the rows' adapter matrices by row: one small kernel per call, ordinary launch (everything behind it sees the table)
    if (!io.rows_resolved)
      CK(run(c, MLORA_PROF_MISC, [&] {
        return launch_lean_rowptr(io.adapter_idx, c->tabA, c->tabB, c->ad_scale, d.max_adapters, c->L * 7, io.n, c->step_rowA,
                                  c->step_rowB, c->step_rowscale, st);
      }));
    a.adapter_idx = io.adapter_idx; a.rows_direct = 1;
    a.tabA = c->step_rowA; a.tabB = c->step_rowB; a.scale = c->step_rowscale;
    a.tab_stride = c->L * 7; a.n_slots = CHAIN_MAX_ROWS;
  }
  a.rank = (d.max_adapters > 0 && d.lora_targets != 0) ? d.lora_rank : 0;
  a.rank_log2 = lean_rank_log2(a.rank);
  a.X = c->X; a.logits = io.logits; a.tacc = c->step_tacc; a.ssq = c->step_ssq;
  const bool fused = io.fused_next != nullptr && d.vocab > 0;
  if (fused) { a.logits = nullptr; a.amax = c->step_ssq + (size_t)c->n_ssq * CHAIN_MAX_ROWS; }
  const bool trace = c->dbg_trace && c->step_trace != nullptr;
  if (trace) CK(cudaMemsetAsync(c->step_trace, 0, (size_t)c->n_step_phases * 2 * 12 * sizeof(long long), st));
  for (size_t p = 0; p < c->step_phases_host.size(); ++p) {
    const StepPhase& ph = c->step_phases_host[p];
    if (trace) {                                       // this launch's rows of the timeline: first CTA, last CTA
      a.trace0 = c->step_trace + p * 12;
      a.trace1 = c->step_trace + ((size_t)c->n_step_phases + p) * 12;
    }
    if (ph.kind == SK_EMBED) {
      CK(run(c, MLORA_PROF_MISC, [&] {
        return launch_lean_embed(a, ph, io.tokens, (const __half*)d.embed, d.vocab, io.hidden_in, c->status, st);
      }));
    } else if (ph.kind == SK_GEMM) {
      if (ph.epi == EPI_F32 && ph.out_f32 == nullptr && io.logits == nullptr && !fused) continue;   // lm_head not wanted
      CK(run(c, MLORA_PROF_GEMM, [&] { return launch_lean_gemm(a, ph, st); }));
    } else if (ph.kind == SK_ATTN) {
      const int l = ph.layer;
      AttnArgs at = io.plan;
      at.qkv_f32 = c->qkv; at.cs_table = c->cs_table; at.pos_base = io.pos_base; at.depth = nullptr;   // one row per stream: depth 0, nothing to read
      at.prefix_k = c->prefix_k + (size_t)l * c->prefix_layer_stride;
      at.prefix_v = c->prefix_v + (size_t)l * c->prefix_layer_stride;
      at.prefix_head_stride = c->prefix_head_stride;
      at.own_k = c->own_k + (size_t)l * c->own_layer_stride; at.own_v = c->own_v + (size_t)l * c->own_layer_stride;
      at.own_stream_stride = c->own_stream_stride; at.own_head_stride = c->own_head_stride;
      at.suffix_len = io.suffix_len; at.anc = c->anc; at.causal = 0; at.out = c->attn16; at.status = c->status;
      at.pdl = 1;
      at.trace0 = trace ? c->step_trace + p * 12 : nullptr;
      if (lora && ph.next_nseg > 0) {
        at.o_tacc = c->step_tacc + (size_t)ph.t_out * CHAIN_MAX_ROWS * 3 * a.rank;
        at.o_tabA = c->step_rowA; at.o_adapter_idx = io.adapter_idx; at.o_direct = 1; at.o_proj_index = ph.next_proj[0]; at.o_rank = a.rank;
        at.o_tab_stride = c->L * 7; at.o_n_slots = CHAIN_MAX_ROWS;
      }
      CK(run(c, MLORA_PROF_ATTN, [&] { return launch_attention(at, st); }));
    }
  }
  if (fused) {
    CK(run(c, MLORA_PROF_MISC, [&] { return launch_lean_finish(a.amax, io.fused_next, c->suffix_len, io.n, st); }));
    io.fused_done = true;
  }
  return MLORA_OK;
}

int forward(mlora_ctx* c, PassIO& io) {
  if (lean_eligible(c, io)) return forward_lean(c, io);
  if (chain_eligible(c, io)) return forward_chain(c, io);
  const mlora_model_desc& d = c->d;
  cudaStream_t st = c->stream;
  const int M = io.n * io.T;
  const int dm = d.d_model, F = d.d_ffn;
  CK(run(c, MLORA_PROF_MISC, [&] { return launch_embed(io.tokens, (const __half*)d.embed, io.hidden_in, c->X, M, dm, d.vocab, c->status, st, c->forecast, c->n_forecast); }));
  CK(run(c, MLORA_PROF_MISC, [&] { return launch_tree_prep(io.parent, io.n, io.T, c->anc, c->depth, c->status, st); }));
  for (int l = 0; l < c->L; ++l) {
    // attention block
    {
      const int projs[3] = {0, 1, 2}, widths[3] = {c->Nq, c->Nkv, c->Nkv};
      ShrinkArgs s{};
      s.x_f32 = c->X; s.gain = c->rms_attn[l]; s.eps = d.rms_eps; s.h_out = c->h; s.M = M; s.K = dm;
      s.lora = lora_args(c, io, l, 3, projs, widths);
      CK(run(c, MLORA_PROF_SHRINK, [&] { return launch_shrink(s, st); }));
      GemmArgs g{};
      const PackedWeight& w = c->w_qkv[l];
      g.w = w.data; g.K = w.K; g.N = w.N; g.G = w.G; g.h = c->h; g.M = M;
      g.mode = MODE_QKV; g.epi = EPI_F32; g.seg_n0 = c->Nq; g.seg_n1 = c->Nkv;
      g.out_f32 = c->qkv; g.ldo = c->Nqkv;
      g.partial = c->partial; g.partial_capacity = c->partial_floats; g.counters = c->counters;
      g.lora = s.lora;
      CK(run(c, MLORA_PROF_GEMM, [&] { return launch_projection(c, g, st); }));
    }
    {
      int rc = launch_attention_block(c, io, l);
      if (rc != MLORA_OK) return rc;
    }
    {
      const int projs[1] = {3}, widths[1] = {dm};
      LoraArgs la = lora_args(c, io, l, 1, projs, widths);
      if (la.adapter_idx) {
        ShrinkArgs s{};
        s.h_in = c->attn16; s.M = M; s.K = c->Nq; s.lora = la;
        CK(run(c, MLORA_PROF_SHRINK, [&] { return launch_shrink(s, st); }));
      }
      GemmArgs g{};
      const PackedWeight& w = c->w_o[l];
      g.w = w.data; g.K = w.K; g.N = w.N; g.G = w.G; g.h = c->attn16; g.M = M;
      g.mode = MODE_PLAIN; g.epi = EPI_RESID; g.resid = c->X;
      g.partial = c->partial; g.partial_capacity = c->partial_floats; g.counters = c->counters;
      g.lora = la;
      CK(run(c, MLORA_PROF_GEMM, [&] { return launch_projection(c, g, st); }));
    }
    // MLP block
    {
      const int projs[2] = {4, 5}, widths[2] = {F, F};
      ShrinkArgs s{};
      s.x_f32 = c->X; s.gain = c->rms_ffn[l]; s.eps = d.rms_eps; s.h_out = c->h; s.M = M; s.K = dm;
      s.lora = lora_args(c, io, l, 2, projs, widths);
      CK(run(c, MLORA_PROF_SHRINK, [&] { return launch_shrink(s, st); }));
      GemmArgs g{};
      const PackedWeight& w = c->w_gateup[l];
      g.w = w.data; g.K = w.K; g.N = w.N; g.G = w.G; g.h = c->h; g.M = M;
      g.mode = MODE_GATEUP; g.epi = EPI_SWIGLU; g.out_f16 = c->act16;
      g.partial = c->partial; g.partial_capacity = c->partial_floats; g.counters = c->counters;
      g.lora = s.lora;
      CK(run(c, MLORA_PROF_GEMM, [&] { return launch_projection(c, g, st); }));
    }
    {
      const int projs[1] = {6}, widths[1] = {dm};
      LoraArgs la = lora_args(c, io, l, 1, projs, widths);
      if (la.adapter_idx) {
        ShrinkArgs s{};
        s.h_in = c->act16; s.M = M; s.K = F; s.lora = la;
        CK(run(c, MLORA_PROF_SHRINK, [&] { return launch_shrink(s, st); }));
      }
      GemmArgs g{};
      const PackedWeight& w = c->w_down[l];
      g.w = w.data; g.K = w.K; g.N = w.N; g.G = w.G; g.h = c->act16; g.M = M;
      g.mode = MODE_PLAIN; g.epi = EPI_RESID; g.resid = c->X;
      g.partial = c->partial; g.partial_capacity = c->partial_floats; g.counters = c->counters;
      g.lora = la;
      CK(run(c, MLORA_PROF_GEMM, [&] { return launch_projection(c, g, st); }));
    }
  }
  if (d.vocab > 0 && io.logits != nullptr) {
    const int Ml = io.last_row_logits ? 1 : M;           // rows that get logits: the last Ml of the pass
    ShrinkArgs s{};
    s.x_f32 = c->X + (size_t)(M - Ml) * dm; s.gain = (const __half*)d.rms_final; s.eps = d.rms_eps; s.h_out = c->h; s.M = Ml; s.K = dm;
    CK(run(c, MLORA_PROF_SHRINK, [&] { return launch_shrink(s, st); }));
    GemmArgs g{};
    const PackedWeight& w = c->w_lm;
    g.w = w.data; g.K = w.K; g.N = w.N; g.G = w.G; g.h = c->h; g.M = Ml;
    g.mode = MODE_PLAIN; g.epi = EPI_F32; g.out_f32 = io.logits; g.ldo = d.vocab;
    g.partial = c->partial; g.partial_capacity = c->partial_floats; g.counters = c->counters;
    CK(run(c, MLORA_PROF_GEMM, [&] { return launch_projection(c, g, st); }));
  }
  return MLORA_OK;
}

// runs `body` directly, or captures it once into a CUDA graph and replays it
template <class F>
int replay_or_run(mlora_ctx* c, const GraphKey& key, F&& body) {
  // the legacy default stream cannot be captured: launch directly there
  if (c->dbg_no_graph || c->profiling || c->stream == nullptr) return body();
  auto it = c->graphs.find(key);
  if (it == c->graphs.end()) {
    cudaGraph_t graph = nullptr;
    c->capturing = true;
    c->captured_nodes = 0;
    cudaError_t e = cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal);
    if (e != cudaSuccess) { c->capturing = false; return fail(MLORA_ERR_CUDA, std::string("begin capture: ") + cudaGetErrorString(e)); }
    int rc = body();
    e = cudaStreamEndCapture(c->stream, &graph);
    c->capturing = false;
    if (rc != MLORA_OK) { if (graph) cudaGraphDestroy(graph); return rc; }
    if (e != cudaSuccess) return fail(MLORA_ERR_CUDA, std::string("end capture: ") + cudaGetErrorString(e));
    GraphEntry ent{};
    e = cudaGraphInstantiate(&ent.exec, graph, 0);
    cudaGraphDestroy(graph);
    if (e != cudaSuccess) return fail(MLORA_ERR_CUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
    ent.nodes = c->captured_nodes;
    if (c->graphs.size() > 256) {                      // bound the cache
      for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
      c->graphs.clear();
    }
    it = c->graphs.emplace(key, ent).first;
  }
  CK(cudaGraphLaunch(it->second.exec, c->stream));
  c->launches += it->second.nodes;
  return MLORA_OK;
}

// refreshes the host's upper bound on the suffix lengths from the last finished snapshot
void poll_snapshot(mlora_ctx* c) {
  if (c->snap_pending && cudaEventQuery(c->snap_event) == cudaSuccess) {
    int mx = 0;
    for (int s = 0; s < c->d.max_streams; ++s) mx = c->snap[s] > mx ? c->snap[s] : mx;
    c->suffix_bound = mx + c->snap_inc;
    c->snap_pending = false;
  }
}
int ensure_capacity(mlora_ctx* c, int T) {
  poll_snapshot(c);
  if (c->suffix_bound + T <= c->cap) return MLORA_OK;
  // the bound is pessimistic after verify rounds: read the true lengths once
  CK(cudaStreamSynchronize(c->stream));
  CK(cudaMemcpy(c->snap, c->suffix_len, sizeof(int32_t) * c->d.max_streams, cudaMemcpyDeviceToHost));
  int mx = 0;
  for (int s = 0; s < c->d.max_streams; ++s) mx = c->snap[s] > mx ? c->snap[s] : mx;
  c->suffix_bound = mx;
  c->snap_pending = false;
  if (mx + T > c->cap) return fail(MLORA_ERR_CAPACITY, "own KV segment full");
  return MLORA_OK;
}

int init_kernels() {
  // the opt-in shared-memory sizes are per device: once for every device a context or weight is created on
  static bool done_on[64] = {};
  static std::mutex mu;
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(MLORA_ERR_UNSUPPORTED, "device ordinal out of range");
  std::lock_guard<std::mutex> lock(mu);
  bool& done = done_on[dev];
  if (done) return MLORA_OK;
  CK(init_gemm());
  CK(init_shrink());
  CK(init_attention());
  CK(init_lean());
  CK(init_chain());
  CK(init_step());
  CK(init_gemm_tc());
  done = true;
  return MLORA_OK;
}

int check_ctx(mlora_ctx* c) { return c ? MLORA_OK : fail(MLORA_ERR_ARG, "null context"); }

int prefill_impl(mlora_ctx* c, const int32_t* ids, const __half* hidden, int n, float* out_last) {
  if (n <= 0) return fail(MLORA_ERR_ARG, "prefill needs at least one position");
  if (n > c->d.max_prefix) return fail(MLORA_ERR_CAPACITY, "prompt longer than max_prefix");
  // a chunk of the prompt is one causal pass of up to PREFILL_ROWS rows (row blocks of 256 in the tensor-core GEMMs: the
  // weights are unpacked once per pass and slab, whatever the number of row blocks)
  const int chunk = c->Mmax >= PREFILL_ROWS ? PREFILL_ROWS : c->Mmax / 64 * 64;
  const int dm = c->d.d_model;
  for (int p0 = 0; p0 < n; p0 += chunk) {
    PassIO io;
    io.n = 1;
    io.T = (n - p0 < chunk) ? (n - p0) : chunk;
    io.tokens = ids ? ids + p0 : nullptr;
    io.hidden_in = hidden ? hidden + (size_t)p0 * dm : nullptr;
    io.parent = nullptr;                    // causal: the attention kernel compares row indices
    io.prefill = true;
    io.pos_base = p0;
    io.suffix_len = c->zero_len;
    io.suffix_bound = 0;
    const bool last = (p0 + io.T >= n);
    io.logits = (last && c->d.vocab > 0 && out_last) ? c->logits : nullptr;
    io.last_row_logits = true;
    plan_pass(c, io);
    int rc = forward(c, io);
    if (rc != MLORA_OK) return rc;
    if (last && out_last) {
      const float* src = c->d.vocab > 0 ? c->logits : c->X + (size_t)(io.T - 1) * dm;
      const size_t cnt = c->d.vocab > 0 ? (size_t)c->d.vocab : (size_t)dm;
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_copy_rows_f32(src, out_last, cnt, c->stream); }));
    }
  }
  CK(cudaMemsetAsync(c->suffix_len, 0, sizeof(int32_t) * c->d.max_streams, c->stream));
  c->P = n;
  c->prefilled = true;
  c->suffix_bound = 0;
  c->snap_pending = false;
  return MLORA_OK;
}

int step_common_checks(mlora_ctx* c, int n_streams, const void* adapter_idx, int T) {
  if (!c->prefilled) return fail(MLORA_ERR_STATE, "no shared prefill yet");
  if (n_streams <= 0 || n_streams > c->d.max_streams) return fail(MLORA_ERR_ARG, "n_streams out of range");
  if (adapter_idx == nullptr) return fail(MLORA_ERR_ARG, "adapter_idx is null");
  if (T < 1 || T > c->d.max_tree) return fail(MLORA_ERR_CAPACITY, "tree larger than max_tree");
  return ensure_capacity(c, T);
}

}  // namespace

// ============================================================================= C ABI
extern "C" {

const char* mlora_last_error(mlora_ctx*) { return g_last_error.c_str(); }

int mlora_create(const mlora_model_desc* desc, mlora_ctx** out) {
  if (!desc || !out) return fail(MLORA_ERR_ARG, "null argument");
  const mlora_model_desc& d = *desc;
  if (d.n_layers <= 0 || d.d_model <= 0 || d.n_q_heads <= 0 || d.n_kv_heads <= 0 || d.d_ffn <= 0 || d.vocab < 0)
    return fail(MLORA_ERR_ARG, "non-positive model dimension");
  if (!d.qweight || !d.scales || !d.rms_attn || !d.rms_ffn) return fail(MLORA_ERR_ARG, "null weight table");
  if (d.vocab > 0 && (!d.embed || !d.rms_final)) return fail(MLORA_ERR_ARG, "vocab > 0 needs embed and rms_final");
  if (d.head_dim != 64 && d.head_dim != 128) return fail(MLORA_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (d.rope_style != 0) return fail(MLORA_ERR_UNSUPPORTED, "rope_style must be 0 (half-split pairs)");
  if (d.n_q_heads % d.n_kv_heads) return fail(MLORA_ERR_ARG, "n_q_heads must be a multiple of n_kv_heads");
  if (!wlayout_group_ok(d.group_size))
    return fail(MLORA_ERR_UNSUPPORTED, "group_size must be 64, 128, 256 or a multiple of 512");
  const int Nq = d.n_q_heads * d.head_dim, Nkv = d.n_kv_heads * d.head_dim;
  for (int K : {d.d_model, Nq, d.d_ffn})
    if (K % 64 || K % d.group_size) return fail(MLORA_ERR_UNSUPPORTED, "every input width must be a multiple of 64 and of group_size");
  for (int N : {d.d_model, Nq, Nkv, d.d_ffn, d.vocab})
    if (N % 16) return fail(MLORA_ERR_UNSUPPORTED, "every output width must be a multiple of 16");
  if (d.max_tree < 1 || d.max_tree > 64) return fail(MLORA_ERR_ARG, "max_tree must be in 1..64");
  if (d.max_streams < 1 || d.max_prefix < 1 || d.max_suffix < 1 || d.max_adapters < 0 || d.lora_rank < 0)
    return fail(MLORA_ERR_ARG, "bad capacity");

  if (init_kernels() != MLORA_OK) return MLORA_ERR_CUDA;
  mlora_ctx* c = new mlora_ctx();
  c->d = d;
  c->stream = (cudaStream_t)d.cuda_stream;
  c->L = d.n_layers; c->Nq = Nq; c->Nkv = Nkv; c->Nqkv = Nq + 2 * Nkv;
  c->cap = d.max_suffix + d.max_tree;
  c->Mmax = d.max_streams * d.max_tree;
  if (c->Mmax < PREFILL_ROWS) c->Mmax = PREFILL_ROWS;        // prefill passes have up to this many rows
#define CKC(call)                                                                                  \
  do {                                                                                             \
    cudaError_t e__ = (call);                                                                      \
    if (e__ != cudaSuccess) {                                                                      \
      fail(MLORA_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__));                   \
      mlora_destroy(c);                                                                            \
      return MLORA_ERR_CUDA;                                                                       \
    }                                                                                              \
  } while (0)
  int dev = 0;
  CKC(cudaGetDevice(&dev));
  CKC(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
  cudaStream_t st = c->stream;
  const int L = c->L, dm = d.d_model, F = d.d_ffn, G = d.group_size, hd = d.head_dim;
  // ---- weights: repack into fused fragment-major matrices
  c->w_qkv.resize(L); c->w_o.resize(L); c->w_gateup.resize(L); c->w_down.resize(L);
  c->rms_attn.resize(L); c->rms_ffn.resize(L);
  for (int l = 0; l < L; ++l) {
    const void* const* qw = d.qweight + (size_t)l * 7;
    const void* const* sc = d.scales + (size_t)l * 7;
    for (int p = 0; p < 7; ++p)
      if (!qw[p] || !sc[p]) { fail(MLORA_ERR_ARG, "null weight pointer"); mlora_destroy(c); return MLORA_ERR_ARG; }
    if (!d.rms_attn[l] || !d.rms_ffn[l]) { fail(MLORA_ERR_ARG, "null norm gain"); mlora_destroy(c); return MLORA_ERR_ARG; }
    c->rms_attn[l] = (const __half*)d.rms_attn[l];
    c->rms_ffn[l] = (const __half*)d.rms_ffn[l];
    PackedWeight& wqkv = c->w_qkv[l];
    CKC(alloc_packed(wqkv, dm, c->Nqkv, G));
    CKC(launch_repack((const uint8_t*)qw[0], (const __half*)sc[0], dm, Nq, G, wqkv.data, 0, 1, st));
    CKC(launch_repack((const uint8_t*)qw[1], (const __half*)sc[1], dm, Nkv, G, wqkv.data, Nq / 16, 1, st));
    CKC(launch_repack((const uint8_t*)qw[2], (const __half*)sc[2], dm, Nkv, G, wqkv.data, (Nq + Nkv) / 16, 1, st));
    CKC(alloc_packed(c->w_o[l], Nq, dm, G));
    CKC(launch_repack((const uint8_t*)qw[3], (const __half*)sc[3], Nq, dm, G, c->w_o[l].data, 0, 1, st));
    PackedWeight& wgu = c->w_gateup[l];
    CKC(alloc_packed(wgu, dm, 2 * F, G));
    CKC(launch_repack((const uint8_t*)qw[4], (const __half*)sc[4], dm, F, G, wgu.data, 0, 2, st));
    CKC(launch_repack((const uint8_t*)qw[5], (const __half*)sc[5], dm, F, G, wgu.data, 1, 2, st));
    CKC(alloc_packed(c->w_down[l], F, dm, G));
    CKC(launch_repack((const uint8_t*)qw[6], (const __half*)sc[6], F, dm, G, c->w_down[l].data, 0, 1, st));
  }
  if (d.vocab > 0) {
    const void* qw = d.qweight[(size_t)L * 7];
    const void* sc = d.scales[(size_t)L * 7];
    if (!qw || !sc) { fail(MLORA_ERR_ARG, "null lm_head pointer"); mlora_destroy(c); return MLORA_ERR_ARG; }
    CKC(alloc_packed(c->w_lm, dm, d.vocab, G));
    CKC(launch_repack((const uint8_t*)qw, (const __half*)sc, dm, d.vocab, G, c->w_lm.data, 0, 1, st));
  }
  // ---- KV caches
  c->prefix_head_stride = (size_t)d.max_prefix * hd;
  c->prefix_layer_stride = c->prefix_head_stride * d.n_kv_heads;
  c->own_head_stride = (size_t)c->cap * hd;
  c->own_stream_stride = c->own_head_stride * d.n_kv_heads;
  c->own_layer_stride = c->own_stream_stride * d.max_streams;
  CKC(cudaMalloc(&c->prefix_k, c->prefix_layer_stride * L * sizeof(__half)));
  CKC(cudaMalloc(&c->prefix_v, c->prefix_layer_stride * L * sizeof(__half)));
  CKC(cudaMalloc(&c->own_k, c->own_layer_stride * L * sizeof(__half)));
  CKC(cudaMalloc(&c->own_v, c->own_layer_stride * L * sizeof(__half)));
  // ---- scratch
  const size_t Mm = c->Mmax;
  size_t maxK = dm; if ((size_t)F > maxK) maxK = F; if ((size_t)Nq > maxK) maxK = Nq;
  CKC(cudaMalloc(&c->X, Mm * dm * sizeof(float)));
  CKC(cudaMalloc(&c->qkv, Mm * c->Nqkv * sizeof(float)));
  CKC(cudaMalloc(&c->h, Mm * maxK * sizeof(__half)));
  CKC(cudaMalloc(&c->attn16, Mm * Nq * sizeof(__half)));
  CKC(cudaMalloc(&c->act16, Mm * F * sizeof(__half)));
  if (d.vocab > 0) CKC(cudaMalloc(&c->logits, (size_t)d.max_streams * d.max_tree * d.vocab * sizeof(float)));   // (prefill: one row)
  CKC(cudaMalloc(&c->T, Mm * 3 * (d.lora_rank > 0 ? d.lora_rank : 1) * sizeof(float)));
  c->partial_floats = (size_t)16 << 20;               // 64 MB of split-K scratch
  CKC(cudaMalloc(&c->partial, c->partial_floats * sizeof(float)));
  CKC(cudaMalloc(&c->counters, 4096 * sizeof(unsigned)));
  CKC(cudaMemsetAsync(c->counters, 0, 4096 * sizeof(unsigned), st));
  {
    // attention scratch: rows x chunks never exceeds (rows of one launch) + 64 x (CTAs the planner aims for),
    // once for the shared-prefix chunks and once for the own-segment chunks
    const size_t g_heads = d.n_q_heads / d.n_kv_heads;
    const size_t R_all = Mm * g_heads;
    c->att_ws_floats = ((size_t)d.n_kv_heads * R_all * 2 + (size_t)256 * c->sm_count + 4096) * (hd + 2);
    CKC(cudaMalloc(&c->att_ws, c->att_ws_floats * sizeof(float)));
  }
  CKC(cudaMalloc(&c->host_io, 3 * (size_t)d.max_streams * sizeof(int32_t)));
  CKC(cudaMalloc(&c->draft_cand, (size_t)d.max_streams * MAX_FORECAST * MAX_DRAFT_WIDTH * sizeof(int32_t)));
  CKC(cudaMalloc(&c->anc, Mm * sizeof(unsigned long long)));
  CKC(cudaMalloc(&c->depth, Mm * sizeof(int32_t)));
  CKC(cudaMalloc(&c->argmax, Mm * sizeof(int32_t)));
  CKC(cudaMalloc(&c->suffix_len, d.max_streams * sizeof(int32_t)));
  CKC(cudaMalloc(&c->zero_len, d.max_streams * sizeof(int32_t)));
  CKC(cudaMemsetAsync(c->suffix_len, 0, d.max_streams * sizeof(int32_t), st));
  CKC(cudaMemsetAsync(c->zero_len, 0, d.max_streams * sizeof(int32_t), st));
  CKC(cudaMalloc(&c->status, sizeof(int)));
  CKC(cudaMemsetAsync(c->status, 0, sizeof(int), st));
  {
    std::vector<int32_t> chain(64), root(d.max_streams, -1);
    for (int i = 0; i < 64; ++i) chain[i] = i - 1;
    CKC(cudaMalloc(&c->chain_parent, 64 * sizeof(int32_t)));
    CKC(cudaMalloc(&c->root_parent, d.max_streams * sizeof(int32_t)));
    CKC(cudaMemcpyAsync(c->chain_parent, chain.data(), 64 * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CKC(cudaMemcpyAsync(c->root_parent, root.data(), d.max_streams * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    CKC(cudaStreamSynchronize(st));
  }
  {
    // cos/sin of pos * theta^(-2i/hd), evaluated in double
    const int maxpos = d.max_prefix + c->cap + 1;
    const int half = hd / 2;
    std::vector<float2> tab((size_t)maxpos * half);
    for (int i = 0; i < half; ++i) {
      const double inv = std::pow((double)d.rope_theta, -2.0 * i / hd);
      for (int p = 0; p < maxpos; ++p) {
        const double ang = (double)p * inv;
        tab[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
      }
    }
    CKC(cudaMalloc(&c->cs_table, tab.size() * sizeof(float2)));
    CKC(cudaMemcpyAsync(c->cs_table, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, st));
    CKC(cudaStreamSynchronize(st));
  }
  // ---- adapter tables
  if (d.max_adapters > 0) {
    const size_t ents = (size_t)d.max_adapters * L * 7;
    CKC(cudaMalloc(&c->tabA, ents * sizeof(void*)));
    CKC(cudaMalloc(&c->tabB, ents * sizeof(void*)));
    CKC(cudaMalloc(&c->ad_scale, d.max_adapters * sizeof(float)));
    CKC(cudaMemsetAsync(c->tabA, 0, ents * sizeof(void*), st));
    CKC(cudaMemsetAsync(c->tabB, 0, ents * sizeof(void*), st));
    CKC(cudaMemsetAsync(c->ad_scale, 0, d.max_adapters * sizeof(float), st));
    CKC(cudaMallocHost(&c->stageA, ents * sizeof(void*)));
    CKC(cudaMallocHost(&c->stageB, ents * sizeof(void*)));
    CKC(cudaMallocHost(&c->stage_scale, d.max_adapters * sizeof(float)));
    CKC(cudaMalloc(&c->tmapA, ents * STEP_TMAP_BYTES));
    CKC(cudaMalloc(&c->tmapB, ents * STEP_TMAP_BYTES));
    CKC(cudaMemsetAsync(c->tmapA, 0, ents * STEP_TMAP_BYTES, st));
    CKC(cudaMemsetAsync(c->tmapB, 0, ents * STEP_TMAP_BYTES, st));
    CKC(cudaMallocHost(&c->stage_tmA, ents * STEP_TMAP_BYTES));
    CKC(cudaMallocHost(&c->stage_tmB, ents * STEP_TMAP_BYTES));
  }
  // ---- phase descriptors of the persistent projection chain
  {
    size_t kmax = dm; if ((size_t)F > kmax) kmax = F; if ((size_t)Nq > kmax) kmax = Nq;
    c->chain_kmax = (int)kmax;
    c->chain_stages = chain_pick_stages(c->chain_kmax, d.lora_rank);
    std::vector<ChainPhase> ph;
    const int tg = d.lora_rank > 0 && d.max_adapters > 0 ? d.lora_targets : 0;
    for (int l = 0; l < L; ++l) {
      ChainPhase q{};
      q.w = c->w_qkv[l].data; q.K = dm; q.N = c->Nqkv; q.G = G; q.mode = MODE_QKV; q.epi = EPI_F32; q.in_kind = IN_NORM;
      q.seg_n0 = Nq; q.seg_n1 = Nkv; q.x_f32 = c->X; q.gain = c->rms_attn[l]; q.out_f32 = c->qkv; q.ldo = c->Nqkv;
      if (tg & (MLORA_Q | MLORA_K | MLORA_V)) {
        q.lora_nseg = 3;
        for (int i = 0; i < 3; ++i) q.lora_proj[i] = l * 7 + i;
        q.lora_n[0] = Nq; q.lora_n[1] = Nkv; q.lora_n[2] = Nkv;
      }
      ph.push_back(q);
      ChainPhase o{};
      o.w = c->w_o[l].data; o.K = Nq; o.N = dm; o.G = G; o.mode = MODE_PLAIN; o.epi = EPI_RESID; o.in_kind = IN_F16;
      o.h_in = c->attn16; o.resid = c->X;
      if (tg & MLORA_O) { o.lora_nseg = 1; o.lora_proj[0] = l * 7 + 3; o.lora_n[0] = dm; }
      ph.push_back(o);
      ChainPhase gu{};
      gu.w = c->w_gateup[l].data; gu.K = dm; gu.N = 2 * F; gu.G = G; gu.mode = MODE_GATEUP; gu.epi = EPI_SWIGLU;
      gu.in_kind = IN_NORM; gu.x_f32 = c->X; gu.gain = c->rms_ffn[l]; gu.out_f16 = c->act16;
      if (tg & (MLORA_GATE | MLORA_UP)) {
        gu.lora_nseg = 2; gu.lora_proj[0] = l * 7 + 4; gu.lora_proj[1] = l * 7 + 5; gu.lora_n[0] = F; gu.lora_n[1] = F;
      }
      ph.push_back(gu);
      ChainPhase dn{};
      dn.w = c->w_down[l].data; dn.K = F; dn.N = dm; dn.G = G; dn.mode = MODE_PLAIN; dn.epi = EPI_RESID; dn.in_kind = IN_F16;
      dn.h_in = c->act16; dn.resid = c->X;
      if (tg & MLORA_DOWN) { dn.lora_nseg = 1; dn.lora_proj[0] = l * 7 + 6; dn.lora_n[0] = dm; }
      ph.push_back(dn);
    }
    if (d.vocab > 0) {
      ChainPhase lm{};
      lm.w = c->w_lm.data; lm.K = dm; lm.N = d.vocab; lm.G = G; lm.mode = MODE_PLAIN; lm.epi = EPI_F32; lm.in_kind = IN_NORM;
      lm.x_f32 = c->X; lm.gain = (const __half*)d.rms_final; lm.out_f32 = nullptr; lm.ldo = d.vocab;
      ph.push_back(lm);
    }
    for (const ChainPhase& q : ph)
      if (c->chain_stages > 0 && !chain_phase_fits(q.K, q.mode, q.lora_nseg, d.lora_rank, c->chain_stages, c->sm_count))
        c->chain_stages = 0;
    c->n_phases = (int)ph.size();
    CKC(cudaMalloc(&c->phases, ph.size() * sizeof(ChainPhase)));
    CKC(cudaMemcpy(c->phases, ph.data(), ph.size() * sizeof(ChainPhase), cudaMemcpyHostToDevice));
    CKC(cudaMalloc(&c->chain_sync, 4 * sizeof(unsigned long long)));
    CKC(cudaMemsetAsync(c->chain_sync, 0, 4 * sizeof(unsigned long long), st));
  }
  // ---- phase descriptors and scratch of the single-kernel decode step
  {
    const int tg = d.lora_rank > 0 && d.max_adapters > 0 ? d.lora_targets : 0;
    c->step_stages = step_plan(dm, F, Nq, Nkv, hd, d.lora_rank, tg, c->sm_count, &c->step_own_tiles);
    c->lean_ok = lean_shapes_ok(dm, F, Nq, Nkv, tg ? d.lora_rank : 0) &&
                 attn_decode_o_slice_fits(hd, d.n_q_heads / d.n_kv_heads, (tg & MLORA_O) ? d.lora_rank : 0);
    if (d.max_streams > 0 && (c->step_stages > 0 || c->lean_ok)) {
      const int rr = tg ? d.lora_rank : 0;
      c->n_tacc = 4 * L; c->n_ssq = 2 * L + 1;
      CKC(cudaMalloc(&c->xg_attn, (size_t)CHAIN_MAX_ROWS * dm * sizeof(__half)));
      CKC(cudaMalloc(&c->xg_ffn, (size_t)CHAIN_MAX_ROWS * dm * sizeof(__half)));
      const size_t tacc_bytes = (size_t)c->n_tacc * CHAIN_MAX_ROWS * 3 * (rr > 0 ? rr : 1) * sizeof(unsigned long long);
      // (one allocation for both kinds of accumulators: one memset clears a step's worth)
      const size_t ssq_bytes = (size_t)c->n_ssq * CHAIN_MAX_ROWS * sizeof(unsigned long long);
      const size_t amax_bytes = CHAIN_MAX_ROWS * sizeof(unsigned long long);   // row maxima of the lm_head (lean path)
      CKC(cudaMalloc(&c->step_tacc, tacc_bytes + ssq_bytes + amax_bytes));
      CKC(cudaMemsetAsync(c->step_tacc, 0, tacc_bytes + ssq_bytes + amax_bytes, st));
      c->step_ssq = c->step_tacc + tacc_bytes / sizeof(unsigned long long);
      c->step_acc_bytes = tacc_bytes + ssq_bytes + amax_bytes;
      CKC(cudaMalloc(&c->step_rowA, (size_t)CHAIN_MAX_ROWS * L * 7 * sizeof(__half*)));
      CKC(cudaMalloc(&c->step_rowB, (size_t)CHAIN_MAX_ROWS * L * 7 * sizeof(__half*)));
      CKC(cudaMalloc(&c->step_rowscale, CHAIN_MAX_ROWS * sizeof(float)));
      CKC(cudaMalloc(&c->step_amax, (size_t)c->sm_count * CHAIN_MAX_ROWS * sizeof(unsigned long long)));
      CKC(cudaMemsetAsync(c->step_amax, 0, (size_t)c->sm_count * CHAIN_MAX_ROWS * sizeof(unsigned long long), st));
      std::vector<StepPhase> sp;
      auto next_qkv = [&](StepPhase& q, int l) {          // the consuming group is q,k,v of layer l
        if (tg & (MLORA_Q | MLORA_K | MLORA_V)) {
          q.next_nseg = 3;
          for (int i = 0; i < 3; ++i) q.next_proj[i] = l * 7 + i;
          q.next_ld = dm; q.t_out = 4 * l;
        }
      };
      StepPhase e{};
      e.kind = SK_EMBED; e.N = dm; e.out16 = c->xg_attn; e.gain_next = c->rms_attn[0]; e.ssq_out = 0; e.norm_in = -1;
      next_qkv(e, 0);
      sp.push_back(e);
      for (int l = 0; l < L; ++l) {
        StepPhase q{};
        q.kind = SK_GEMM; q.layer = l; q.w = c->w_qkv[l].data; q.K = dm; q.N = c->Nqkv; q.G = G; q.mode = MODE_QKV; q.epi = EPI_F32;
        q.seg_n0 = Nq; q.seg_n1 = Nkv; q.in16 = c->xg_attn; q.norm_in = 2 * l; q.out_f32 = c->qkv; q.ldo = c->Nqkv; q.ssq_out = -1;
        if (tg & (MLORA_Q | MLORA_K | MLORA_V)) {
          q.lora_nseg = 3;
          for (int i = 0; i < 3; ++i) q.lora_proj[i] = l * 7 + i;
          q.lora_n[0] = Nq; q.lora_n[1] = Nkv; q.lora_n[2] = Nkv; q.t_in = 4 * l;
        }
        sp.push_back(q);
        StepPhase at{};
        at.kind = SK_ATTN; at.layer = l; at.out16 = c->attn16; at.norm_in = -1; at.ssq_out = -1;
        if (tg & MLORA_O) { at.next_nseg = 1; at.next_proj[0] = l * 7 + 3; at.next_ld = Nq; at.t_out = 4 * l + 1; }
        sp.push_back(at);
        StepPhase o{};
        o.kind = SK_GEMM; o.layer = l; o.w = c->w_o[l].data; o.K = Nq; o.N = dm; o.G = G; o.mode = MODE_PLAIN; o.epi = EPI_RESID;
        o.in16 = c->attn16; o.norm_in = -1; o.out16 = c->xg_ffn; o.gain_next = c->rms_ffn[l]; o.ssq_out = 2 * l + 1;
        if (tg & MLORA_O) { o.lora_nseg = 1; o.lora_proj[0] = l * 7 + 3; o.lora_n[0] = dm; o.t_in = 4 * l + 1; }
        if (tg & (MLORA_GATE | MLORA_UP)) {
          o.next_nseg = 2; o.next_proj[0] = l * 7 + 4; o.next_proj[1] = l * 7 + 5; o.next_ld = dm; o.t_out = 4 * l + 2;
        }
        sp.push_back(o);
        StepPhase gu{};
        gu.kind = SK_GEMM; gu.layer = l; gu.w = c->w_gateup[l].data; gu.K = dm; gu.N = 2 * F; gu.G = G; gu.mode = MODE_GATEUP;
        gu.epi = EPI_SWIGLU; gu.in16 = c->xg_ffn; gu.norm_in = 2 * l + 1; gu.out16 = c->act16; gu.ssq_out = -1;
        if (tg & (MLORA_GATE | MLORA_UP)) {
          gu.lora_nseg = 2; gu.lora_proj[0] = l * 7 + 4; gu.lora_proj[1] = l * 7 + 5; gu.lora_n[0] = F; gu.lora_n[1] = F;
          gu.t_in = 4 * l + 2;
        }
        if (tg & MLORA_DOWN) { gu.next_nseg = 1; gu.next_proj[0] = l * 7 + 6; gu.next_ld = F; gu.t_out = 4 * l + 3; }
        sp.push_back(gu);
        StepPhase dn{};
        dn.kind = SK_GEMM; dn.layer = l; dn.w = c->w_down[l].data; dn.K = F; dn.N = dm; dn.G = G; dn.mode = MODE_PLAIN;
        dn.epi = EPI_RESID; dn.in16 = c->act16; dn.norm_in = -1; dn.ssq_out = -1;
        if (tg & MLORA_DOWN) { dn.lora_nseg = 1; dn.lora_proj[0] = l * 7 + 6; dn.lora_n[0] = dm; dn.t_in = 4 * l + 3; }
        if (l + 1 < L) {
          dn.out16 = c->xg_attn; dn.gain_next = c->rms_attn[l + 1]; dn.ssq_out = 2 * (l + 1);
          next_qkv(dn, l + 1);
        } else if (d.vocab > 0) {
          dn.out16 = c->xg_attn; dn.gain_next = (const __half*)d.rms_final; dn.ssq_out = 2 * L;
        } else {
          dn.last = 1;
        }
        sp.push_back(dn);
      }
      if (d.vocab > 0) {
        StepPhase lm{};
        lm.kind = SK_GEMM; lm.layer = L; lm.w = c->w_lm.data; lm.K = dm; lm.N = d.vocab; lm.G = G; lm.mode = MODE_PLAIN;
        lm.epi = EPI_F32; lm.in16 = c->xg_attn; lm.norm_in = 2 * L; lm.out_f32 = nullptr; lm.ldo = d.vocab; lm.ssq_out = -1;
        sp.push_back(lm);
      }
      StepPhase fin{};
      fin.kind = SK_FIN; fin.norm_in = -1; fin.ssq_out = -1;
      sp.push_back(fin);
      // each projection phase names the weights of the next one (the step after the lm_head starts with layer 0 again):
      // its CTAs ask for them in L2 while they run (kernel-per-projection path)
      {
        std::vector<int> gi;
        for (size_t i = 0; i < sp.size(); ++i) if (sp[i].kind == SK_GEMM) gi.push_back((int)i);
        for (size_t k = 0; k < gi.size(); ++k) {
          const StepPhase& nx = sp[gi[(k + 1) % gi.size()]];
          const WLayout nl = make_wlayout(nx.K, nx.N, nx.G);
          const unsigned long long bytes = (unsigned long long)nl.NT * nl.unit_bytes;
          sp[gi[k]].pf_w = nx.w;
          sp[gi[k]].pf_bytes = bytes < LEAN_PF_MAX_BYTES ? bytes : LEAN_PF_MAX_BYTES;
        }
      }
      c->n_step_phases = (int)sp.size();
      CKC(cudaMalloc(&c->step_trace, sp.size() * 2 * 12 * sizeof(long long)));
      CKC(cudaMemsetAsync(c->step_trace, 0, sp.size() * 2 * 12 * sizeof(long long), st));
      CKC(cudaMalloc(&c->step_phases, sp.size() * sizeof(StepPhase)));
      CKC(cudaMemcpy(c->step_phases, sp.data(), sp.size() * sizeof(StepPhase), cudaMemcpyHostToDevice));
      c->step_phases_host = sp;
    }
  }
  CKC(cudaMallocHost(&c->snap, d.max_streams * sizeof(int32_t)));
  CKC(cudaEventCreateWithFlags(&c->snap_event, cudaEventDisableTiming));
  CKC(cudaStreamSynchronize(st));
#undef CKC
  *out = c;
  return MLORA_OK;
}

int mlora_destroy(mlora_ctx* c) {
  if (!c) return MLORA_OK;
  cudaStreamSynchronize(c->stream);
  for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
  for (auto& w : c->w_qkv) free_packed(w);
  for (auto& w : c->w_o) free_packed(w);
  for (auto& w : c->w_gateup) free_packed(w);
  for (auto& w : c->w_down) free_packed(w);
  free_packed(c->w_lm);
  void* dev_ptrs[] = {c->prefix_k, c->prefix_v, c->own_k, c->own_v, c->X, c->qkv, c->logits, c->T, c->partial, c->att_ws,
                      c->h, c->attn16, c->act16, c->counters, c->anc, c->depth, c->argmax, c->suffix_len,
                      c->zero_len, c->chain_parent, c->root_parent, c->status, c->cs_table, (void*)c->tabA,
                      (void*)c->tabB, c->ad_scale, c->phases, c->chain_sync, c->host_io, c->step_phases, c->xg_attn, c->xg_ffn,
                      c->step_tacc, c->step_amax, c->step_trace, c->tmapA, c->tmapB, c->gen_tokens, c->draft_cand,
                      (void*)c->step_rowA, (void*)c->step_rowB, c->step_rowscale};
  for (void* p : dev_ptrs) if (p) cudaFree(p);
  if (c->stageA) cudaFreeHost((void*)c->stageA);
  if (c->stageB) cudaFreeHost((void*)c->stageB);
  if (c->stage_scale) cudaFreeHost(c->stage_scale);
  if (c->stage_tmA) cudaFreeHost(c->stage_tmA);
  if (c->stage_tmB) cudaFreeHost(c->stage_tmB);
  if (c->snap) cudaFreeHost(c->snap);
  if (c->snap_event) cudaEventDestroy(c->snap_event);
  for (auto& e : c->evs) { cudaEventDestroy(e.a); cudaEventDestroy(e.b); }
  for (auto& e : c->ev_pool) cudaEventDestroy(e);
  delete c;
  return MLORA_OK;
}

int mlora_set_adapter(mlora_ctx* c, int32_t slot, const void* const* A, const void* const* B, float alpha) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (slot < 0 || slot >= c->d.max_adapters) return fail(MLORA_ERR_ARG, "adapter slot out of range");
  if ((A == nullptr) != (B == nullptr)) return fail(MLORA_ERR_ARG, "A and B must both be given or both be NULL");
  if (c->d.lora_rank <= 0) return fail(MLORA_ERR_STATE, "context was created with lora_rank 0");
  const size_t per = (size_t)c->L * 7;
  // the staging row of this slot may still be in flight from an earlier call on the same slot
  CK(cudaStreamSynchronize(c->stream));
  for (size_t i = 0; A != nullptr && i < per; ++i)
    if ((c->d.lora_targets & (1 << (int)(i % 7))) && (A[i] == nullptr || B[i] == nullptr))
      return fail(MLORA_ERR_ARG, "null adapter tensor for a targeted projection");
  for (size_t i = 0; A != nullptr && i < per; ++i)
    if ((c->d.lora_targets & (1 << (int)(i % 7))) && (((uintptr_t)A[i] | (uintptr_t)B[i]) & 15))
      return fail(MLORA_ERR_ARG, "adapter tensors must be 16-byte aligned");
  for (size_t i = 0; i < per; ++i) {
    const int p = (int)(i % 7);
    const bool on = A != nullptr && (c->d.lora_targets & (1 << p));
    c->stageA[slot * per + i] = on ? (const __half*)A[i] : nullptr;
    c->stageB[slot * per + i] = on ? (const __half*)B[i] : nullptr;
  }
  c->stage_scale[slot] = A ? alpha / (float)c->d.lora_rank : 0.f;
  // tensor maps over the caller's matrices for the single-kernel decode step (its producer warp copies 16-column
  // slices of them; nothing of the matrices themselves is copied or repacked here)
  if (c->step_stages > 0) {
    const mlora_model_desc& d = c->d;
    const int widthK[7] = {d.d_model, d.d_model, d.d_model, c->Nq, d.d_model, d.d_model, d.d_ffn};
    const int widthN[7] = {c->Nq, c->Nkv, c->Nkv, d.d_model, d.d_ffn, d.d_ffn, d.d_model};
    for (size_t i = 0; i < per; ++i) {
      const int p = (int)(i % 7);
      unsigned char* ma = c->stage_tmA + (slot * per + i) * STEP_TMAP_BYTES;
      unsigned char* mb = c->stage_tmB + (slot * per + i) * STEP_TMAP_BYTES;
      if (c->stageA[slot * per + i] != nullptr) {
        CK(step_encode_slice_map(c->stageA[slot * per + i], widthK[p], d.lora_rank, ma));
        CK(step_encode_slice_map(c->stageB[slot * per + i], widthN[p], d.lora_rank, mb));
      } else {
        std::memset(ma, 0, STEP_TMAP_BYTES);
        std::memset(mb, 0, STEP_TMAP_BYTES);
      }
    }
    CK(cudaMemcpyAsync(c->tmapA + slot * per * STEP_TMAP_BYTES, c->stage_tmA + slot * per * STEP_TMAP_BYTES, per * STEP_TMAP_BYTES,
                       cudaMemcpyHostToDevice, c->stream));
    CK(cudaMemcpyAsync(c->tmapB + slot * per * STEP_TMAP_BYTES, c->stage_tmB + slot * per * STEP_TMAP_BYTES, per * STEP_TMAP_BYTES,
                       cudaMemcpyHostToDevice, c->stream));
  }
  CK(cudaMemcpyAsync(c->tabA + slot * per, c->stageA + slot * per, per * sizeof(void*), cudaMemcpyHostToDevice, c->stream));
  CK(cudaMemcpyAsync(c->tabB + slot * per, c->stageB + slot * per, per * sizeof(void*), cudaMemcpyHostToDevice, c->stream));
  CK(cudaMemcpyAsync(c->ad_scale + slot, c->stage_scale + slot, sizeof(float), cudaMemcpyHostToDevice, c->stream));
  return MLORA_OK;
}

int mlora_prefill_shared(mlora_ctx* c, const int32_t* prompt_ids, int32_t n, float* out_last_logits) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary: use mlora_prefill_shared_h");
  if (!prompt_ids) return fail(MLORA_ERR_ARG, "prompt_ids is null");
  return prefill_impl(c, prompt_ids, nullptr, n, out_last_logits);
}

int mlora_prefill_shared_h(mlora_ctx* c, const void* hidden, int32_t n, float* out_last_hidden) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!hidden) return fail(MLORA_ERR_ARG, "hidden is null");
  return prefill_impl(c, nullptr, (const __half*)hidden, n, out_last_hidden);
}

static int decode_impl(mlora_ctx* c, int n, const int32_t* adapter_idx, const int32_t* tokens, const __half* hidden,
                       int32_t* out_next, float* out_logits, float* hidden_out) {
  int rc = step_common_checks(c, n, adapter_idx, 1);
  if (rc != MLORA_OK) return rc;
  if (step_eligible(c, n, 1)) {
    rc = forward_step(c, n, adapter_idx, tokens, hidden, out_next, out_logits, hidden_out);
    if (rc != MLORA_OK) return rc;
    c->suffix_bound += 1;
    if (c->snap_pending) c->snap_inc += 1;
    return MLORA_OK;
  }
  PassIO io;
  io.n = n; io.T = 1; io.tokens = tokens; io.hidden_in = hidden; io.adapter_idx = adapter_idx;
  io.parent = c->root_parent; io.pos_base = c->P; io.suffix_len = c->suffix_len; io.suffix_bound = c->suffix_bound;
  io.logits = c->d.vocab > 0 ? (out_logits ? out_logits : c->logits) : nullptr;
  if (c->d.vocab > 0 && out_logits == nullptr) io.fused_next = out_next;     // (taken up by the path that can)
  plan_pass(c, io);
  GraphKey key{};
  key.kind = hidden ? 2 : 1; key.n = n; key.T = 1;
  key.prefix_chunk = io.plan.prefix_chunk; key.n_prefix_chunks = io.plan.n_prefix_chunks;
  key.own_chunk = io.plan.own_chunk; key.n_own_chunks = io.plan.n_own_chunks;
  key.flags = ((c->P * 4 + c->dbg_inject_stall * 2 + c->dbg_no_chain) * 4 + c->step_mode) * 2 + c->dbg_trace;
  key.suffix_bound = io.plan.suffix_bound;     // (rounded up by plan_pass: the kernels' launch shape and prefetch extents)
  key.p[0] = adapter_idx; key.p[1] = tokens; key.p[2] = hidden; key.p[3] = out_next; key.p[4] = out_logits; key.p[5] = hidden_out;
  rc = replay_or_run(c, key, [&]() -> int {
    int r = forward(c, io);
    if (r != MLORA_OK) return r;
    if (io.fused_done) return MLORA_OK;               // tokens written, suffix lengths advanced
    if (c->d.vocab > 0) {
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_argmax(io.logits, n, c->d.vocab, out_next, c->stream); }));
    } else {
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_copy_rows_f32(c->X, hidden_out, (size_t)n * c->d.d_model, c->stream); }));
    }
    CK(run(c, MLORA_PROF_MISC, [&] { return launch_advance(c->suffix_len, nullptr, n, 1, c->stream); }));
    return MLORA_OK;
  });
  if (rc != MLORA_OK) return rc;
  c->suffix_bound += 1;
  if (c->snap_pending) c->snap_inc += 1;
  return MLORA_OK;
}

int mlora_decode_step(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, const int32_t* tokens,
                      int32_t* out_next, float* out_logits) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary: use mlora_decode_step_h");
  if (!tokens || !out_next) return fail(MLORA_ERR_ARG, "tokens/out_next is null");
  return decode_impl(c, n_streams, adapter_idx, tokens, nullptr, out_next, out_logits, nullptr);
}

int mlora_decode_step_host(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx_host, const int32_t* tokens_host,
                           int32_t* out_next_host) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary");
  if (!adapter_idx_host || !tokens_host || !out_next_host) return fail(MLORA_ERR_ARG, "null host buffer");
  if (n_streams <= 0 || n_streams > c->d.max_streams) return fail(MLORA_ERR_ARG, "n_streams out of range");
  int32_t* d_ad = c->host_io;
  int32_t* d_tok = c->host_io + c->d.max_streams;
  int32_t* d_next = c->host_io + 2 * (size_t)c->d.max_streams;
  const size_t bytes = (size_t)n_streams * sizeof(int32_t);
  CK(cudaMemcpyAsync(d_ad, adapter_idx_host, bytes, cudaMemcpyHostToDevice, c->stream));
  CK(cudaMemcpyAsync(d_tok, tokens_host, bytes, cudaMemcpyHostToDevice, c->stream));
  int rc = decode_impl(c, n_streams, d_ad, d_tok, nullptr, d_next, nullptr, nullptr);
  if (rc != MLORA_OK) return rc;
  CK(cudaMemcpyAsync(out_next_host, d_next, bytes, cudaMemcpyDeviceToHost, c->stream));
  CK(cudaStreamSynchronize(c->stream));
  return MLORA_OK;
}

int mlora_sample_first(mlora_ctx* c, const float* logits, int32_t n, int32_t* out_tokens) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary");
  if (!logits || !out_tokens) return fail(MLORA_ERR_ARG, "logits/out_tokens is null");
  if (n < 1 || n > c->d.vocab) return fail(MLORA_ERR_ARG, "n must be between 1 and the vocabulary size");
  CK(run(c, MLORA_PROF_MISC, [&] { return launch_topn(logits, c->d.vocab, n, out_tokens, c->stream); }));
  return MLORA_OK;
}

// k decode steps enqueued back to back (captured as ONE graph where the stream allows it): step j reads the tokens that
// step j - 1 wrote, on the device
static int generate_impl(mlora_ctx* c, int n, const int32_t* adapter_idx, const int32_t* first, int k, int32_t* out) {
  int rc = step_common_checks(c, n, adapter_idx, 1);
  if (rc != MLORA_OK) return rc;
  if (k > 1) { rc = ensure_capacity(c, k); if (rc != MLORA_OK) return rc; }
  const int bound0 = c->suffix_bound;
  GraphKey key{};
  key.kind = 4; key.n = n; key.T = k;
  key.flags = (c->P * 16 + c->step_mode * 4 + c->dbg_inject_stall * 2 + c->dbg_no_chain) * 2 + c->dbg_trace;
  key.suffix_bound = bound0;                           // every step's launch shapes follow from the bound at the start
  key.p[0] = adapter_idx; key.p[1] = first; key.p[2] = out;
  rc = replay_or_run(c, key, [&]() -> int {
    for (int j = 0; j < k; ++j) {
      const int32_t* tok = j ? out + (size_t)(j - 1) * n : first;
      int32_t* next = out + (size_t)j * n;
      if (step_eligible(c, n, 1)) {
        int r = forward_step(c, n, adapter_idx, tok, nullptr, next, nullptr, nullptr);
        if (r != MLORA_OK) return r;
        continue;
      }
      PassIO io;
      io.n = n; io.T = 1; io.tokens = tok; io.adapter_idx = adapter_idx;
      io.parent = c->root_parent; io.pos_base = c->P; io.suffix_len = c->suffix_len; io.suffix_bound = bound0 + j;
      io.logits = c->logits;
      io.fused_next = next;
      io.rows_resolved = j > 0;
      plan_pass(c, io);
      int r = forward(c, io);
      if (r != MLORA_OK) return r;
      if (io.fused_done) continue;
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_argmax(io.logits, n, c->d.vocab, next, c->stream); }));
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_advance(c->suffix_len, nullptr, n, 1, c->stream); }));
    }
    return MLORA_OK;
  });
  if (rc != MLORA_OK) return rc;
  c->suffix_bound += k;
  if (c->snap_pending) c->snap_inc += k;
  return MLORA_OK;
}

int mlora_generate(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, const int32_t* first_tokens, int32_t k_steps,
                   int32_t* out_tokens) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary");
  if (!first_tokens || !out_tokens) return fail(MLORA_ERR_ARG, "first_tokens/out_tokens is null");
  if (k_steps < 1) return fail(MLORA_ERR_ARG, "k_steps must be at least 1");
  return generate_impl(c, n_streams, adapter_idx, first_tokens, k_steps, out_tokens);
}

int mlora_generate_host(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx_host, const int32_t* first_tokens_host,
                        int32_t k_steps, int32_t* out_tokens_host) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "context has no vocabulary");
  if (!adapter_idx_host || !first_tokens_host || !out_tokens_host) return fail(MLORA_ERR_ARG, "null host buffer");
  if (n_streams <= 0 || n_streams > c->d.max_streams) return fail(MLORA_ERR_ARG, "n_streams out of range");
  if (k_steps < 1) return fail(MLORA_ERR_ARG, "k_steps must be at least 1");
  const size_t need = (size_t)k_steps * n_streams;
  if (need > c->gen_capacity) {                        // (grown outside any timed loop: the first call of a new size)
    CK(cudaStreamSynchronize(c->stream));
    if (c->gen_tokens) cudaFree(c->gen_tokens);
    c->gen_tokens = nullptr; c->gen_capacity = 0;
    CK(cudaMalloc(&c->gen_tokens, need * sizeof(int32_t)));
    c->gen_capacity = need;
  }
  int32_t* d_ad = c->host_io;
  int32_t* d_tok = c->host_io + c->d.max_streams;
  const size_t bytes = (size_t)n_streams * sizeof(int32_t);
  CK(cudaMemcpyAsync(d_ad, adapter_idx_host, bytes, cudaMemcpyHostToDevice, c->stream));
  CK(cudaMemcpyAsync(d_tok, first_tokens_host, bytes, cudaMemcpyHostToDevice, c->stream));
  int rc = generate_impl(c, n_streams, d_ad, d_tok, k_steps, c->gen_tokens);
  if (rc != MLORA_OK) return rc;
  CK(cudaMemcpyAsync(out_tokens_host, c->gen_tokens, need * sizeof(int32_t), cudaMemcpyDeviceToHost, c->stream));
  CK(cudaStreamSynchronize(c->stream));
  return MLORA_OK;
}

int mlora_decode_step_h(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, const void* hidden_in,
                        float* hidden_out) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!hidden_in || !hidden_out) return fail(MLORA_ERR_ARG, "hidden_in/hidden_out is null");
  if (c->d.vocab != 0) return fail(MLORA_ERR_STATE, "context has a vocabulary: use mlora_decode_step");
  return decode_impl(c, n_streams, adapter_idx, nullptr, (const __half*)hidden_in, nullptr, nullptr, hidden_out);
}

// what a drafting round adds to a verify pass (all device arrays; the templates are shared by the streams)
struct DraftIO {
  const int32_t *level, *rank, *forecast_of, *widths;
  int m, wmax;
  int32_t* out_tokens;
};

static int verify_impl(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, int32_t n_nodes,
                       const int32_t* tree_tokens, const int32_t* tree_parent, int32_t* out_accept_len,
                       int32_t* out_accept_idx, int32_t* out_next, float* out_logits, const DraftIO* draft) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "verification needs logits: context has no vocabulary");
  if (!tree_tokens || !tree_parent || !out_accept_len || !out_accept_idx || !out_next)
    return fail(MLORA_ERR_ARG, "null argument");
  int rc = step_common_checks(c, n_streams, adapter_idx, n_nodes);
  if (rc != MLORA_OK) return rc;
  const int n = n_streams, T = n_nodes;
  PassIO io;
  io.n = n; io.T = T; io.tokens = tree_tokens; io.adapter_idx = adapter_idx; io.parent = tree_parent;
  io.pos_base = c->P; io.suffix_len = c->suffix_len; io.suffix_bound = c->suffix_bound;
  io.logits = out_logits ? out_logits : c->logits;
  plan_pass(c, io);
  GraphKey key{};
  key.kind = draft ? 5 : 3; key.n = n; key.T = T;
  key.prefix_chunk = io.plan.prefix_chunk; key.n_prefix_chunks = io.plan.n_prefix_chunks;
  key.own_chunk = io.plan.own_chunk; key.n_own_chunks = io.plan.n_own_chunks;
  key.flags = c->P * 8 + c->dbg_no_tc * 4 + c->dbg_skip_compact * 2 + c->dbg_no_chain;
  key.suffix_bound = io.plan.suffix_bound;
  key.p[0] = adapter_idx; key.p[1] = tree_tokens; key.p[2] = tree_parent; key.p[3] = out_accept_len;
  key.p[4] = out_accept_idx; key.p[5] = out_next; key.p[6] = out_logits;
  if (draft) {
    key.p[7] = draft->level; key.p[8] = draft->rank; key.p[9] = draft->forecast_of; key.p[10] = draft->widths;
    key.p[11] = draft->out_tokens;
    key.flags += (draft->m * 64 + draft->wmax) * 65536;
  }
  key.pad_ = c->n_forecast;
  rc = replay_or_run(c, key, [&]() -> int {
    int r = forward(c, io);
    if (r != MLORA_OK) return r;
    cudaStream_t st = c->stream;
    CK(run(c, MLORA_PROF_MISC, [&] { return launch_argmax(io.logits, n * T, c->d.vocab, c->argmax, st); }));
    CK(run(c, MLORA_PROF_MISC, [&] { return launch_accept(tree_tokens, tree_parent, c->argmax, n, T, out_accept_len, out_accept_idx, out_next, st); }));
    if (!c->dbg_skip_compact) {
      CK(run(c, MLORA_PROF_MISC, [&] {
        return launch_compact(c->own_k, c->own_v, c->own_layer_stride, c->own_stream_stride, c->own_head_stride, c->L, n,
                              c->d.n_kv_heads, c->d.head_dim, c->suffix_len, out_accept_len, out_accept_idx, T, st);
      }));
      CK(run(c, MLORA_PROF_MISC, [&] { return launch_advance(c->suffix_len, out_accept_len, n, 0, st); }));
    }
    if (draft) {
      // the next tree, from the forecast rows of every stream's last accepted node (two launches)
      if (c->capturing) c->captured_nodes++;
      else c->launches++;
      CK(run(c, MLORA_PROF_MISC, [&] {
        return launch_draft(io.logits, c->d.vocab, n, T, draft->m, draft->wmax, draft->widths, draft->level, draft->rank,
                            draft->forecast_of, out_accept_len, out_accept_idx, out_next, c->draft_cand, draft->out_tokens,
                            c->status, st);
      }));
    }
    return MLORA_OK;
  });
  if (rc != MLORA_OK) return rc;
  if (!c->dbg_skip_compact) {
    c->suffix_bound += T;
    if (c->snap_pending) c->snap_inc += T;
    else if (!c->profiling) {
      // ask for the true lengths so that the pessimistic bound can be tightened a few rounds later
      CK(cudaMemcpyAsync(c->snap, c->suffix_len, sizeof(int32_t) * c->d.max_streams, cudaMemcpyDeviceToHost, c->stream));
      CK(cudaEventRecord(c->snap_event, c->stream));
      c->snap_pending = true;
      c->snap_inc = 0;
    }
  }
  return MLORA_OK;
}

int mlora_verify_tree(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, int32_t n_nodes,
                      const int32_t* tree_tokens, const int32_t* tree_parent, int32_t* out_accept_len,
                      int32_t* out_accept_idx, int32_t* out_next, float* out_logits) {
  return verify_impl(c, n_streams, adapter_idx, n_nodes, tree_tokens, tree_parent, out_accept_len, out_accept_idx, out_next,
                     out_logits, nullptr);
}

int mlora_set_forecast(mlora_ctx* c, const void* forecast, int32_t m) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (c->d.vocab == 0) return fail(MLORA_ERR_STATE, "forecast rows need a vocabulary");
  if (forecast == nullptr || m == 0) { c->forecast = nullptr; c->n_forecast = 0; return MLORA_OK; }
  if (m < 0 || m > MAX_FORECAST) return fail(MLORA_ERR_ARG, "between 1 and 8 forecast embeddings");
  if (reinterpret_cast<uintptr_t>(forecast) & 3) return fail(MLORA_ERR_ARG, "forecast must be 4-byte aligned");
  c->forecast = (const __half*)forecast;
  c->n_forecast = m;
  return MLORA_OK;
}

int mlora_ds2d_round(mlora_ctx* c, int32_t n_streams, const int32_t* adapter_idx, int32_t n_rows, const int32_t* tree_tokens,
                     const int32_t* tree_parent, const int32_t* row_level, const int32_t* row_rank,
                     const int32_t* forecast_of, const int32_t* widths, int32_t m, int32_t max_width,
                     int32_t* out_accept_len, int32_t* out_accept_idx, int32_t* out_next, int32_t* out_tree_tokens,
                     float* out_logits) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!row_level || !row_rank || !forecast_of || !widths || !out_tree_tokens) return fail(MLORA_ERR_ARG, "null argument");
  if (c->n_forecast == 0) return fail(MLORA_ERR_STATE, "no forecast embeddings: call mlora_set_forecast first");
  if (m < 1 || m > c->n_forecast) return fail(MLORA_ERR_ARG, "m exceeds the forecast embeddings set");
  if (max_width < 1 || max_width > MAX_DRAFT_WIDTH || max_width > c->d.vocab) return fail(MLORA_ERR_ARG, "max_width must be 1..32");
  if (out_tree_tokens == tree_tokens) return fail(MLORA_ERR_ARG, "out_tree_tokens must not alias tree_tokens");
  DraftIO dr{row_level, row_rank, forecast_of, widths, m, max_width, out_tree_tokens};
  return verify_impl(c, n_streams, adapter_idx, n_rows, tree_tokens, tree_parent, out_accept_len, out_accept_idx, out_next,
                     out_logits, &dr);
}

int mlora_reset_streams(mlora_ctx* c) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  CK(cudaMemsetAsync(c->suffix_len, 0, sizeof(int32_t) * c->d.max_streams, c->stream));
  c->suffix_bound = 0;
  c->snap_pending = false;
  return MLORA_OK;
}

int mlora_sync_status(mlora_ctx* c) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  CK(cudaStreamSynchronize(c->stream));
  int st = 0;
  CK(cudaMemcpy(&st, c->status, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0) {
    CK(cudaMemset(c->status, 0, sizeof(int)));
    unsigned long long where = 0;
    CK(cudaMemcpy(&where, c->chain_sync + 3, sizeof(where), cudaMemcpyDeviceToHost));
    // a wait that ran out leaves the barrier counters of the persistent kernel mid-count: start them afresh
    CK(cudaMemset(c->chain_sync, 0, 4 * sizeof(unsigned long long)));
    // ... and the step kernel's accumulators part-filled
    if (c->step_tacc) {
      const int rr = c->d.lora_rank > 0 && c->d.max_adapters > 0 && c->d.lora_targets ? c->d.lora_rank : 1;
      CK(cudaMemset(c->step_tacc, 0, (size_t)c->n_tacc * CHAIN_MAX_ROWS * 3 * rr * sizeof(unsigned long long)));
      CK(cudaMemset(c->step_ssq, 0, (size_t)c->n_ssq * CHAIN_MAX_ROWS * sizeof(unsigned long long)));
    }
    if (st == MLORA_ERR_TIMEOUT) {
      char buf[160];
      std::snprintf(buf, sizeof(buf), "device status: a bounded wait ran out (wait kind %d, phase %d, block %d, thread %d)",
                    (int)(where >> 48), (int)((where >> 32) & 0xffff), (int)((where >> 16) & 0xffff), (int)(where & 0xffff));
      return fail(st, buf);
    }
    return fail(st, "device status: malformed tree or token id out of range");
  }
  return MLORA_OK;
}

int mlora_export_kv(mlora_ctx* c, int32_t layer, int32_t stream, int32_t first, int32_t count, int32_t* suffix_len,
                    void* k_out, void* v_out) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (layer < 0 || layer >= c->L || stream < -1 || stream >= c->d.max_streams || first < 0 || count < 0)
    return fail(MLORA_ERR_ARG, "export_kv: index out of range");
  CK(cudaStreamSynchronize(c->stream));
  const int hd = c->d.head_dim, Hkv = c->d.n_kv_heads;
  const __half *ks, *vs;
  size_t head_stride;
  int limit;
  if (stream < 0) {
    ks = c->prefix_k + (size_t)layer * c->prefix_layer_stride;
    vs = c->prefix_v + (size_t)layer * c->prefix_layer_stride;
    head_stride = c->prefix_head_stride; limit = c->d.max_prefix;
    if (suffix_len) *suffix_len = c->P;
  } else {
    ks = c->own_k + (size_t)layer * c->own_layer_stride + (size_t)stream * c->own_stream_stride;
    vs = c->own_v + (size_t)layer * c->own_layer_stride + (size_t)stream * c->own_stream_stride;
    head_stride = c->own_head_stride; limit = c->cap;
    if (suffix_len) CK(cudaMemcpy(suffix_len, c->suffix_len + stream, sizeof(int32_t), cudaMemcpyDeviceToHost));
  }
  if (first + count > limit) return fail(MLORA_ERR_ARG, "export_kv: rows beyond the segment");
  if (count == 0) return MLORA_OK;
  if (!k_out || !v_out) return fail(MLORA_ERR_ARG, "export_kv: null output");
  for (int kh = 0; kh < Hkv; ++kh) {
    CK(cudaMemcpy2DAsync((__half*)k_out + (size_t)kh * hd, (size_t)Hkv * hd * 2, ks + kh * head_stride + (size_t)first * hd,
                         (size_t)hd * 2, (size_t)hd * 2, count, cudaMemcpyDeviceToDevice, c->stream));
    CK(cudaMemcpy2DAsync((__half*)v_out + (size_t)kh * hd, (size_t)Hkv * hd * 2, vs + kh * head_stride + (size_t)first * hd,
                         (size_t)hd * 2, (size_t)hd * 2, count, cudaMemcpyDeviceToDevice, c->stream));
  }
  CK(cudaStreamSynchronize(c->stream));
  return MLORA_OK;
}

int mlora_export_state(mlora_ctx* c, int32_t layer, int32_t stream, int32_t* suffix_len, void* k_out, void* v_out) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!suffix_len) return fail(MLORA_ERR_ARG, "export_state: suffix_len is null");
  if (stream < 0) return fail(MLORA_ERR_ARG, "export_state: stream out of range");
  int rc = mlora_export_kv(c, layer, stream, 0, 0, suffix_len, nullptr, nullptr);
  if (rc != MLORA_OK || *suffix_len == 0) return rc;
  return mlora_export_kv(c, layer, stream, 0, *suffix_len, suffix_len, k_out, v_out);
}

int mlora_debug_dequant(mlora_ctx* c, int32_t layer, int32_t proj, void* out_fp16) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!out_fp16) return fail(MLORA_ERR_ARG, "null output");
  const PackedWeight* w = nullptr;
  int N = 0, off = 0, stride = 1;
  const int F = c->d.d_ffn;
  if (layer == c->L && proj == 0 && c->d.vocab > 0) { w = &c->w_lm; N = c->d.vocab; }
  else if (layer >= 0 && layer < c->L && proj >= 0 && proj < 7) {
    switch (proj) {
      case 0: w = &c->w_qkv[layer]; N = c->Nq; break;
      case 1: w = &c->w_qkv[layer]; N = c->Nkv; off = c->Nq / 16; break;
      case 2: w = &c->w_qkv[layer]; N = c->Nkv; off = (c->Nq + c->Nkv) / 16; break;
      case 3: w = &c->w_o[layer]; N = c->d.d_model; break;
      case 4: w = &c->w_gateup[layer]; N = F; stride = 2; break;
      case 5: w = &c->w_gateup[layer]; N = F; off = 1; stride = 2; break;
      default: w = &c->w_down[layer]; N = c->d.d_model; break;
    }
  } else return fail(MLORA_ERR_ARG, "debug_dequant: no such projection");
  CK(launch_dequant(w->data, w->K, N, w->G, off, stride, (__half*)out_fp16, c->stream));
  c->launches++;
  return MLORA_OK;
}

int mlora_debug_set(mlora_ctx* c, int32_t key, int32_t value) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (key == 1) c->dbg_skip_compact = value ? 1 : 0;
  else if (key == 2) c->dbg_no_graph = value ? 1 : 0;
  else if (key == 3) c->dbg_no_chain = value ? 1 : 0;
  else if (key == 4) c->dbg_no_tc = value ? 1 : 0;
  else if (key == 5) c->dbg_inject_stall = value ? 1 : 0;
  else if (key == 6) {
    c->step_mode = (value >= 0 && value <= 3) ? value : 0;
    // the single-kernel step expects the step's accumulators zero when it starts (it clears them on its way out); the
    // kernel-per-projection path clears them when a step starts and leaves them used: clear them at every switch
    if (c->step_tacc != nullptr) CK(cudaMemsetAsync(c->step_tacc, 0, c->step_acc_bytes, c->stream));
    if (c->step_amax != nullptr) CK(cudaMemsetAsync(c->step_amax, 0, (size_t)c->sm_count * CHAIN_MAX_ROWS * sizeof(unsigned long long), c->stream));
  }
  else if (key == 7) c->dbg_trace = value ? 1 : 0;
  else return fail(MLORA_ERR_ARG, "unknown debug key");
  return MLORA_OK;
}

int mlora_profile_begin(mlora_ctx* c) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  CK(cudaStreamSynchronize(c->stream));
  c->profiling = true;
  return MLORA_OK;
}

int mlora_profile_end(mlora_ctx* c, float* ms, int32_t* launches) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  prof_close(c);
  CK(cudaStreamSynchronize(c->stream));
  c->profiling = false;
  for (int i = 0; i < MLORA_PROF_FAMILIES; ++i) { if (ms) ms[i] = 0.f; if (launches) launches[i] = 0; }
  for (auto& e : c->evs) {
    float t = 0.f;
    cudaEventElapsedTime(&t, e.a, e.b);
    if (ms) ms[e.fam] += t;
    if (launches) launches[e.fam] += e.count;
    c->ev_pool.push_back(e.a);
    c->ev_pool.push_back(e.b);
  }
  c->evs.clear();
  return MLORA_OK;
}

int64_t mlora_launch_count(mlora_ctx* c) { return c ? c->launches : 0; }

int mlora_step_timeline(mlora_ctx* c, int64_t* host_out, int32_t capacity, int32_t* n_phases) {
  if (check_ctx(c)) return MLORA_ERR_ARG;
  if (!n_phases) return fail(MLORA_ERR_ARG, "null argument");
  *n_phases = c->n_step_phases;
  if (c->step_trace == nullptr) return fail(MLORA_ERR_STATE, "this context has no single-kernel decode step");
  const size_t n = (size_t)c->n_step_phases * 2 * 12;
  if (!host_out || (size_t)capacity < n) return fail(MLORA_ERR_CAPACITY, "timeline needs 24 values per phase");
  CK(cudaStreamSynchronize(c->stream));
  CK(cudaMemcpy(host_out, c->step_trace, n * sizeof(long long), cudaMemcpyDeviceToHost));
  return MLORA_OK;
}

// ----------------------------------------------------------------------------- kernel-level calls
int mlora_weight_create(const void* qweight, const void* scales, int32_t K, int32_t N, int32_t G, void* cuda_stream,
                        mlora_weight** out) {
  if (!qweight || !scales || !out) return fail(MLORA_ERR_ARG, "null argument");
  if (init_kernels() != MLORA_OK) return MLORA_ERR_CUDA;
  if (K <= 0 || N <= 0 || G <= 0 || K % 64 || N % 16 || K % G || !wlayout_group_ok(G))
    return fail(MLORA_ERR_UNSUPPORTED, "need K%64==0, N%16==0, K%G==0, G in {64,128,256} or a multiple of 512");
  mlora_weight* w = new mlora_weight();
  w->stream = (cudaStream_t)cuda_stream;
  cudaError_t e = alloc_packed(w->w, K, N, G);
  if (e == cudaSuccess) e = launch_repack((const uint8_t*)qweight, (const __half*)scales, K, N, G, w->w.data, 0, 1, w->stream);
  if (e == cudaSuccess) {
    int dev = 0;
    e = cudaGetDevice(&dev);
    w->device = dev;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&w->sm_count, cudaDevAttrMultiProcessorCount, dev);
  }
  if (e == cudaSuccess) e = cudaMalloc(&w->phase, sizeof(ChainPhase));
  if (e == cudaSuccess) {
    ChainPhase ph{};                    // input and output pointers come with each call
    ph.w = w->w.data; ph.K = K; ph.N = N; ph.G = G; ph.mode = MODE_PLAIN; ph.epi = EPI_F32; ph.in_kind = IN_F16;
    ph.ldo = N; ph.lora_nseg = 1; ph.lora_proj[0] = 0; ph.lora_n[0] = N;
    e = cudaMemcpy(w->phase, &ph, sizeof(ph), cudaMemcpyHostToDevice);
  }
  if (e == cudaSuccess) e = cudaStreamSynchronize(w->stream);
  if (e != cudaSuccess) {
    free_packed(w->w);
    if (w->phase) cudaFree(w->phase);
    delete w;
    return fail(MLORA_ERR_CUDA, cudaGetErrorString(e));
  }
  *out = w;
  return MLORA_OK;
}

int mlora_weight_destroy(mlora_weight* w) {
  if (!w) return MLORA_OK;
  cudaStreamSynchronize(w->stream);
  free_packed(w->w);
  if (w->phase) cudaFree(w->phase);
  delete w;
  return MLORA_OK;
}

int mlora_weight_dequant(mlora_weight* w, void* out_fp16) {
  if (!w || !out_fp16) return fail(MLORA_ERR_ARG, "null argument");
  CK(launch_dequant(w->w.data, w->w.K, w->w.N, w->w.G, 0, 1, (__half*)out_fp16, w->stream));
  return MLORA_OK;
}

// workspace head: 64 bytes of barrier words for the persistent kernel, then the split-K arrival counters
static const size_t LIN_SYNC_BYTES = 64;
static const size_t LIN_COUNTER_BYTES = 16640;
static size_t lin_T_bytes(int M, int rank) { return (((size_t)M * (rank > 0 ? rank : 1) * sizeof(float)) + 255) / 256 * 256; }
static const size_t LIN_ACC_BYTES = (size_t)CHAIN_MAX_ROWS * 3 * 64 * sizeof(unsigned long long);   // shrink sums of <= 8 rows

size_t mlora_linear_workspace_bytes(const mlora_weight* w, int32_t M, int32_t rank) {
  if (!w || M <= 0) return 0;
  // counters + T + split-K partials for up to 8 splits (the planner uses fewer when this does not fit)
  return LIN_COUNTER_BYTES + lin_T_bytes(M, rank) + LIN_ACC_BYTES + (size_t)8 * M * w->w.N * sizeof(float);
}

int mlora_linear(mlora_weight* w, const void* x, int32_t M, const int32_t* row_adapter, const void* const* A,
                 const void* const* B, const float* scale, int32_t n_adapters, int32_t rank, float* y, void* workspace,
                 size_t workspace_bytes) {
  if (!w || !x || !y || !workspace) return fail(MLORA_ERR_ARG, "null argument");
  if (M <= 0 || M > 4096) return fail(MLORA_ERR_UNSUPPORTED, "M must be in 1..4096");
  if (((uintptr_t)x | (uintptr_t)y | (uintptr_t)workspace) & 15) return fail(MLORA_ERR_ARG, "x, y and workspace must be 16-byte aligned");
  const bool lora = row_adapter != nullptr;
  if (lora && (!A || !B || !scale || n_adapters <= 0 || rank <= 0)) return fail(MLORA_ERR_ARG, "incomplete adapter arguments");
  const size_t fixed = LIN_COUNTER_BYTES + lin_T_bytes(M, rank) + LIN_ACC_BYTES;
  if (workspace_bytes < fixed + (size_t)M * w->w.N * sizeof(float)) return fail(MLORA_ERR_CAPACITY, "workspace too small");
  const int m_blocks = (M + GEMM_MAX_MT * 8 - 1) / (GEMM_MAX_MT * 8);
  if ((size_t)((w->w.N + GEMM_NB - 1) / GEMM_NB) * m_blocks > 4096) return fail(MLORA_ERR_UNSUPPORTED, "too many output blocks");
  unsigned char* ws = (unsigned char*)workspace;
  if (M <= CHAIN_MAX_ROWS && (!lora || rank <= 64) && w->w.K % 64 == 0 && w->w.K <= 16384) {
    // few rows: a shrink kernel (the rows' dot products with the adapters' A rows, added to fixed-point sums) and the
    // projection kernel of the decode path, whose weights are in flight while the shrink runs
    LeanArgs a{};
    a.M = M; a.eps = 0.f;
    StepPhase ph{};
    ph.kind = SK_GEMM; ph.w = w->w.data; ph.K = w->w.K; ph.N = w->w.N; ph.G = w->w.G; ph.mode = MODE_PLAIN; ph.epi = EPI_F32;
    ph.in16 = (const __half*)x; ph.norm_in = -1; ph.out_f32 = y; ph.ldo = w->w.N; ph.ssq_out = -1;
    if (lora) {
      a.adapter_idx = row_adapter; a.tabA = (const __half* const*)A; a.tabB = (const __half* const*)B; a.scale = scale;
      a.tab_stride = 1; a.n_slots = n_adapters; a.rank = rank; a.rank_log2 = lean_rank_log2(rank);
      a.tacc = (unsigned long long*)(ws + LIN_COUNTER_BYTES + lin_T_bytes(M, rank));
      ph.lora_nseg = 1; ph.lora_proj[0] = 0; ph.lora_n[0] = w->w.N; ph.t_in = 0;
      StepPhase sh{};
      sh.kind = SK_EMBED; sh.N = w->w.K; sh.norm_in = -1; sh.ssq_out = -1;
      // short rows: whole dot products, stored (a row without adapter is never read); long rows: 1024-element pieces
      // added to sums that a memset zeroes first (measured: 12.8 vs 14.4 us at K = 4096, 35.3 vs 30.7 us at K = 14336)
      sh.pad_ = w->w.K <= 8192 ? 1 : 0;
      if (!sh.pad_) CK(cudaMemsetAsync(a.tacc, 0, (size_t)CHAIN_MAX_ROWS * 3 * rank * sizeof(unsigned long long), w->stream));
      sh.next_nseg = 1; sh.next_proj[0] = 0; sh.next_ld = w->w.K; sh.t_out = 0;
      CK(launch_lean_embed(a, sh, nullptr, nullptr, 0, (const __half*)x, (int*)(ws + 32), w->stream));
      a.late_wait = 1;
    }
    CK(launch_lean_gemm(a, ph, w->stream));
    return MLORA_OK;
  }
  if (M <= CHAIN_MAX_ROWS) {
    // (shapes outside the kernels above) one persistent kernel does shrink, GEMM and expand
    const int stages = chain_pick_stages(w->w.K, lora ? rank : 0);
    if (stages > 0 && chain_phase_fits(w->w.K, MODE_PLAIN, lora ? 1 : 0, rank, stages, w->sm_count)) {
      ChainArgs a{};
      a.phases = w->phase; a.p0 = 0; a.p1 = 1; a.M = M; a.logits = y; a.h_in = (const __half*)x;
      if (lora) {
        a.adapter_idx = row_adapter; a.rows_per_stream = 1;
        a.tabA = (const __half* const*)A; a.tabB = (const __half* const*)B; a.scale = scale;
        a.tab_stride = 1; a.n_slots = n_adapters; a.rank = rank;
      }
      a.T = (float*)(ws + LIN_COUNTER_BYTES);
      a.sync = (unsigned long long*)ws;
      a.status = (int*)(ws + 32);
      a.nstages = stages; a.kmax = w->w.K;
      CK(launch_chain(a, w->sm_count, w->stream));
      return MLORA_OK;
    }
  }
  LoraArgs la{};
  if (lora) {
    la.adapter_idx = row_adapter; la.rows_per_stream = 1;
    la.tabA = (const __half* const*)A; la.tabB = (const __half* const*)B; la.scale = scale;
    la.tab_stride = 1; la.n_slots = n_adapters; la.rank = rank; la.nseg = 1;
    la.seg[0].proj_index = 0; la.seg[0].n = w->w.N;
    la.T = (float*)(ws + LIN_COUNTER_BYTES);
    ShrinkArgs s{};
    s.h_in = (const __half*)x; s.M = M; s.K = w->w.K; s.lora = la;
    CK(launch_shrink(s, w->stream));
  }
  GemmArgs g{};
  g.w = w->w.data; g.K = w->w.K; g.N = w->w.N; g.G = w->w.G; g.h = (const __half*)x; g.M = M;
  g.mode = MODE_PLAIN; g.epi = EPI_F32; g.out_f32 = y; g.ldo = w->w.N;
  g.partial = (float*)(ws + fixed); g.partial_capacity = (workspace_bytes - fixed) / sizeof(float);
  g.counters = (unsigned*)(ws + LIN_SYNC_BYTES);
  g.lora = la;
  if (gemm_tc_eligible(g)) CK(launch_gemm_tc(g, w->sm_count, (int*)(ws + 32), w->stream));
  else CK(launch_gemm(g, w->stream));
  return MLORA_OK;
}

// ----------------------------------------------------------------------------- allocation-free projection
// Scratch of mlora_linear_noalloc: the persistent kernel's barrier words and status (first 64 bytes) and the
// LoRA intermediate T (8 rows x rank 64 floats at most).  Lives in every GPU that loads the library.
static const size_t NOALLOC_SCRATCH_BYTES = 4096;
static const size_t NOALLOC_HEAD_BYTES = 64;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];
static const int NOALLOC_MAX_DEVICES = 64;
static void* g_noalloc_ptr[NOALLOC_MAX_DEVICES];      // device address of the array on each device, once asked for
static std::mutex g_noalloc_mutex;

int mlora_linear_noalloc(mlora_weight* w, const void* x, int32_t M, const int32_t* row_adapter, const void* const* A,
                         const void* const* B, const float* scale, int32_t n_adapters, int32_t rank, float* y) {
  if (!w || !x || !y) return fail(MLORA_ERR_ARG, "null argument");
  const bool lora = row_adapter != nullptr;
  if (lora && (!A || !B || !scale || n_adapters <= 0 || rank <= 0)) return fail(MLORA_ERR_ARG, "incomplete adapter arguments");
  if (((uintptr_t)x | (uintptr_t)y) & 15) return fail(MLORA_ERR_ARG, "x and y must be 16-byte aligned");
  if (M < 1 || M > CHAIN_MAX_ROWS) return fail(MLORA_ERR_CAPACITY, "mlora_linear_noalloc takes 1..8 rows");
  if (lora && rank > CHAIN_MAX_RANK) return fail(MLORA_ERR_CAPACITY, "mlora_linear_noalloc takes LoRA ranks up to 64");
  if (NOALLOC_HEAD_BYTES + (size_t)M * (lora ? rank : 1) * sizeof(float) > NOALLOC_SCRATCH_BYTES)
    return fail(MLORA_ERR_CAPACITY, "rows x rank exceeds the built-in scratch");
  const int stages = chain_pick_stages(w->w.K, lora ? rank : 0);
  if (stages <= 0 || !chain_phase_fits(w->w.K, MODE_PLAIN, lora ? 1 : 0, rank, stages, w->sm_count))
    return fail(MLORA_ERR_CAPACITY, "input width too large for the built-in scratch path: use mlora_linear");
  // the array is looked up on the device the weight lives on; that device must be the current one (the address
  // query below and the launch both go to the current device)
  int dev = 0;
  CK(cudaGetDevice(&dev));
  if (dev != w->device) return fail(MLORA_ERR_ARG, "the weight's device is not the current device");
  if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return fail(MLORA_ERR_UNSUPPORTED, "device ordinal out of range");
  void* scratch = nullptr;
  {
    // the array's name is only a host-side handle: ask the runtime, once per device and with that device
    // current, where the array lives on the device
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_ptr[dev] == nullptr) {
      void* ptr = nullptr;
      CK(cudaGetSymbolAddress(&ptr, g_noalloc_scratch));
      g_noalloc_ptr[dev] = ptr;
    }
    scratch = g_noalloc_ptr[dev];
  }
  // barrier words, abort flag and status start from zero on every call (the array keeps the last call's contents)
  CK(cudaMemsetAsync(scratch, 0, NOALLOC_HEAD_BYTES, w->stream));
  unsigned char* ws = (unsigned char*)scratch;
  ChainArgs a{};
  a.phases = w->phase; a.p0 = 0; a.p1 = 1; a.M = M; a.logits = y; a.h_in = (const __half*)x;
  if (lora) {
    a.adapter_idx = row_adapter; a.rows_per_stream = 1;
    a.tabA = (const __half* const*)A; a.tabB = (const __half* const*)B; a.scale = scale;
    a.tab_stride = 1; a.n_slots = n_adapters; a.rank = rank;
  }
  a.T = (float*)(ws + NOALLOC_HEAD_BYTES);
  a.sync = (unsigned long long*)ws;
  a.status = (int*)(ws + 32);
  a.nstages = stages; a.kmax = w->w.K;
  CK(launch_chain(a, w->sm_count, w->stream));
  return MLORA_OK;
}

int mlora_linear_status(mlora_weight* w, void* workspace) {
  if (!w) return fail(MLORA_ERR_ARG, "null weight");
  unsigned char* ws = (unsigned char*)workspace;
  if (ws == nullptr) {                                   // the built-in array of mlora_linear_noalloc
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev != w->device) return fail(MLORA_ERR_ARG, "the weight's device is not the current device");
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES || g_noalloc_ptr[dev] == nullptr) return MLORA_OK;   // never used: nothing to report
    ws = (unsigned char*)g_noalloc_ptr[dev];
  }
  CK(cudaStreamSynchronize(w->stream));
  int st = 0;
  CK(cudaMemcpy(&st, ws + 32, sizeof(int), cudaMemcpyDeviceToHost));
  if (st != 0) {
    // the barrier words, the abort flag and the status start afresh
    CK(cudaMemset(ws, 0, LIN_SYNC_BYTES));
    return fail(st, st == MLORA_ERR_TIMEOUT ? "device status: a bounded wait of the projection kernel ran out" : "device status");
  }
  return MLORA_OK;
}

static void attn_fill(AttnArgs& a, int n, int T, int Hq, int Hkv, int hd, int P, int suffix_bound) {
  a = AttnArgs{};
  a.P = P; a.n = n; a.T = T; a.Hq = Hq; a.Hkv = Hkv; a.hd = hd;
  a.suffix_bound = suffix_bound;
  attn_plan(a, 148);
}

size_t mlora_attention_workspace_bytes(int32_t n, int32_t T, int32_t Hq, int32_t Hkv, int32_t hd, int32_t P,
                                       int32_t own_capacity) {
  if (n <= 0 || T <= 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv) return 0;
  // the chunking, and with it the scratch, depends on the suffix bound of the call (not monotonically): take the
  // largest need over every bound the capacity allows
  size_t floats = 0;
  for (int sb = 0; sb <= (own_capacity > T ? own_capacity - T : 0); ++sb) {
    AttnArgs a;
    attn_fill(a, n, T, Hq, Hkv, hd, P, sb);
    const size_t f = attn_workspace_floats(a);
    floats = f > floats ? f : floats;
  }
  const size_t rows = (size_t)n * T;
  return rows * (sizeof(unsigned long long) + sizeof(int32_t)) + 256 + floats * sizeof(float);
}

int mlora_attention(const void* q, const void* prefix_k, const void* prefix_v, int32_t P, const void* own_k,
                    const void* own_v, int32_t own_capacity, const int32_t* suffix_len, int32_t suffix_bound,
                    const int32_t* tree_parent, int32_t n, int32_t T, int32_t Hq, int32_t Hkv, int32_t hd, void* out,
                    void* workspace, size_t workspace_bytes, int32_t* status, void* cuda_stream) {
  if (!q || !own_k || !own_v || !suffix_len || !tree_parent || !out || !workspace || !status)
    return fail(MLORA_ERR_ARG, "null argument");
  if (P > 0 && (!prefix_k || !prefix_v)) return fail(MLORA_ERR_ARG, "null prefix");
  if (n <= 0 || T <= 0 || T > 64 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || P < 0) return fail(MLORA_ERR_ARG, "bad shape");
  if (hd != 64 && hd != 128) return fail(MLORA_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  if (suffix_bound < 0 || suffix_bound + T > own_capacity) return fail(MLORA_ERR_CAPACITY, "suffix_bound + n_nodes exceeds own_capacity");
  if (init_kernels() != MLORA_OK) return MLORA_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  AttnArgs a;
  attn_fill(a, n, T, Hq, Hkv, hd, P, suffix_bound);
  const size_t rows = (size_t)n * T;
  const size_t head = (rows * (sizeof(unsigned long long) + sizeof(int32_t)) + 255) / 256 * 256;
  if (workspace_bytes < head + attn_workspace_floats(a) * sizeof(float)) return fail(MLORA_ERR_CAPACITY, "workspace too small");
  unsigned char* ws = (unsigned char*)workspace;
  unsigned long long* anc = (unsigned long long*)ws;
  int32_t* depth = (int32_t*)(ws + rows * sizeof(unsigned long long));
  CK(launch_tree_prep(tree_parent, n, T, anc, depth, status, st));
  a.q = (const __half*)q;
  a.prefix_k = (const __half*)prefix_k; a.prefix_v = (const __half*)prefix_v; a.prefix_head_stride = (size_t)P * hd;
  a.own_k = (const __half*)own_k; a.own_v = (const __half*)own_v;
  a.own_head_stride = (size_t)own_capacity * hd; a.own_stream_stride = a.own_head_stride * Hkv;
  a.suffix_len = suffix_len; a.anc = anc; a.out = (__half*)out; a.status = status; a.depth = depth;
  a.part_o = (float*)(ws + head);
  a.part_ml = a.part_o + (attn_workspace_floats(a) / (hd + 2)) * hd;
  CK(launch_attention(a, st));
  CK(launch_attention_merge(a, st));
  return MLORA_OK;
}

int mlora_quantize_act_int8(const void* x_fp16, int64_t count, float scale, void* out_int8, void* cuda_stream) {
  if (!x_fp16 || !out_int8 || count < 0) return fail(MLORA_ERR_ARG, "quantize_act_int8: null buffer or negative count");
  if (!(scale > 0.f)) return fail(MLORA_ERR_ARG, "quantize_act_int8: scale must be positive");
  if (count == 0) return MLORA_OK;
  CK(launch_quant_act((const __half*)x_fp16, (long long)count, scale, (signed char*)out_int8, (cudaStream_t)cuda_stream));
  return MLORA_OK;
}

int mlora_linear_w4a8(const void* qweight, const void* w_scale, const void* qx, float x_scale, int32_t M, int32_t K,
                      int32_t N, float* y, void* cuda_stream) {
  if (!qweight || !w_scale || !qx || !y) return fail(MLORA_ERR_ARG, "linear_w4a8: null argument");
  if (M < 1 || K < 1 || N < 1) return fail(MLORA_ERR_ARG, "linear_w4a8: non-positive size");
  if (!w4a8_shape_ok(M, K, N))
    return fail(MLORA_ERR_UNSUPPORTED, "linear_w4a8: needs M <= 64, K a multiple of 256 (below 2^31 / 1016), N a multiple of 16");
  if ((reinterpret_cast<uintptr_t>(qweight) & 15) || (reinterpret_cast<uintptr_t>(qx) & 15))
    return fail(MLORA_ERR_ARG, "linear_w4a8: qweight and qx must be 16-byte aligned");
  CK(launch_w4a8((const unsigned char*)qweight, (const __half*)w_scale, (const signed char*)qx, x_scale, M, K, N, y,
                 (cudaStream_t)cuda_stream));
  return MLORA_OK;
}

}  // extern "C"
