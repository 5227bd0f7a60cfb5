/*
 * mlora.h -- C ABI of the multi-LoRA / multi-stream / DS2D decode hot path (sm_100a).
 *
 * One decode or tree-verify step of a LLaMA-style decoder (paper Sec. 3.1) with
 *   - INT4 group-quantised weights, dequantised in registers (Sec. 3.3 "LLM Quantization"),
 *   - one LoRA adapter per stream, handed in at run time as device pointers and selected per row,
 *     never merged into the weights (Sec. 3.2, approach (c); projection formula Eq. 1-4),
 *   - one shared prompt KV segment plus one private KV segment per stream (Sec. 3.4, App. A.1),
 *   - DS2D draft trees verified in a single pass under a tree-ancestor mask, resolved by a greedy
 *     longest-accepted-path rule that compacts the accepted rows' KV (Sec. 3.5, App. A.2).
 *
 * Conventions
 *   - Every function returns an int status (MLORA_OK or a negative MLORA_ERR_*); nothing throws.
 *   - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are host memory.
 *     The library never frees caller memory and writes only to the outputs named below.
 *   - All work is enqueued on the stream given at creation; calls return without synchronising
 *     unless stated.  Argument errors that the host can see are returned at once; errors only the
 *     device can see (a malformed parent array) set a device status word, read by mlora_sync_status.
 *   - Row order of a step with n_streams streams and n_nodes tree nodes: row m = stream * n_nodes + node.
 *   - fp16 = IEEE binary16.  Weight interchange format ("canonical"): for a projection with K input
 *     and N output features, nibbles uint8 [K][N/2] where byte [k][j] holds column 2j in its low and
 *     column 2j+1 in its high nibble, stored nibble = q + 8 with q in [-8,7]; scales fp16 [K/G][N].
 *     Dequantised weight = fp16_round_to_nearest_even(q * scale)  (one fp16 multiply).
 *   - LoRA tensors: A fp16 [r][K] and B fp16 [r][N] (both row-major); the projection computes
 *     y = x W + (alpha/r) * (x A^T) B, i.e. Eq. 1-4 with the low-rank factors A^T (K x r) and B (r x N).
 */
#ifndef MLORA_H
#define MLORA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MLORA_OK = 0,
  MLORA_ERR_ARG = -1,         /* bad argument (null pointer, size out of range, malformed tree) */
  MLORA_ERR_STATE = -2,       /* call out of order (decode before prefill, ...) */
  MLORA_ERR_CAPACITY = -3,    /* a KV segment, the tree size or a workspace would overflow */
  MLORA_ERR_CUDA = -4,        /* a CUDA runtime call failed; see mlora_last_error */
  MLORA_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out */
  MLORA_ERR_UNSUPPORTED = -6  /* shape outside what the kernels implement */
};

/* Projection bits for lora_targets (paper applies LoRA to q,k,v,o -- Sec. 3.1; the MLP ones are an extension). */
enum { MLORA_Q = 1, MLORA_K = 2, MLORA_V = 4, MLORA_O = 8, MLORA_GATE = 16, MLORA_UP = 32, MLORA_DOWN = 64 };

typedef struct mlora_ctx mlora_ctx;       /* a model instance with its KV caches and scratch */
typedef struct mlora_weight mlora_weight; /* one repacked INT4 projection, for the kernel-level calls */

/* Model description (Sec. 3.1).  Pointer arrays are HOST arrays of DEVICE pointers; the tensors
 * they name are read during mlora_create only (weights are repacked into a private layout), except
 * embed and the RMSNorm gains, which are read in place and must outlive the context. */
typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn;
  int32_t vocab;             /* 0: hidden-state input/output, no embedding and no lm_head */
  int32_t group_size;        /* 64 or 128 (any multiple of 64 dividing every K) */
  float rope_theta;          /* RoPE base */
  float rms_eps;
  int32_t rope_style;        /* 0 = half-split pairs (i, i + head_dim/2); anything else: MLORA_ERR_UNSUPPORTED */
  int32_t lora_rank;         /* one rank for all adapters (Sec. 6: all LoRAs have identical shape) */
  int32_t lora_targets;      /* OR of MLORA_Q.. */
  int32_t max_adapters;      /* adapter slots */
  int32_t max_streams;       /* concurrent streams n (Sec. 3.4) */
  int32_t max_prefix;        /* capacity of the shared prompt segment, positions */
  int32_t max_suffix;        /* capacity of each stream's own segment, positions (excluding tree rows) */
  int32_t max_tree;          /* largest draft tree incl. root, <= 64 */
  const void* embed;         /* dev fp16 [vocab][d_model], or NULL when vocab == 0 */
  const void* const* qweight;/* host array [n_layers*7 (+1)]: order q,k,v,o,gate,up,down per layer; last = lm_head */
  const void* const* scales; /* same indexing, dev fp16 [K/G][N] */
  const void* const* rms_attn;/* host array [n_layers] of dev fp16 [d_model] */
  const void* const* rms_ffn;
  const void* rms_final;     /* dev fp16 [d_model], or NULL when vocab == 0 */
  void* cuda_stream;         /* cudaStream_t for every launch; NULL = the legacy default stream */
} mlora_model_desc;

/* Validates the description, allocates KV caches and scratch, repacks the weights (synchronises once).
 * Errors: ARG (null/shape), UNSUPPORTED (head_dim not 64/128, K not a multiple of 64, ...), CUDA. */
int mlora_create(const mlora_model_desc* desc, mlora_ctx** out);
int mlora_destroy(mlora_ctx* ctx);

/* Run-time adapter (Sec. 3.2 (c)): records, for slot, the device pointers A[l*7+p] (fp16 [r][K_p]) and
 * B[l*7+p] (fp16 [r][N_p]) and the scale alpha/r in a device table.  A and B are HOST arrays of
 * n_layers*7 device pointers; entries of projections outside lora_targets are ignored and may be NULL.
 * Nothing is merged, repacked or recompiled; the tensors must stay alive and unchanged until the slot is
 * overwritten.  A == NULL clears the slot (rows that select it then use the base weights).
 * Takes effect for steps enqueued after the call.  Errors: ARG (slot out of range). */
int mlora_set_adapter(mlora_ctx* ctx, int32_t slot, const void* const* A, const void* const* B, float alpha);

/* Shared prefill (App. A.1: one prefill for all streams): runs the n prompt tokens through the BASE
 * weights with a causal mask, fills the shared KV segment, empties every stream's own segment.
 * prompt_ids: dev int32 [n].  out_last_logits: dev fp32 [vocab] or NULL.
 * Errors: ARG, CAPACITY (n > max_prefix), STATE (vocab == 0: use the _h variant). */
int mlora_prefill_shared(mlora_ctx* ctx, const int32_t* prompt_ids, int32_t n, float* out_last_logits);
/* Same with hidden states: hidden dev fp16 [n][d_model]; out_last_hidden dev fp32 [d_model] or NULL. */
int mlora_prefill_shared_h(mlora_ctx* ctx, const void* hidden, int32_t n, float* out_last_hidden);

/* One decode step for n_streams streams (Sec. 3.4): stream s feeds tokens[s] with adapter
 * adapter_idx[s] (-1 = base weights), attends to the shared segment and its own segment, appends its
 * K/V to its own segment and returns the greedy next token.
 * adapter_idx, tokens, out_next: dev int32 [n_streams]; out_logits: dev fp32 [n_streams][vocab] or NULL (then no
 * logits are formed anywhere: the lm_head keeps only each row's running maximum, lowest id on ties).
 * Errors: ARG, STATE (no prefill yet), CAPACITY (own segment full). */
int mlora_decode_step(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx, const int32_t* tokens,
                      int32_t* out_next, float* out_logits);
/* The same step for a caller that holds HOST arrays (Sec. 3.4; the application side of the paper's flow): copies
 * adapter_idx and tokens (host int32 [n_streams], pinned or pageable) to the device on the context's stream,
 * runs the step, copies the greedy next tokens back to out_next_host and synchronises the stream before
 * returning.  Errors: as mlora_decode_step. */
int mlora_decode_step_host(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx_host,
                           const int32_t* tokens_host, int32_t* out_next_host);
/* First tokens of the streams (App. A.1: after the single prefill a sampler picks n distinct tokens, one per stream).
 * logits: dev fp32 [vocab] (the prefill's out_last_logits); out_tokens: dev int32 [n] = the ids of the n largest
 * logits in order of falling logit, equal logits in order of rising id; NaN counts as the smallest value.
 * 1 <= n <= vocab.  Enqueued on the context's stream.  Errors: ARG, STATE (no vocabulary), CUDA. */
int mlora_sample_first(mlora_ctx* ctx, const float* logits, int32_t n, int32_t* out_tokens);
/* A whole generation without host round trips (App. A.1 flowsheet: first tokens, then the n-fold generative model
 * step after step): k_steps greedy decode steps of n_streams streams; step 0 consumes first_tokens, step j the tokens
 * step j - 1 produced, read on the device.  out_tokens: dev int32 [k_steps][n_streams], row j = the tokens produced by
 * step j (row k_steps - 1 is not yet in the cache, like out_next of mlora_decode_step).  Gives exactly the tokens
 * and the cache that k_steps calls of mlora_decode_step give.  On a capturable stream the k_steps steps are ONE CUDA
 * graph, cached by (pointers, k_steps, state of the own segments at the start).  adapter_idx, first_tokens: dev int32
 * [n_streams].  Errors: ARG, STATE, CAPACITY (own segments cannot take k_steps more rows), CUDA. */
int mlora_generate(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx, const int32_t* first_tokens,
                   int32_t k_steps, int32_t* out_tokens);
/* The same with HOST arrays (adapter_idx_host, first_tokens_host: [n_streams]; out_tokens_host: [k_steps][n_streams]):
 * copies in, runs, copies out and synchronises.  The device buffer behind out_tokens_host is allocated at the
 * first call of a larger k_steps * n_streams than any before. */
int mlora_generate_host(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx_host,
                        const int32_t* first_tokens_host, int32_t k_steps, int32_t* out_tokens_host);
/* Hidden-state variant: hidden_in dev fp16 [n_streams][d_model]; hidden_out dev fp32 [n_streams][d_model]
 * (residual stream after the last layer). */
int mlora_decode_step_h(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx, const void* hidden_in,
                        float* hidden_out);

/* DS2D verification (Sec. 3.5): every stream carries a tree of n_nodes tokens; node 0 is the last
 * accepted token (not yet in the cache), parent[0] = -1 and 0 <= parent[i] < i.  All n_streams*n_nodes
 * rows run in one pass; node t sits at position prefix + suffix_s + depth(t) and sees the shared segment,
 * its stream's own segment and its own root path.  Then, per stream, the greedy walk: from the root move to
 * the lowest-index child whose token equals the argmax at the current node, until none matches.
 * out_accept_len [n_streams]: path length (>= 1); out_accept_idx [n_streams][n_nodes]: path node indices,
 * -1 padded; out_next [n_streams]: argmax at the last accepted node (the bonus token).  The accepted rows'
 * K/V are compacted into the stream's own segment, which grows by accept_len.
 * out_logits: dev fp32 [n_streams*n_nodes][vocab] or NULL.  All arrays dev int32.
 * Errors: ARG, STATE, CAPACITY; a malformed parent array sets the device status to MLORA_ERR_ARG. */
int mlora_verify_tree(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx, int32_t n_nodes,
                      const int32_t* tree_tokens, const int32_t* tree_parent, int32_t* out_accept_len,
                      int32_t* out_accept_idx, int32_t* out_next, float* out_logits);

/* DS2D draft generation (Sec. 3.5 inference steps 1-2, App. A.2).  m forecast embeddings (dev fp16 [m][d_model],
 * caller-owned, must stay valid; 1 <= m <= 8) ride along with the tokens of a pass: from now on an input id
 * vocab + j - 1 (j = 1..m) in tree_tokens of mlora_verify_tree / mlora_ds2d_round denotes forecast row j, whose input
 * row is forecast[j - 1].  A forecast row is an ordinary tree row for attention (chain it under its token node with
 * tree_parent); it can never be accepted and its K/V never reaches the cache.  forecast == NULL or m == 0 switches the
 * ids off again.  Errors: ARG, STATE (no vocabulary). */
int mlora_set_forecast(mlora_ctx* ctx, const void* forecast, int32_t m);
/* One DS2D inference step: verifies the tree in tree_tokens exactly as mlora_verify_tree does AND drafts the next tree
 * from the forecast rows of every stream's last accepted node, without a host round trip.  The n_rows rows of a stream
 * are described by four dev int32 arrays shared by all streams: tree_parent as in mlora_verify_tree (here [n_streams]
 * [n_rows] as well); row_level [n_rows]: 0 = root, d >= 1 = draft node of depth d, -j = forecast row j; row_rank
 * [n_rows]: a draft node's position among its parent's children; forecast_of [n_rows]: for a token node the row index
 * of its forecast row 1 (its m forecast rows are consecutive), else ignored; widths [m]: children per node at depth
 * 1..m (each <= max_width <= 32).  out_tree_tokens dev int32 [n_streams][n_rows] (must not alias tree_tokens) receives
 * the next pass's inputs: the bonus token at the root; at a draft node of depth d and rank r the r-th most probable id
 * (ties by rising id) of forecast row d of the last accepted node; vocab + j - 1 at forecast rows.
 * out_logits: dev fp32 [n_streams * n_rows][vocab] or NULL.  n_rows <= max_tree.  Errors: as mlora_verify_tree, plus STATE (no forecast embeddings set); a template that points
 * outside the pass sets the device status to MLORA_ERR_ARG. */
int mlora_ds2d_round(mlora_ctx* ctx, int32_t n_streams, const int32_t* adapter_idx, int32_t n_rows,
                     const int32_t* tree_tokens, const int32_t* tree_parent, const int32_t* row_level,
                     const int32_t* row_rank, const int32_t* forecast_of, const int32_t* widths, int32_t m,
                     int32_t max_width, int32_t* out_accept_len, int32_t* out_accept_idx, int32_t* out_next,
                     int32_t* out_tree_tokens, float* out_logits);

/* ---- state / diagnostics ---- */
int mlora_reset_streams(mlora_ctx* ctx);        /* empties every stream's own segment; keeps the shared one */
int mlora_sync_status(mlora_ctx* ctx);          /* synchronises the stream; returns and clears the device status */
const char* mlora_last_error(mlora_ctx* ctx);   /* text of the last host-side error (ctx may be NULL) */
/* Copies `count` rows starting at row `first` of stream's own segment of `layer` to k_out/v_out
 * (dev fp16 [count][n_kv_heads][head_dim]); writes the stream's current suffix length to *suffix_len (host).
 * stream == -1 reads the shared segment (suffix_len receives the prefix length).  Synchronises. */
int mlora_export_kv(mlora_ctx* ctx, int32_t layer, int32_t stream, int32_t first, int32_t count,
                    int32_t* suffix_len, void* k_out, void* v_out);
/* The whole own segment of one stream in one layer (Sec. 3.4: the stream's private KV segment; the check of the KV
 * compaction of Sec. 3.5 reads it): writes the stream's suffix length to *suffix_len (host) and its first suffix_len
 * rows to k_out/v_out (dev fp16 [suffix_len][n_kv_heads][head_dim]; the buffers must hold max_suffix + max_tree rows).
 * Synchronises.  Errors: ARG, CUDA. */
int mlora_export_state(mlora_ctx* ctx, int32_t layer, int32_t stream, int32_t* suffix_len, void* k_out, void* v_out);
/* Writes the dequantised weights of (layer, proj) as the GEMM kernel's own unpack path produces them:
 * out dev fp16 [K][N].  proj 0..6 = q,k,v,o,gate,up,down; layer == n_layers, proj == 0 = lm_head. */
int mlora_debug_dequant(mlora_ctx* ctx, int32_t layer, int32_t proj, void* out_fp16);
/* Debug switches: key 1 = skip KV compaction and suffix growth in mlora_verify_tree (tree rows stay where
 * the pass wrote them: rows suffix_len .. suffix_len + n_nodes - 1 of the own segment).
 * key 2 = 1 disables CUDA-graph replay of steps (every kernel launched directly).
 * key 3 = 1 runs decode-sized passes through the general split-K kernels (one per operation: norm + shrink, projection,
 *         attention, ...) instead of any of the decode paths of key 6.
 * key 4 = 1 runs passes of 32 rows and more through the split-K mma.sync kernels instead of the tcgen05 projection kernel.
 * key 5 = 1 makes the first wait of the next decode step (paths 1 and 2 of key 6) run out, on a flag nothing sets: the
 *         step returns the timeout status instead of hanging (the test of the bounded waits).
 * key 6 picks the path of decode steps (one row per stream, at most 8 streams): 1 = the per-layer persistent projection
 *         kernel plus attention kernels; 2 = ONE kernel that does the whole step (embedding to greedy token; where the
 *         model's shapes allow it, else the per-layer path); 3 = one small kernel per projection group, launched
 *         programmatically so that each one's weights are in flight while the one before it drains (contexts up to
 *         2047 keys; longer ones take the per-layer path); 0 = the library's choice (3 where it applies: the fastest of
 *         the three at the 1B / 8-stream shapes).  All are replayed from CUDA graphs.
 * key 7 = 1 makes decode steps of paths 2 and 3 (key 6) record a timeline (see mlora_step_timeline); path 3 then runs
 *         instantiations of its kernels that carry the stamps (the untraced ones carry none). */
int mlora_debug_set(mlora_ctx* ctx, int32_t key, int32_t value);
/* Timeline of the LAST decode step that ran with debug key 7 set (Sec. 3.1 decoder: the step's phases are the
 * embedding, then q,k,v projection / attention / o projection / gate,up projection / down projection per layer,
 * then lm_head and the closing phase).  host_out receives [2][n_phases][12] values taken by thread 0 of the first
 * (index 0) and of the last (index 1) CTA: slots 0..9 are readings of that SM's cycle counter (only differences
 * within one CTA mean anything): 0 phase start, 7 phase set-up done, 8 first weights in shared memory, 9 first tile
 * multiplied, 10 all tiles of the first batch multiplied, 1 main loop (attention: the row's q,k,v in shared memory) done, 2 partial sums parked (attention: all
 * key tiles done), 3 epilogue done, 4 phase work done, 5 CTA at the grid barrier, 6 barrier passed; 0 where a point
 * does not apply.  Slot 11 of the first phase / of the last phase holds the GPU's global nanosecond timer at the
 * step's start / end.
 * Path 3 (one kernel per projection group; the embedding and closing phases are not stamped): every slot is a reading of
 * the GPU's GLOBAL nanosecond timer, comparable across CTAs and kernels: 0 kernel start, 1 its wait for the kernel ahead
 * returned, 2 main loop (attention: key tiles) done, 3 end, for thread 0 of the launch's first CTA (index 0) and of its
 * last CTA (index 1; not for attention); slot 4 of index 0 = the latest end over ALL CTAs of the launch.
 * capacity = values host_out holds (>= 24 * n_phases); *n_phases receives the phase count.
 * Synchronises.  Errors: ARG, STATE, CAPACITY, CUDA. */
int mlora_step_timeline(mlora_ctx* ctx, int64_t* host_out, int32_t capacity, int32_t* n_phases);
/* Per-kernel-family device time of the NEXT steps, measured with CUDA events on the context's stream.
 * mlora_profile_begin switches to direct launches with an event pair around every run of consecutive launches of one
 * family (kernels of a run keep whatever overlap they have among themselves); mlora_profile_end
 * synchronises, switches back, and fills ms[family] / launches[family] (host arrays of MLORA_PROF_FAMILIES). */
enum { MLORA_PROF_GEMM = 0, MLORA_PROF_SHRINK = 1, MLORA_PROF_ATTN = 2, MLORA_PROF_ATTN_MERGE = 3,
       MLORA_PROF_ROPE_KV = 4 /* unused: RoPE and the KV append run inside the attention kernel */, MLORA_PROF_MISC = 5,
       MLORA_PROF_FAMILIES = 6 };
int mlora_profile_begin(mlora_ctx* ctx);
int mlora_profile_end(mlora_ctx* ctx, float* ms, int32_t* launches);
/* Kernels launched by this context since creation (direct launches plus graph-replayed nodes). */
int64_t mlora_launch_count(mlora_ctx* ctx);

/* ---- kernel-level calls (single projection, single attention pass) ---- */

/* Repacks one canonical INT4 projection (dev qweight uint8 [K][N/2], dev scales fp16 [K/G][N]) into the
 * kernels' private layout.  Synchronises.  K % 64 == 0, N % 16 == 0, G % 64 == 0, K % G == 0. */
int mlora_weight_create(const void* qweight, const void* scales, int32_t K, int32_t N, int32_t G,
                        void* cuda_stream, mlora_weight** out);
int mlora_weight_destroy(mlora_weight* w);
int mlora_weight_dequant(mlora_weight* w, void* out_fp16 /* dev [K][N] */);

/* Bytes of caller-provided scratch mlora_linear needs for M rows on w with rank-r adapters. */
size_t mlora_linear_workspace_bytes(const mlora_weight* w, int32_t M, int32_t rank);
/* y[m] = x[m] Wdeq + scale[a] * (x[m] A[a]^T) B[a], a = row_adapter[m] (Eq. 1-4; fused INT4 GEMM + LoRA).
 * x dev fp16 [M][K]; row_adapter dev int32 [M] (-1 = base) or NULL for no LoRA; A, B: DEV arrays of
 * n_adapters device pointers (fp16 [rank][K], fp16 [rank][N]); scale dev fp32 [n_adapters] (= alpha/r);
 * y dev fp32 [M][N]; workspace dev, zero-filled before first use (the call leaves it zeroed where it matters).
 * x, y, workspace and every A[a], B[a] must be 16-byte aligned (the kernels use 128-bit loads and bulk copies).
 * Errors: ARG (null or misaligned pointer), CAPACITY (workspace too small), UNSUPPORTED (M > 4096).  A bounded wait
 * that runs out on the device is reported by mlora_linear_status. */
int mlora_linear(mlora_weight* w, const void* x, int32_t M, const int32_t* row_adapter, const void* const* A,
                 const void* const* B, const float* scale, int32_t n_adapters, int32_t rank, float* y,
                 void* workspace, size_t workspace_bytes);

/* Allocation-free variant of mlora_linear for at most 8 rows (the paper has no counterpart: this is a
 * convenience of this library).  It is meant for callers that must not allocate device memory when they
 * issue work: a serving loop whose memory was reserved up front and that cannot afford the device-wide
 * synchronisation an allocation may cause, or code that holds no allocator at all at that point.  Same
 * operation, arguments and result as mlora_linear, but the kernel's scratch (its barrier words and the LoRA
 * intermediate) is a 4096-byte array built into the library, present on every GPU that loads it; the call
 * itself makes no cudaMalloc/cudaFree and calls no allocating routine.  (mlora_weight_create, done once
 * beforehand, does allocate.)
 * Limits: 1 <= M <= 8, rank <= 64, and an input width K small enough for the single-kernel path (K <= 8192
 * on a B200); anything beyond returns MLORA_ERR_CAPACITY and runs nothing -- use mlora_linear there.
 * The array used is the one on the weight's device, which must be the current device (else MLORA_ERR_ARG).
 * The first call on a device looks up the array's device address; make that call outside any stream capture.
 * All calls on a device share the one array: two calls that overlap on the GPU (different streams) race;
 * calls on the weight's own stream, or otherwise ordered, are fine.
 * A bounded wait that runs out on the device (e.g. after such a race) leaves garbage in y: mlora_linear_status(w, NULL)
 * reports and clears it.  Errors: ARG (null or misaligned pointer, wrong device), CAPACITY, UNSUPPORTED, CUDA. */
int mlora_linear_noalloc(mlora_weight* w, const void* x, int32_t M, const int32_t* row_adapter, const void* const* A,
                         const void* const* B, const float* scale, int32_t n_adapters, int32_t rank, float* y);

/* Device status of the mlora_linear calls made with `workspace` (workspace == NULL: of the mlora_linear_noalloc calls
 * on the weight's device, which must be current).  Synchronises the weight's stream; returns MLORA_OK, or the status
 * (MLORA_ERR_TIMEOUT: a bounded wait ran out and the last result is garbage) after clearing it together with the
 * kernel's barrier words, so that the next call starts afresh.  Allocates nothing.  Errors: ARG, CUDA, TIMEOUT. */
int mlora_linear_status(mlora_weight* w, void* workspace);

/* ---- the paper's own precision regime, single projection (Sec. 3.3 "LLM Quantization": activations quantised per
 * tensor to Int8, weights per channel to Int4) ----
 * mlora_quantize_act_int8: out[i] = clip(round_half_even(x[i] / scale), -127, 127) with the division in float32.
 * x dev fp16 [count], out dev int8 [count], scale > 0 (host).  Enqueued on cuda_stream.  Errors: ARG, CUDA.
 * mlora_linear_w4a8: y[m][n] = float32(sum_k qx[m][k] * qw[n][k]) * (x_scale * float32(w_scale[n])): the sum in exact
 * integer arithmetic (tensor cores, s8 x s8 -> s32), the two products in float32, so the result is reproducible bit
 * for bit.  qweight dev uint8 [N][K/2] (channel-major; the nibble of input k is q + 8, even k in the low nibble);
 * w_scale dev fp16 [N]; qx dev int8 [M][K]; y dev fp32 [M][N].  qweight and qx 16-byte aligned.  1 <= M <= 64,
 * K a multiple of 256, N a multiple of 16 (UNSUPPORTED otherwise).  No adapter term, no scratch memory.
 * Errors: ARG, UNSUPPORTED, CUDA. */
int mlora_quantize_act_int8(const void* x_fp16, int64_t count, float scale, void* out_int8, void* cuda_stream);
int mlora_linear_w4a8(const void* qweight, const void* w_scale, const void* qx, float x_scale, int32_t M, int32_t K,
                      int32_t N, float* y, void* cuda_stream);

/* Bytes of scratch for mlora_attention (the largest need over every suffix_bound up to own_capacity - n_nodes). */
size_t mlora_attention_workspace_bytes(int32_t n_streams, int32_t n_nodes, int32_t n_q_heads, int32_t n_kv_heads,
                                       int32_t head_dim, int32_t prefix_len, int32_t own_capacity);
/* Shared-prefix + own-segment + tree-ancestor attention (Sec. 3.4/3.5, App. A.1/A.2) for
 * n_streams*n_nodes query rows.  q dev fp16 [rows][n_q_heads][head_dim] (already rotated);
 * prefix_k/v dev fp16 [n_kv_heads][prefix_len][head_dim]; own_k/v dev fp16 [n_streams][n_kv_heads][own_capacity][head_dim]
 * holding suffix_len[s] cached rows followed by the n_nodes tree rows; suffix_len dev int32 [n_streams];
 * suffix_bound host upper bound of all suffix_len; tree_parent dev int32 [n_streams][n_nodes];
 * out dev fp16 [rows][n_q_heads][head_dim].  status dev int32 [1] receives MLORA_ERR_ARG for a bad tree. */
int mlora_attention(const void* q, const void* prefix_k, const void* prefix_v, int32_t prefix_len,
                    const void* own_k, const void* own_v, int32_t own_capacity, const int32_t* suffix_len,
                    int32_t suffix_bound, const int32_t* tree_parent, int32_t n_streams, int32_t n_nodes,
                    int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, void* out, void* workspace,
                    size_t workspace_bytes, int32_t* status, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* MLORA_H */
