// Small kernels around the projections: embedding gather, draft-tree preparation (ancestor masks and
// depths, Sec. 3.5 / App. A.2), row argmax, the streams' first tokens (App. A.1), the greedy longest-accepted-path
// walk and the KV compaction that follows it (Sec. 3.5).  (RoPE and the KV append of a pass happen inside the attention kernel.)
#include "../../include/mlora.h"
#include "common.cuh"

namespace mlora {

// ----------------------------------------------------------------------------- embedding / hidden input
// An id in [vocab, vocab + n_forecast) stands for a forecast row (Sec. 3.5: forecast embeddings ride along with the
// tokens of a DS2D pass): its input is the forecast embedding of that index.
__global__ void embed_kernel(const int32_t* __restrict__ tokens, const __half* __restrict__ embed,
                             const __half* __restrict__ hidden_in, float* __restrict__ X, int d, int vocab,
                             const __half* __restrict__ forecast, int n_forecast, int* __restrict__ status) {
  const int m = blockIdx.x;
  const __half* src;
  if (hidden_in != nullptr) {
    src = hidden_in + (size_t)m * d;
  } else {
    int tok = tokens[m];
    if (tok >= vocab && tok < vocab + n_forecast) {
      src = forecast + (size_t)(tok - vocab) * d;
    } else {
      if (tok < 0 || tok >= vocab) {         // keep the access in bounds, report through the status word
        if (threadIdx.x == 0) atomicCAS(status, 0, -1);
        tok = 0;
      }
      src = embed + (size_t)tok * d;
    }
  }
  for (int k = threadIdx.x * 2; k < d; k += blockDim.x * 2) {
    const float2 v = __half22float2(*reinterpret_cast<const __half2*>(src + k));
    *reinterpret_cast<float2*>(X + (size_t)m * d + k) = v;
  }
}

cudaError_t launch_embed(const int32_t* tokens, const __half* embed, const __half* hidden_in, float* X, int M, int d,
                         int vocab, int* status, cudaStream_t st, const __half* forecast, int n_forecast) {
  embed_kernel<<<M, 256, 0, st>>>(tokens, embed, hidden_in, X, d, vocab, forecast, forecast ? n_forecast : 0, status);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- tree preparation
// One thread per (stream, node): walks to the root, collecting the ancestor-or-self bit mask and the depth.
// A parent outside [0, i) (or a non-root node 0) sets the status word and is treated as the root's child,
// which keeps every later access in bounds.
__global__ void tree_prep_kernel(const int32_t* __restrict__ parent, int n, int T, unsigned long long* __restrict__ anc,
                                 int32_t* __restrict__ depth, int* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * T) return;
  const int s = i / T, t = i % T;
  if (parent == nullptr) {                 // a chain of any length (prefill): no mask word, depth = index
    anc[i] = ~0ull;
    depth[i] = t;
    return;
  }
  const int32_t* par = parent + (size_t)s * T;
  unsigned long long mask = 0ull;
  int d = 0, c = t;
  bool bad = (par[0] != -1);
  for (int it = 0; it < 64 && c > 0; ++it) {
    mask |= 1ull << c;
    int pc = par[c];
    if (pc < 0 || pc >= c) { bad = true; pc = 0; }
    c = pc;
    ++d;
  }
  mask |= 1ull;
  anc[i] = mask;
  depth[i] = d;
  if (bad) atomicCAS(status, 0, -1);
}

cudaError_t launch_tree_prep(const int32_t* parent, int n, int T, unsigned long long* anc, int32_t* depth, int* status,
                             cudaStream_t st) {
  const int total = n * T;
  tree_prep_kernel<<<(total + 127) / 128, 128, 0, st>>>(parent, n, T, anc, depth, status);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- argmax (lowest index on ties)
__global__ void argmax_kernel(const float* __restrict__ logits, int V, int32_t* __restrict__ out) {
  const int m = blockIdx.x;
  const float* row = logits + (size_t)m * V;
  float best = -INFINITY;
  int bi = 0x7fffffff;
  auto take = [&](float v, int i) { if (v > best || (v == best && i < bi)) { best = v; bi = i; } };
  if ((V & 3) == 0 && (reinterpret_cast<uintptr_t>(row) & 15) == 0) {
    // four 16-byte loads per thread in flight (a scalar loop pays one L2 round trip per element)
    const float4* row4 = reinterpret_cast<const float4*>(row);
    const int nv = V >> 2, bd = blockDim.x;
    for (int b = threadIdx.x; b < nv; b += 4 * bd) {
      float4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = (b + u * bd < nv) ? __ldcs(row4 + b + u * bd) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = (b + u * bd) << 2;
        if (b + u * bd < nv) { take(v[u].x, i); take(v[u].y, i + 1); take(v[u].z, i + 2); take(v[u].w, i + 3); }
      }
    }
  } else {
    for (int i = threadIdx.x; i < V; i += blockDim.x) take(row[i], i);
  }
  __shared__ float sb[32];
  __shared__ int si[32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ob = __shfl_xor_sync(0xffffffffu, best, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { sb[warp] = best; si[warp] = bi; }
  __syncthreads();
  if (warp == 0) {
    const int nw = blockDim.x >> 5;
    best = lane < nw ? sb[lane] : -INFINITY;
    bi = lane < nw ? si[lane] : 0x7fffffff;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    if (lane == 0) out[m] = (bi == 0x7fffffff) ? 0 : bi;
  }
}

cudaError_t launch_argmax(const float* logits, int M, int V, int32_t* out, cudaStream_t st) {
  argmax_kernel<<<M, 1024, 0, st>>>(logits, V, out);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- first tokens of the streams (App. A.1)
// After the shared prefill a sampler hands every stream a different first token: the n most probable ids of the
// prefill's last logits, in order of falling logit, equal logits by rising id.  One CTA; round i finds the largest
// key below round i-1's winner.  Key = order-preserving image of the float in the high word (NaN lowest), the
// complemented id in the low word: one unsigned compare gives both rules.  The n rounds re-read the row from L2.
__device__ __forceinline__ unsigned long long topn_key(float v, int i) {
  if (v == 0.f) v = 0.f;                                // -0 and +0 are equal logits: one image for both
  const unsigned b = __float_as_uint(v);
  const unsigned ord = (v != v) ? 0u : ((b & 0x80000000u) ? ~b : (b | 0x80000000u));
  return ((unsigned long long)ord << 32) | (unsigned)(0xffffffffu - (unsigned)i);
}

// the n largest entries of logits[0..V) by a whole CTA of 1024 threads; out may be global or shared memory
__device__ __forceinline__ void block_topn(const float* __restrict__ logits, int V, int n, int32_t* out) {
  __shared__ unsigned long long sb[32];
  __shared__ unsigned long long s_prev;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned long long prev = ~0ull;
  for (int r = 0; r < n; ++r) {
    unsigned long long best = 0ull;                     // below every key (ids are below 2^31: a key's low word is not 0)
    for (int i = threadIdx.x; i < V; i += blockDim.x) {
      const unsigned long long k = topn_key(logits[i], i);
      if (k < prev && k > best) best = k;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
      best = ob > best ? ob : best;
    }
    if (lane == 0) sb[warp] = best;
    __syncthreads();
    if (warp == 0) {
      best = sb[lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
        best = ob > best ? ob : best;
      }
      if (lane == 0) {
        s_prev = best;
        out[r] = (int32_t)(0xffffffffu - (unsigned)(best & 0xffffffffull));
      }
    }
    __syncthreads();
    prev = s_prev;
  }
}

__global__ void __launch_bounds__(1024) topn_kernel(const float* __restrict__ logits, int V, int n, int32_t* __restrict__ out) {
  block_topn(logits, V, n, out);
}

// ----------------------------------------------------------------------------- DS2D draft generation (Sec. 3.5, App. A.2)
// After the accept walk the next tree hangs off the LAST ACCEPTED node: CTA (j, s) takes the logits of forecast row
// j + 1 of that node of stream s and lists its widths[j] most probable ids (ties by rising id) in cand[s][j][.].
__global__ void __launch_bounds__(1024) draft_topk_kernel(const float* __restrict__ logits, int V, int R, int m, int wmax,
                                                        const int32_t* __restrict__ widths, const int32_t* __restrict__ forecast_of,
                                                        const int32_t* __restrict__ acc_len, const int32_t* __restrict__ acc_idx,
                                                        int32_t* __restrict__ cand, int* __restrict__ status) {
  const int j = blockIdx.x, s = blockIdx.y;
  int leaf = acc_idx[(size_t)s * R + acc_len[s] - 1];
  if (leaf < 0 || leaf >= R) leaf = 0;
  int row = forecast_of[leaf] + j;
  int w = widths[j];
  if (row < 0 || row >= R || w < 0 || w > wmax) {      // a malformed template: stay in bounds, report
    if (threadIdx.x == 0) atomicCAS(status, 0, MLORA_ERR_ARG);
    row = 0;
    w = w < 0 ? 0 : wmax;
  }
  block_topn(logits + ((size_t)s * R + row) * V, V, w, cand + ((size_t)s * m + j) * wmax);
}
// The next pass's inputs, row by row: the root takes the bonus token, a draft node of depth d and sibling rank r the
// r-th candidate of forecast row d, a forecast row j the id vocab + j - 1.
__global__ void draft_fill_kernel(const int32_t* __restrict__ level, const int32_t* __restrict__ rank,
                                  const int32_t* __restrict__ cand, const int32_t* __restrict__ next, int n, int R, int m,
                                  int wmax, int V, int32_t* __restrict__ out_tokens, int* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n * R) return;
  const int s = i / R, lv = level[i % R], rk = rank[i % R];
  int tok;
  if (lv == 0) tok = next[s];
  else if (lv > 0 && lv <= m && rk >= 0 && rk < wmax) tok = cand[((size_t)s * m + (lv - 1)) * wmax + rk];
  else if (lv < 0 && -lv <= m) tok = V + (-lv) - 1;
  else { atomicCAS(status, 0, MLORA_ERR_ARG); tok = 0; }
  out_tokens[i] = tok;
}

cudaError_t launch_draft(const float* logits, int V, int n, int R, int m, int wmax, const int32_t* widths,
                         const int32_t* level, const int32_t* rank, const int32_t* forecast_of, const int32_t* acc_len,
                         const int32_t* acc_idx, const int32_t* next, int32_t* cand, int32_t* out_tokens, int* status,
                         cudaStream_t st) {
  draft_topk_kernel<<<dim3((unsigned)m, (unsigned)n), 1024, 0, st>>>(logits, V, R, m, wmax, widths, forecast_of, acc_len, acc_idx, cand, status);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  draft_fill_kernel<<<(n * R + 255) / 256, 256, 0, st>>>(level, rank, cand, next, n, R, m, wmax, V, out_tokens, status);
  return cudaGetLastError();
}

cudaError_t launch_topn(const float* logits, int V, int n, int32_t* out, cudaStream_t st) {
  topn_kernel<<<1, 1024, 0, st>>>(logits, V, n, out);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- greedy longest accepted path
// One warp per stream.  From the root: g = argmax at the current node; the lanes test the candidate
// children in parallel and the lowest matching node index wins; stop when no child carries g.
__global__ void accept_kernel(const int32_t* __restrict__ tokens, const int32_t* __restrict__ parent,
                              const int32_t* __restrict__ argmax, int T, int32_t* __restrict__ acc_len,
                              int32_t* __restrict__ acc_idx, int32_t* __restrict__ next) {
  const int s = blockIdx.x;
  const int lane = threadIdx.x;
  const int32_t* tok = tokens + (size_t)s * T;
  const int32_t* par = parent + (size_t)s * T;
  const int32_t* am = argmax + (size_t)s * T;
  int32_t* idx = acc_idx + (size_t)s * T;
  for (int i = lane; i < T; i += 32) idx[i] = -1;
  __syncwarp();
  int c = 0, len = 1;
  if (lane == 0) idx[0] = 0;
  for (int it = 0; it < T; ++it) {
    const int g = am[c];
    int found = -1;
    for (int base = c + 1; base < T && found < 0; base += 32) {
      const int u = base + lane;
      const bool hit = (u < T) && (par[u] == c) && (tok[u] == g);
      const unsigned b = __ballot_sync(0xffffffffu, hit);
      if (b) found = base + __ffs(b) - 1;
    }
    if (found < 0) break;
    c = found;
    if (lane == 0) idx[len] = c;
    ++len;
  }
  if (lane == 0) {
    acc_len[s] = len;
    next[s] = am[c];
  }
}

cudaError_t launch_accept(const int32_t* tokens, const int32_t* parent, const int32_t* argmax, int n, int T,
                          int32_t* acc_len, int32_t* acc_idx, int32_t* next, cudaStream_t st) {
  accept_kernel<<<n, 32, 0, st>>>(tokens, parent, argmax, T, acc_len, acc_idx, next);
  return cudaGetLastError();
}

// ----------------------------------------------------------------------------- KV compaction
// For (layer, stream, kv head): row suffix+acc_idx[j] moves to row suffix+j, j ascending.  Path indices are
// strictly increasing with acc_idx[j] >= j, so a destination never covers a source that is still to be read.
__global__ void compact_kernel(__half* __restrict__ own_k, __half* __restrict__ own_v, size_t layer_stride,
                               size_t stream_stride, size_t head_stride, int hd, const int32_t* __restrict__ suffix_len,
                               const int32_t* __restrict__ acc_len, const int32_t* __restrict__ acc_idx, int T) {
  const int l = blockIdx.z, s = blockIdx.y, kh = blockIdx.x;
  const int len = acc_len[s], S = suffix_len[s];
  const size_t base = (size_t)l * layer_stride + (size_t)s * stream_stride + (size_t)kh * head_stride;
  const int vecs = hd / 8;                                   // 16-byte pieces per row
  for (int j = 1; j < len; ++j) {
    const int src = acc_idx[(size_t)s * T + j];
    if (src != j) {
      uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if ((int)threadIdx.x < vecs) {
        kv = *reinterpret_cast<const uint4*>(own_k + base + (size_t)(S + src) * hd + threadIdx.x * 8);
        vv = *reinterpret_cast<const uint4*>(own_v + base + (size_t)(S + src) * hd + threadIdx.x * 8);
      }
      __syncthreads();
      if ((int)threadIdx.x < vecs) {
        *reinterpret_cast<uint4*>(own_k + base + (size_t)(S + j) * hd + threadIdx.x * 8) = kv;
        *reinterpret_cast<uint4*>(own_v + base + (size_t)(S + j) * hd + threadIdx.x * 8) = vv;
      }
      __syncthreads();
    }
  }
}

cudaError_t launch_compact(__half* own_k, __half* own_v, size_t layer_stride, size_t stream_stride, size_t head_stride,
                           int L, int n, int Hkv, int hd, const int32_t* suffix_len, const int32_t* acc_len,
                           const int32_t* acc_idx, int T, cudaStream_t st) {
  dim3 grid(Hkv, n, L);
  compact_kernel<<<grid, 32, 0, st>>>(own_k, own_v, layer_stride, stream_stride, head_stride, hd, suffix_len, acc_len,
                                      acc_idx, T);
  return cudaGetLastError();
}

__global__ void advance_kernel(int32_t* __restrict__ suffix_len, const int32_t* __restrict__ acc_len, int n, int fixed) {
  const int s = threadIdx.x;
  if (s < n) suffix_len[s] += (acc_len != nullptr) ? acc_len[s] : fixed;
}

cudaError_t launch_advance(int32_t* suffix_len, const int32_t* acc_len, int n, int fixed, cudaStream_t st) {
  advance_kernel<<<1, 256, 0, st>>>(suffix_len, acc_len, n, fixed);
  return cudaGetLastError();
}

__global__ void copy_f32_kernel(const float* __restrict__ src, float* __restrict__ dst, size_t count) {
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

cudaError_t launch_copy_rows_f32(const float* src, float* dst, size_t count, cudaStream_t st) {
  int blocks = (int)((count + 255) / 256);
  if (blocks > 1024) blocks = 1024;
  if (blocks < 1) blocks = 1;
  copy_f32_kernel<<<blocks, 256, 0, st>>>(src, dst, count);
  return cudaGetLastError();
}

}  // namespace mlora
