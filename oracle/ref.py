"""CPU oracle for the multi-LoRA / multi-stream / DS2D decode step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, dense restatement of what one decode or tree-verify step computes, written from
the paper's definitions.  It shares no code with the CUDA path and must never be imported by
the product: only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

What follows which passage:
  * LoRA-augmented projection  Y = X W + X (s A B)                      -- Sec. 3.1, Eq. 1-4
  * adapters handed in at run time, all of one shape, picked per stream  -- Sec. 3.2 (approach c), Sec. 6
  * decoder block: RMSNorm, q/k/v projections, RoPE on q and k, attention,
    o projection, RMSNorm, gated MLP                                     -- Sec. 3.1
  * INT4 weights (here symmetric, per group along the input dimension,
    fp16 scales; dequantised value = fp16(q * scale))                    -- Sec. 3.3 "LLM Quantization"
  * one shared prefill KV segment + one isolated KV segment per stream;
    a stream's token sees the prefill segment and its own segment only  -- Sec. 3.4, App. A.1 (CTG mask)
  * draft tree from a branch configuration, verified in one pass in which
    a node sees the cached context plus its own ancestors               -- Sec. 3.5, App. A.2 (DS2D mask)
  * accepted drafts form one root path ("1-3-5"); first emitted token is
    the frozen model's own token (lossless)                              -- Sec. 3.5
  * the paper's own precision regime: activations per-tensor INT8, weights
    per-channel INT4, integer contraction (single projection)            -- Sec. 3.3 "LLM Quantization"
  * after the single prefill a sampler gives the n streams n distinct
    first tokens (here: the n most probable, by falling logit, ties by
    rising id), then the n-fold model runs step after step              -- App. A.1 (flowsheet)
  * m forecast embeddings ride along with every token node of the pass
    as further rows chained under it; the top-b_j ids of forecast row j
    of the last accepted node become the next tree's depth-j drafts     -- Sec. 3.5 (inference steps 1-2), App. A.2

Arithmetic: everything after dequantisation is carried in ``dtype`` (float64 by default; float32
for the 1B/3B shapes where the dense weights would not fit twice in memory).  No blocking, no
fusion, no reordering: projections are full matmuls, attention is a softmax over an explicitly
concatenated key list, the accept rule is a sequential walk.

Pins (tests/test_oracle_*.py): dequant against hand-decoded bytes and an independent int/Fraction
computation; base projection against numpy matmul; run-time LoRA against the merged dense matrix
and the one-hot-masked sum of Sec. 3.2 (approach b); stream isolation; tree rows against sequential
decode of each root path; shared-prefix attention against plain causal attention over the
concatenated sequence; RoPE/RMSNorm/SiLU closed forms; accept walk against brute force on every
small tree; the (3,2) -> 9/10/30 node counts and the 32-row budgets of Table 7; the wiring of a decoder block
(norm placement, residuals, gate/up roles, final norm) against scalar loops written from the definitions
(tests/test_oracle_wiring_pin.py); the first-token sampler against exhaustive selection on small rows with ties and
against argmax for n = 1 (tests/test_oracle_generate.py); DS2D drafting: the printed row counts of the (3,2) example,
forecast rows against the same vectors planted as ordinary embedding rows, draft placement by explicit loops, and
losslessness of whole drafting rounds against plain greedy decoding (tests/test_oracle_ds2d_draft.py); the INT4 x INT8
projection against Python-integer brute force, the float product of the dequantised operands and the quantisation error
bound (tests/test_oracle_w4a8.py).
Parity unpinned by the paper: absolute activation values of a forward pass of ITS model (it prints none).
"""
import numpy as np

PROJ = ("q", "k", "v", "o", "gate", "up", "down")
PROJ_BIT = {"q": 1, "k": 2, "v": 4, "o": 8, "gate": 16, "up": 32, "down": 64}


# ----------------------------------------------------------------------------- INT4 (Sec. 3.3)
def unpack_int4(qbytes: np.ndarray) -> np.ndarray:
    """uint8 [K][N/2] -> int8 [K][N] in [-8, 7].  Low nibble = even column; stored nibble is q + 8."""
    K, half = qbytes.shape
    q = np.empty((K, half * 2), dtype=np.int16)
    q[:, 0::2] = qbytes & 0x0F
    q[:, 1::2] = qbytes >> 4
    return (q - 8).astype(np.int8)


def dequant(qbytes: np.ndarray, scales: np.ndarray, group: int) -> np.ndarray:
    """Dequantised weights as fp16 values: fp16_round_nearest_even(q * scale).

    q in [-8,7] times an fp16 scale is exact in float32 (4 + 11 significand bits), so the single
    conversion to float16 is the only rounding.
    """
    q = unpack_int4(qbytes).astype(np.float32)
    s = np.repeat(scales.astype(np.float32), group, axis=0)
    assert s.shape == q.shape
    with np.errstate(over="ignore"):
        return (q * s).astype(np.float16)


# ----------------------------------------------------------------------------- the INT4 x INT8 regime (Sec. 3.3)
def quantize_act_int8(x, scale):
    """Per-tensor symmetric INT8 activations: q = clip(round_half_even(x / scale), -127, 127), the division carried in
    float32 (the precision the kernel takes this decision in)."""
    q = np.rint(np.asarray(x, dtype=np.float32) / np.float32(scale))
    return np.clip(q, -127, 127).astype(np.int8)


def linear_w4a8(qx, x_scale, qw_bytes, w_scale):
    """Projection with per-channel INT4 weights and per-tensor INT8 activations (Sec. 3.3 "LLM Quantization":
    activations per-tensor to Int8, weights per-channel to Int4).

    qx int8 [M][K]; qw_bytes uint8 [N][K/2] (channel-major, nibble q + 8, even k low); w_scale fp16 [N].
    The contraction is exact integer arithmetic; y[m][n] = float32(acc) * (float32(x_scale) * float32(w_scale[n])),
    both products in float32 (the format fixes this precision, so the result is reproducible bit for bit)."""
    qw = unpack_int4(np.asarray(qw_bytes)).astype(np.int64)            # [N][K]
    acc = np.asarray(qx).astype(np.int64) @ qw.T                        # exact
    assert np.abs(acc).max() < 2 ** 31
    f = np.float32(x_scale) * np.asarray(w_scale).astype(np.float32)    # [N], float32
    return acc.astype(np.float32) * f[None, :]


# ----------------------------------------------------------------------------- elementwise pieces (Sec. 3.1)
def rmsnorm(x, gain, eps):
    x = np.asarray(x)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def silu(x):
    return x / (1.0 + np.exp(-x))


def rope(x, pos, theta):
    """Rotary embedding, half-split pairing: element i rotates with element i + hd/2.

    x: [..., hd]; pos: integer positions broadcastable to x.shape[:-1]; angle = pos * theta^(-2i/hd).
    """
    hd = x.shape[-1]
    half = hd // 2
    inv = theta ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv
    c, s = np.cos(ang).astype(x.dtype), np.sin(ang).astype(x.dtype)
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


# ----------------------------------------------------------------------------- LoRA projection (Eq. 1-4)
def linear_lora(h, W, row_adapter=None, A=None, B=None, scale=None):
    """y[m] = h[m] W + scale[a] * (h[m] A[a]^T) B[a],  a = row_adapter[m]  (a < 0: base only).

    W: [K][N] dense (dequantised) weights.  A[a]: [r][K], B[a]: [r][N] as stored; in the paper's
    row-vector notation the low-rank factors are A^T (K x r) and B (r x N).
    """
    y = h @ W
    if row_adapter is None:
        return y
    for m, a in enumerate(row_adapter):
        if a < 0 or A[a] is None:
            continue
        t = h[m] @ A[a].T.astype(h.dtype)
        y[m] += scale[a] * (t @ B[a].astype(h.dtype))
    return y


# ----------------------------------------------------------------------------- attention
def attend(q, keys, vals):
    """Softmax attention of one query row over an explicit key list.

    q: [Hq][hd]; keys, vals: [n][Hkv][hd]; query head j uses kv head j // (Hq/Hkv).
    """
    Hq, hd = q.shape
    Hkv = keys.shape[1]
    g = Hq // Hkv
    out = np.empty_like(q)
    for j in range(Hq):
        k = keys[:, j // g, :]
        v = vals[:, j // g, :]
        s = (k @ q[j]) / np.sqrt(hd)
        s = s - s.max()
        p = np.exp(s)
        out[j] = (p / p.sum()) @ v
    return out


def causal_attention(q, k, v):
    """Plain causal attention over one sequence: q [P][Hq][hd], k/v [P][Hkv][hd] -> [P][Hq][hd]."""
    P, Hq, hd = q.shape
    g = Hq // k.shape[1]
    out = np.empty_like(q)
    mask = np.triu(np.ones((P, P), dtype=bool), 1)
    for j in range(Hq):
        s = (q[:, j, :] @ k[:, j // g, :].T) / np.sqrt(hd)
        s[mask] = -np.inf
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        out[:, j, :] = (p / p.sum(axis=1, keepdims=True)) @ v[:, j // g, :]
    return out


def tree_attention(q, prefix_k, prefix_v, suf_k, suf_v, tree_k, tree_v, parents):
    """Attention of n*T tree rows (row m = s*T + t) under the stream-isolation and tree-ancestor masks.

    Row (s,t) sees, in this order: every shared-prefix position, stream s's own suffix, and the tree
    rows of stream s that lie on the root path of t (t included).  q: [n*T][Hq][hd];
    prefix_*: [P][Hkv][hd]; suf_*[s]: [S_s][Hkv][hd]; tree_*: [n*T][Hkv][hd]; parents[s]: parent list.
    """
    n = len(parents)
    T = len(parents[0])
    o = np.empty_like(q)
    for m in range(n * T):
        s, t = divmod(m, T)
        own = [s * T + u for u in ancestors_and_self(parents[s], t)]
        keys = np.concatenate([prefix_k, suf_k[s], tree_k[own]], axis=0)
        vals = np.concatenate([prefix_v, suf_v[s], tree_v[own]], axis=0)
        o[m] = attend(q[m], keys, vals)
    return o


# ----------------------------------------------------------------------------- draft trees (Sec. 3.5)
def check_parents(parent):
    parent = [int(p) for p in parent]
    if len(parent) == 0 or parent[0] != -1:
        raise ValueError("node 0 must be the root (parent -1)")
    for i in range(1, len(parent)):
        if not (0 <= parent[i] < i):
            raise ValueError("parent[i] must satisfy 0 <= parent[i] < i")
    return parent


def ancestors_and_self(parent, t):
    """Indices, ascending, of the nodes a draft node may see among the tree rows: its root path."""
    path = []
    while t >= 0:
        path.append(t)
        t = int(parent[t])
    return path[::-1]


def depths(parent):
    d = [0] * len(parent)
    for i in range(1, len(parent)):
        d[i] = d[int(parent[i])] + 1
    return d


def accept_walk(tokens, parent, argmax):
    """Greedy longest accepted root path.

    Start at the root (always accepted).  At the current node c the model's own next token is
    argmax[c]; move to the lowest-index child of c whose draft token equals it, stop when there is
    none.  Returns (path indices, bonus token = argmax at the last accepted node).
    """
    parent = check_parents(parent)
    c, path = 0, [0]
    while True:
        g = int(argmax[c])
        nxt = -1
        for u in range(c + 1, len(parent)):
            if parent[u] == c and int(tokens[u]) == g:
                nxt = u
                break
        if nxt < 0:
            return path, g
        c = nxt
        path.append(c)


def first_tokens(logits, n):
    """The n distinct first tokens of the streams (App. A.1): the ids of the n largest logits, listed by
    falling logit, equal logits by rising id.  NaN ranks below every number."""
    vals = [float(v) for v in np.asarray(logits).reshape(-1)]
    vals = [float("-inf") if v != v else v for v in vals]
    nan_ids = {i for i, v in enumerate(np.asarray(logits).reshape(-1)) if v != v}
    # a NaN ranks below a true -inf: second sort key
    order = sorted(range(len(vals)), key=lambda i: (-vals[i], i in nan_ids, i))
    assert 1 <= n <= len(vals)
    return np.array(order[:n], dtype=np.int32)


# ----------------------------------------------------------------------------- the model
class OracleModel:
    """Dense CPU model with a shared-prefix KV segment and one private KV segment per stream."""

    def __init__(self, cfg, qweight, scales, rms_attn, rms_ffn, rms_final=None, embed=None,
                 dtype=np.float64, max_adapters=64):
        self.cfg = cfg
        self.dt = np.dtype(dtype)
        self.qweight, self.scales = qweight, scales
        self.rms_attn = [g.astype(self.dt) for g in rms_attn]
        self.rms_ffn = [g.astype(self.dt) for g in rms_ffn]
        self.rms_final = None if rms_final is None else rms_final.astype(self.dt)
        self.embed = embed
        self._W = {}
        self.A = [None] * max_adapters
        self.B = [None] * max_adapters
        self.s = [0.0] * max_adapters
        self.prefix_k, self.prefix_v = None, None   # per layer [P][Hkv][hd]
        self.suf_k, self.suf_v = None, None         # [layer][stream] -> [S][Hkv][hd]

    @classmethod
    def from_synth(cls, m, **kw):
        return cls(m.cfg, m.qweight, m.scales, m.rms_attn, m.rms_ffn, m.rms_final, m.embed, **kw)

    # -- weights
    def W(self, idx):
        if idx not in self._W:
            self._W[idx] = dequant(self.qweight[idx], self.scales[idx], self.cfg.group_size).astype(self.dt)
        return self._W[idx]

    def set_adapter(self, slot, A, B, alpha):
        """Run-time adapter: lists indexed layer*7+proj of fp16 [r][K] / [r][N]; scale s = alpha / r."""
        if A is None:
            self.A[slot] = self.B[slot] = None
            return
        self.A[slot], self.B[slot] = A, B
        r = next(a.shape[0] for a in A if a is not None)
        self.s[slot] = float(alpha) / r

    def _linear(self, l, p, h, row_adapter):
        idx = l * 7 + p
        targeted = self.cfg.lora_targets & PROJ_BIT[PROJ[p]]
        if row_adapter is None or not targeted:
            return h @ self.W(idx)
        A = [None if a is None else a[idx] for a in self.A]
        B = [None if b is None else b[idx] for b in self.B]
        return linear_lora(h, self.W(idx), row_adapter, A, B, self.s)

    # -- state
    @property
    def P(self):
        return 0 if self.prefix_k is None else self.prefix_k[0].shape[0]

    def suffix_len(self, s):
        return self.suf_k[0][s].shape[0]

    def reset_streams(self, n_streams):
        c = self.cfg
        z = lambda: np.zeros((0, c.n_kv_heads, c.head_dim), dtype=self.dt)
        self.suf_k = [[z() for _ in range(n_streams)] for _ in range(c.n_layers)]
        self.suf_v = [[z() for _ in range(n_streams)] for _ in range(c.n_layers)]

    def set_forecast(self, forecast):
        """m forecast embeddings [m][d_model] (Sec. 3.5): an input id vocab + j - 1 stands for forecast row j."""
        self.forecast = None if forecast is None else np.asarray(forecast)

    def _embed(self, tokens):
        tokens = np.asarray(tokens).reshape(-1)
        fc = getattr(self, "forecast", None)
        if fc is None:
            return self.embed[tokens].astype(self.dt)
        V = self.cfg.vocab
        assert tokens.max() < V + len(fc)
        table = np.concatenate([self.embed, fc.astype(self.embed.dtype)], axis=0)
        return table[tokens].astype(self.dt)

    def _mlp(self, l, X, row_adapter):
        c = self.cfg
        h2 = rmsnorm(X, self.rms_ffn[l], c.rms_eps)
        act = silu(self._linear(l, 4, h2, row_adapter)) * self._linear(l, 5, h2, row_adapter)
        return X + self._linear(l, 6, act, row_adapter)

    def _logits(self, X):
        c = self.cfg
        return rmsnorm(X, self.rms_final, c.rms_eps) @ self.W(c.n_layers * 7)

    # -- prefill: base weights, causal, fills the shared segment (App. A.1: "a single Prefill model execution")
    def prefill_shared(self, prompt_ids=None, hidden=None, n_streams=None):
        c = self.cfg
        X = self._embed(prompt_ids) if hidden is None else np.asarray(hidden).astype(self.dt)
        P = X.shape[0]
        pos = np.arange(P)
        self.prefix_k, self.prefix_v = [], []
        for l in range(c.n_layers):
            h = rmsnorm(X, self.rms_attn[l], c.rms_eps)
            q = self._linear(l, 0, h, None).reshape(P, c.n_q_heads, c.head_dim)
            k = self._linear(l, 1, h, None).reshape(P, c.n_kv_heads, c.head_dim)
            v = self._linear(l, 2, h, None).reshape(P, c.n_kv_heads, c.head_dim)
            q = rope(q, pos[:, None], c.rope_theta)
            k = rope(k, pos[:, None], c.rope_theta)
            self.prefix_k.append(k)
            self.prefix_v.append(v)
            o = causal_attention(q, k, v).reshape(P, -1)
            X = X + self._linear(l, 3, o, None)
            X = self._mlp(l, X, None)
        self.reset_streams(n_streams if n_streams is not None else c.n_streams)
        if c.vocab > 0:
            return self._logits(X[-1:])[0]
        return X[-1]

    # -- one verify pass over n_streams trees of T nodes (T = 1: a plain decode step)
    def verify_tree(self, adapter_idx, tree_parent, tree_tokens=None, hidden=None, follow_argmax=None,
                    commit=True):
        """Rows m = s*T + t.  Row (s,t) sits at position P + S_s + depth(t) and sees the shared prefix,
        stream s's own suffix, and the tree rows of stream s on its root path (itself included).

        follow_argmax: optional int array [n][T]; when given, the accept walk uses these per-row
        tokens instead of the oracle's own argmax (used to keep histories aligned when a
        lower-precision implementation breaks a near-tie differently).
        Returns dict(logits | hidden, argmax, accept_len, accept_idx, next).
        """
        c = self.cfg
        adapter_idx = [int(a) for a in adapter_idx]
        n = len(adapter_idx)
        tree_parent = np.asarray(tree_parent).reshape(n, -1)
        T = tree_parent.shape[1]
        par = [check_parents(tree_parent[s]) for s in range(n)]
        dep = [depths(p) for p in par]
        X = self._embed(tree_tokens) if hidden is None else np.asarray(hidden).astype(self.dt).reshape(n * T, -1)
        row_adapter = [adapter_idx[m // T] for m in range(n * T)]
        P = self.P
        pos = np.array([P + self.suffix_len(m // T) + dep[m // T][m % T] for m in range(n * T)])
        new_k, new_v = [], []
        for l in range(c.n_layers):
            h = rmsnorm(X, self.rms_attn[l], c.rms_eps)
            q = self._linear(l, 0, h, row_adapter).reshape(n * T, c.n_q_heads, c.head_dim)
            k = self._linear(l, 1, h, row_adapter).reshape(n * T, c.n_kv_heads, c.head_dim)
            v = self._linear(l, 2, h, row_adapter).reshape(n * T, c.n_kv_heads, c.head_dim)
            q = rope(q, pos[:, None], c.rope_theta)
            k = rope(k, pos[:, None], c.rope_theta)
            new_k.append(k)
            new_v.append(v)
            o = tree_attention(q, self.prefix_k[l], self.prefix_v[l], self.suf_k[l], self.suf_v[l], k, v, par)
            X = X + self._linear(l, 3, o.reshape(n * T, -1), row_adapter)
            X = self._mlp(l, X, row_adapter)
        out = {}
        if c.vocab > 0:
            logits = self._logits(X)
            out["logits"] = logits
            out["argmax"] = np.argmax(logits, axis=1).astype(np.int32).reshape(n, T)
            walk_on = out["argmax"] if follow_argmax is None else np.asarray(follow_argmax).reshape(n, T)
            toks = np.asarray(tree_tokens).reshape(n, T)
            acc_len = np.zeros(n, dtype=np.int32)
            acc_idx = np.full((n, T), -1, dtype=np.int32)
            nxt = np.zeros(n, dtype=np.int32)
            for s in range(n):
                path, bonus = accept_walk(toks[s], par[s], walk_on[s])
                acc_len[s], nxt[s] = len(path), bonus
                acc_idx[s, :len(path)] = path
            out.update(accept_len=acc_len, accept_idx=acc_idx, next=nxt)
        else:
            # hidden-state I/O: no logits to verify against, only the root row is kept
            out["hidden"] = X
            acc_len = np.ones(n, dtype=np.int32)
            acc_idx = np.full((n, T), -1, dtype=np.int32)
            acc_idx[:, 0] = 0
            out.update(accept_len=acc_len, accept_idx=acc_idx)
        out["tree_k"], out["tree_v"] = new_k, new_v
        if commit:
            # KV of the accepted rows joins the stream's own segment, in path order
            for l in range(c.n_layers):
                for s in range(n):
                    rows = [s * T + int(u) for u in acc_idx[s, :acc_len[s]]]
                    self.suf_k[l][s] = np.concatenate([self.suf_k[l][s], new_k[l][rows]], axis=0)
                    self.suf_v[l][s] = np.concatenate([self.suf_v[l][s], new_v[l][rows]], axis=0)
        return out

    def ds2d_round(self, adapter_idx, template, tree_tokens, follow_argmax=None):
        """One DS2D inference step (Sec. 3.5 steps 1-2, App. A.2): the pass verifies the draft tree in `tree_tokens`
        AND, from the forecast rows chained under every token node, drafts the next tree.

        template: row layout of one stream (parent, level, rank, forecast_of, widths; every stream uses the same).
        tree_tokens [n][R]: token ids at the token nodes, vocab + j - 1 at forecast rows j.
        After the accept walk, the drafts hang off the LAST ACCEPTED node: the next tree's nodes of depth d all carry,
        by sibling rank, the widths[d-1] most probable ids of that node's forecast row d (ties by rising id); the next
        root is the bonus token.  Returns verify_tree's dict plus next_tree_tokens [n][R] and drafts [n][m][max width]."""
        n = len(adapter_idx)
        R, m, V = len(template["parent"]), len(template["widths"]), self.cfg.vocab
        tree_tokens = np.asarray(tree_tokens).reshape(n, R)
        out = self.verify_tree(adapter_idx, np.stack([template["parent"]] * n), tree_tokens, follow_argmax=follow_argmax)
        wmax = int(max(template["widths"]))
        drafts = np.full((n, m, wmax), -1, dtype=np.int32)
        nxt = np.empty((n, R), dtype=np.int32)
        for s in range(n):
            leaf = int(out["accept_idx"][s][out["accept_len"][s] - 1])
            for j in range(1, m + 1):
                row = s * R + int(template["forecast_of"][leaf]) + (j - 1)
                w = int(template["widths"][j - 1])
                drafts[s, j - 1, :w] = first_tokens(out["logits"][row], w)
            for i in range(R):
                lv = int(template["level"][i])
                if lv == 0:
                    nxt[s, i] = out["next"][s]
                elif lv > 0:
                    nxt[s, i] = drafts[s, lv - 1, int(template["rank"][i])]
                else:
                    nxt[s, i] = V + (-lv) - 1
        out["next_tree_tokens"], out["drafts"] = nxt, drafts
        return out

    def generate(self, adapter_idx, first, k_steps):
        """k greedy decode steps, every stream fed its own previous token (App. A.1: the n-fold generative model run
        step after step).  Returns (tokens [k][n]: row j = produced by step j, logits [k][n][vocab])."""
        toks, out, lg = np.asarray(first, dtype=np.int32), [], []
        for _ in range(k_steps):
            r = self.decode_step(adapter_idx, tokens=toks)
            toks = np.asarray(r["next"], dtype=np.int32)
            out.append(toks)
            lg.append(r["logits"])
        return np.stack(out), np.stack(lg)

    def decode_step(self, adapter_idx, tokens=None, hidden=None, follow_argmax=None):
        """One token per stream: a verify pass whose tree is the root alone."""
        n = len(adapter_idx)
        par = np.full((n, 1), -1, dtype=np.int32)
        tt = None if tokens is None else np.asarray(tokens).reshape(n, 1)
        return self.verify_tree(adapter_idx, par, tt, hidden, follow_argmax)
