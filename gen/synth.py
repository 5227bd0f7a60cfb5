"""Seeded draws, the INT4 group quantiser and draft-tree shapes.

Every tensor has its own counter-style seed ``[seed, layer, projection, kind]`` so a
tensor can be regenerated alone and the draw order never matters.

Canonical weight interchange format (what the C-ABI takes and what the oracle unpacks):
  * nibble ``u = q + 8`` with ``q`` in [-8, 7];
  * byte ``b[k][j]`` holds output column ``2j`` in its low nibble and ``2j+1`` in its high nibble,
    rows ``k`` (input features) major: uint8 ``[K][N/2]``;
  * scales fp16 ``[K/G][N]``, one per group of ``G`` consecutive input features per column.
"""
from dataclasses import dataclass, field
import numpy as np

from .configs import ModelCfg, PROJ_NAMES, PROJ_BITS, proj_shape

_KIND = {"w": 0, "A": 1, "B": 2, "rms_attn": 3, "rms_ffn": 4, "rms_final": 5, "embed": 6,
         "prompt": 7, "hidden": 8, "cand": 9, "forecast": 10}
_LM_HEAD = 7  # projection index of lm_head in the per-model list (after the 7 per-layer ones)


def _rng(seed, layer, proj, kind, extra=0):
    return np.random.default_rng([int(seed), int(layer), int(proj), _KIND[kind], int(extra)])


def _normal(rng, shape, std):
    return rng.standard_normal(shape, dtype=np.float32) * np.float32(std)


def pack_nibbles(u: np.ndarray) -> np.ndarray:
    """uint8 [K][N] with values 0..15 -> uint8 [K][N/2], even column in the low nibble."""
    assert u.dtype == np.uint8 and u.shape[1] % 2 == 0
    return (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)


def quantize_int4(w: np.ndarray, group: int):
    """Symmetric per-group INT4 quantiser (input preparation).

    scale = fp16(max|w| over the group / 7), replaced by 1 where that is 0;
    q = clip(round_half_even(w / scale), -8, 7).  Returns (packed uint8 [K][N/2], fp16 [K/G][N]).
    """
    K, N = w.shape
    assert K % group == 0
    wg = w.reshape(K // group, group, N).astype(np.float32)
    amax = np.abs(wg).max(axis=1)
    scale = (amax / np.float32(7.0)).astype(np.float16)
    scale = np.where(scale == 0, np.float16(1.0), scale).astype(np.float16)
    q = np.rint(wg / scale.astype(np.float32)[:, None, :])
    q = np.clip(q, -8, 7).astype(np.int8).reshape(K, N)
    return pack_nibbles((q + 8).astype(np.uint8)), scale


def quantize_int4_per_channel(w: np.ndarray):
    """Symmetric per-output-channel INT4 quantiser (input preparation for the INT4 x INT8 regime of Sec. 3.3).

    w [K][N]; scale[n] = fp16(max_k |w[k][n]| / 7) (1 where that is 0); q = clip(round_half_even(w / scale), -8, 7).
    Returns (packed uint8 [N][K/2]: channel-major, nibble q + 8, even k in the low nibble; fp16 [N])."""
    K, N = w.shape
    assert K % 2 == 0
    w = w.astype(np.float32)
    scale = (np.abs(w).max(axis=0) / np.float32(7.0)).astype(np.float16)
    scale = np.where(scale == 0, np.float16(1.0), scale).astype(np.float16)
    q = np.clip(np.rint(w / scale.astype(np.float32)[None, :]), -8, 7).astype(np.int8)
    return pack_nibbles(np.ascontiguousarray((q + 8).astype(np.uint8).T)), scale


@dataclass
class SynthModel:
    cfg: ModelCfg
    seed: int
    qweight: list = field(default_factory=list)   # [n_layers*7 (+1 lm_head)] uint8 [K][N/2]
    scales: list = field(default_factory=list)    # same indexing, fp16 [K/G][N]
    rms_attn: list = field(default_factory=list)  # [n_layers] fp16 [d]
    rms_ffn: list = field(default_factory=list)
    rms_final: np.ndarray = None                  # fp16 [d] or None
    embed: np.ndarray = None                      # fp16 [vocab][d] or None


def make_model(cfg: ModelCfg, seed: int = 0) -> SynthModel:
    m = SynthModel(cfg, seed)
    for l in range(cfg.n_layers):
        for p, name in enumerate(PROJ_NAMES):
            K, N = proj_shape(cfg, name)
            w = _normal(_rng(seed, l, p, "w"), (K, N), cfg.w_std)
            qb, sc = quantize_int4(w, cfg.group_size)
            m.qweight.append(qb)
            m.scales.append(sc)
        # gains 1 + N(0, 0.02): a dropped gain must show up in parity
        m.rms_attn.append((1 + _normal(_rng(seed, l, 0, "rms_attn"), (cfg.d_model,), 0.02)).astype(np.float16))
        m.rms_ffn.append((1 + _normal(_rng(seed, l, 0, "rms_ffn"), (cfg.d_model,), 0.02)).astype(np.float16))
    if cfg.vocab > 0:
        K, N = proj_shape(cfg, "lm_head")
        w = _normal(_rng(seed, 0, _LM_HEAD, "w"), (K, N), cfg.w_std)
        qb, sc = quantize_int4(w, cfg.group_size)
        m.qweight.append(qb)
        m.scales.append(sc)
        m.rms_final = (1 + _normal(_rng(seed, 0, 0, "rms_final"), (cfg.d_model,), 0.02)).astype(np.float16)
        m.embed = _normal(_rng(seed, 0, 0, "embed"), (cfg.vocab, cfg.d_model), cfg.w_std).astype(np.float16)
    return m


def make_adapter(cfg: ModelCfg, slot: int, seed: int = 0, rank: int = None, targets: int = None,
                 b_std: float = None):
    """One adapter: lists A[l*7+p] fp16 [r][K_p], B[l*7+p] fp16 [r][N_p] (None where not targeted)."""
    r = cfg.lora_rank if rank is None else rank
    targets = cfg.lora_targets if targets is None else targets
    b_std = cfg.b_std if b_std is None else b_std
    A, B = [], []
    for l in range(cfg.n_layers):
        for p, name in enumerate(PROJ_NAMES):
            if not (targets & PROJ_BITS[name]):
                A.append(None)
                B.append(None)
                continue
            K, N = proj_shape(cfg, name)
            A.append(_normal(_rng(seed, l, p, "A", slot), (r, K), 1.0 / r).astype(np.float16))
            B.append(_normal(_rng(seed, l, p, "B", slot), (r, N), b_std).astype(np.float16))
    return A, B


def make_prompt_ids(cfg: ModelCfg, seed: int = 0, n: int = None) -> np.ndarray:
    n = cfg.prompt_len if n is None else n
    return _rng(seed, 0, 0, "prompt").integers(0, cfg.vocab, size=n, dtype=np.int32)


def make_hidden(cfg: ModelCfg, rows: int, seed: int = 0, which: int = 0) -> np.ndarray:
    """fp16 [rows][d_model] ~ N(0,1): prompt hidden states (which=0) or decode inputs (which>=1)."""
    return _normal(_rng(seed, 0, 0, "hidden", which), (rows, cfg.d_model), 1.0).astype(np.float16)


def build_tree(branch, n_nodes: int = None) -> np.ndarray:
    """parent[] of a draft tree from a branch configuration (b_1..b_m), root = node 0.

    Breadth-first: every node of depth j-1, in index order, receives b_j children.  With
    ``n_nodes`` given, children stop being added once that many nodes (root included) exist.
    (3,2) -> root + 3 + 6 = 10 nodes, i.e. 9 draft tokens.
    """
    parent = [-1]
    level = [0]
    for b in branch:
        nxt = []
        for node in level:
            for _ in range(b):
                if n_nodes is not None and len(parent) >= n_nodes:
                    break
                parent.append(node)
                nxt.append(len(parent) - 1)
        level = nxt
    if n_nodes is not None:
        assert len(parent) == n_nodes, "branch configuration gives fewer nodes than requested"
    return np.asarray(parent, dtype=np.int32)


def ds2d_template(branch, n_token_nodes: int = None) -> dict:
    """Row layout of one DS2D pass that verifies a draft tree AND drafts the next one (one stream's rows).

    Rows 0 .. T-1 are the tree's token nodes (build_tree order; node 0 = the last accepted token).  Every token node t
    is followed, further down, by its m = len(branch) forecast rows T + t*m + (j-1), j = 1..m, chained under it
    (forecast j sees node t's root path and forecasts 1..j of the same node).  Returns int32 arrays over the
    R = T * (1 + m) rows: parent; level (0 root, d >= 1 draft node of depth d, -j forecast row j); rank (a draft
    node's position among its parent's children); forecast_of (a token node's first forecast row, -1 otherwise);
    and widths[d-1] = children per node at depth d."""
    tok_parent = build_tree(branch, n_token_nodes)
    T, m = len(tok_parent), len(branch)
    R = T * (1 + m)
    parent = np.full(R, -1, dtype=np.int32)
    level = np.zeros(R, dtype=np.int32)
    rank = np.zeros(R, dtype=np.int32)
    forecast_of = np.full(R, -1, dtype=np.int32)
    parent[:T] = tok_parent
    depth = tree_depths(tok_parent)
    seen = {}
    for t in range(T):
        level[t] = depth[t]
        if t:
            rank[t] = seen.get(int(tok_parent[t]), 0)
            seen[int(tok_parent[t])] = rank[t] + 1
        forecast_of[t] = T + t * m
        for j in range(1, m + 1):
            r = T + t * m + (j - 1)
            parent[r] = t if j == 1 else r - 1
            level[r] = -j
    widths = np.array([max([rank[t] + 1 for t in range(T) if level[t] == d] or [0]) for d in range(1, m + 1)], dtype=np.int32)
    return dict(parent=parent, level=level, rank=rank, forecast_of=forecast_of, widths=widths, T=T, m=m, R=R)


def make_forecast(cfg: ModelCfg, m: int, seed: int = 0) -> np.ndarray:
    """m synthetic forecast embeddings fp16 [m][d_model] (stand-ins for the prefix-tuned ones: untrained, so the
    drafts they produce are rarely accepted; shapes and data flow are what they exercise)."""
    return _normal(_rng(seed, 0, 0, "forecast"), (m, cfg.d_model), 0.02).astype(np.float16)


def tree_depths(parent) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return d


def make_candidates(cfg: ModelCfg, rounds: int, n_streams: int, n_nodes: int, seed: int = 0) -> np.ndarray:
    """Uniform-random draft ids, int32 [rounds][n_streams][n_nodes-1] (node 0 is the last accepted token)."""
    return _rng(seed, 0, 0, "cand").integers(0, cfg.vocab, size=(rounds, n_streams, n_nodes - 1), dtype=np.int32)
