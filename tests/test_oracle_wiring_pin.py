"""Pins the WIRING of the oracle's decoder block (Sec. 3.1 with the LoRA term of Eq. 1-4) to a brute-force
computation: one decoder layer of a toy model is evaluated here with scalar Python loops written straight from
the definitions -- pre-norm, q/k/v projections, RoPE on q and k, softmax attention over the shared position and the
stream's own row, residual after the o projection, second pre-norm, silu(gate)*up, down projection, residual,
final norm, logits -- with no call into oracle/ and no matrix routine, and compared with OracleModel.

The self-consistency invariants elsewhere (stream isolation, B = 0, merged weights, root paths) hold for ANY
layer function; this test is the one that fails when gate and up are swapped, a residual is dropped, a norm is
moved behind its projection or the final norm is skipped -- each of which is planted below, on the CPU, to show it."""
import math

import numpy as np
import pytest

import gen
from oracle import ref

# toy shapes, all distinct so that a transposed operand cannot go unnoticed
D, HD, F, V, R = 4, 2, 6, 8, 1          # d_model, head_dim (one q head, one kv head), d_ffn, vocab, LoRA rank
EPS, THETA, ALPHA = 1e-5, 1e4, 2.0
CFG = gen.ModelCfg("pin", 1, D, 1, 1, HD, F, V, 1, R, 127, 1, 1, 1, alpha=ALPHA, rope_theta=THETA, rms_eps=EPS)
SHAPES = {"q": (D, HD), "k": (D, HD), "v": (D, HD), "o": (HD, D), "gate": (D, F), "up": (D, F), "down": (F, D),
          "lm_head": (D, V)}


def toy_inputs(seed=0):
    """Integer INT4 values with power-of-two fp16 scales (so q * scale is exact), packed in the canonical format:
    byte [k][n/2] = (q[k][2j] + 8) | (q[k][2j+1] + 8) << 4, one scale per element (group size 1)."""
    rng = np.random.default_rng(seed)
    dense, qweight, scales = {}, [], []
    for name in list(ref.PROJ) + ["lm_head"]:
        K, N = SHAPES[name]
        q = rng.integers(-8, 8, size=(K, N))
        s = 2.0 ** rng.integers(-4, -1, size=(K, N))
        dense[name] = [[float(q[k, n] * s[k, n]) for n in range(N)] for k in range(K)]
        u = (q + 8).astype(np.uint8)
        qweight.append((u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8))
        scales.append(s.astype(np.float16))
    gains = {g: [float(x) for x in 1.0 + 0.25 * rng.standard_normal(D)] for g in ("attn", "ffn", "final")}
    embed = rng.standard_normal((V, D)).astype(np.float16)
    A = {p: (0.5 * rng.standard_normal((R, SHAPES[p][0]))).astype(np.float16) for p in ref.PROJ}
    B = {p: (0.5 * rng.standard_normal((R, SHAPES[p][1]))).astype(np.float16) for p in ref.PROJ}
    return dense, qweight, scales, gains, embed, A, B


# ----------------------------------------------------------------------------- the definitions, as scalar loops
def b_rmsnorm(x, gain):
    ms = sum(v * v for v in x) / len(x)
    return [v / math.sqrt(ms + EPS) * g for v, g in zip(x, gain)]


def b_project(x, W, A=None, B=None):
    """y_n = sum_k x_k W[k][n]  +  (alpha / r) * sum_j (sum_k x_k A[j][k]) B[j][n]      (Eq. 1-4, row-vector form)"""
    K, N = len(W), len(W[0])
    y = [sum(x[k] * W[k][n] for k in range(K)) for n in range(N)]
    if A is not None:
        t = [sum(x[k] * float(A[j][k]) for k in range(K)) for j in range(R)]
        for n in range(N):
            y[n] += (ALPHA / R) * sum(t[j] * float(B[j][n]) for j in range(R))
    return y


def b_rope(x, pos):
    """pairs (i, i + hd/2), angle pos * theta^(-2i/hd)"""
    half = len(x) // 2
    out = list(x)
    for i in range(half):
        ang = pos * THETA ** (-2.0 * i / len(x))
        out[i] = x[i] * math.cos(ang) - x[i + half] * math.sin(ang)
        out[i + half] = x[i + half] * math.cos(ang) + x[i] * math.sin(ang)
    return out


def b_block(x, dense, gains, pos, keys, vals, A=None, B=None):
    """One decoder layer for one row at position `pos`; keys/vals: the cached rows it may see.  Returns the new
    residual row and the row's own k and v."""
    lo = (lambda p: (A[p], B[p])) if A is not None else (lambda p: (None, None))
    h = b_rmsnorm(x, gains["attn"])
    q = b_rope(b_project(h, dense["q"], *lo("q")), pos)
    k = b_rope(b_project(h, dense["k"], *lo("k")), pos)
    v = b_project(h, dense["v"], *lo("v"))
    ks, vs = keys + [k], vals + [v]
    sc = [sum(q[i] * kk[i] for i in range(HD)) / math.sqrt(HD) for kk in ks]
    mx = max(sc)
    w = [math.exp(s - mx) for s in sc]
    o = [sum(w[j] * vs[j][i] for j in range(len(ks))) / sum(w) for i in range(HD)]
    x = [xi + yi for xi, yi in zip(x, b_project(o, dense["o"], *lo("o")))]
    h2 = b_rmsnorm(x, gains["ffn"])
    g = b_project(h2, dense["gate"], *lo("gate"))
    u = b_project(h2, dense["up"], *lo("up"))
    act = [gi / (1.0 + math.exp(-gi)) * ui for gi, ui in zip(g, u)]
    x = [xi + yi for xi, yi in zip(x, b_project(act, dense["down"], *lo("down")))]
    return x, k, v


def brute_force_logits(dense, gains, embed, A, B, prompt_tok, tok):
    """Shared prefill of one position with the base weights, then one decode row with the adapter."""
    x0 = [float(v) for v in embed[prompt_tok]]
    _, k0, v0 = b_block(x0, dense, gains, 0, [], [])
    x1 = [float(v) for v in embed[tok]]
    x1, _, _ = b_block(x1, dense, gains, 1, [k0], [v0], A, B)
    h = b_rmsnorm(x1, gains["final"])
    return b_project(h, dense["lm_head"])


def oracle_logits(cls, qweight, scales, gains, embed, A, B, prompt_tok, tok):
    g = {k: np.array(v) for k, v in gains.items()}
    orc = cls(CFG, qweight, scales, [g["attn"]], [g["ffn"]], g["final"], embed)
    orc.set_adapter(0, [A[p] for p in ref.PROJ], [B[p] for p in ref.PROJ], ALPHA)
    orc.prefill_shared(np.array([prompt_tok]), n_streams=1)
    return orc.decode_step([0], tokens=np.array([tok]))["logits"][0]


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_block_wiring_matches_scalar_loops(seed):
    dense, qweight, scales, gains, embed, A, B = toy_inputs(seed)
    want = np.array(brute_force_logits(dense, gains, embed, A, B, 3, 5))
    got = oracle_logits(ref.OracleModel, qweight, scales, gains, embed, A, B, 3, 5)
    assert np.abs(want).max() > 1e-2
    np.testing.assert_allclose(got, want, rtol=1e-9, atol=1e-11)


# ----------------------------------------------------------------------------- planted mistakes must be caught
class SwappedGateUp(ref.OracleModel):
    def _mlp(self, l, X, row_adapter):
        h2 = ref.rmsnorm(X, self.rms_ffn[l], self.cfg.rms_eps)
        act = ref.silu(self._linear(l, 5, h2, row_adapter)) * self._linear(l, 4, h2, row_adapter)
        return X + self._linear(l, 6, act, row_adapter)


class NoMlpResidual(ref.OracleModel):
    def _mlp(self, l, X, row_adapter):
        return super()._mlp(l, X, row_adapter) - X


class NormAfterProjection(ref.OracleModel):
    def _mlp(self, l, X, row_adapter):
        g = ref.rmsnorm(self._linear(l, 4, X, row_adapter), np.ones(F), self.cfg.rms_eps)
        u = ref.rmsnorm(self._linear(l, 5, X, row_adapter), np.ones(F), self.cfg.rms_eps)
        return X + self._linear(l, 6, ref.silu(g) * u, row_adapter)


class NoFinalNorm(ref.OracleModel):
    def _logits(self, X):
        return X @ self.W(self.cfg.n_layers * 7)


class NoAttentionResidual(ref.OracleModel):
    def _linear(self, l, p, h, row_adapter):
        y = super()._linear(l, p, h, row_adapter)
        return y * 0.0 if p == 3 else y                          # the o projection contributes nothing


@pytest.mark.parametrize("broken", [SwappedGateUp, NoMlpResidual, NormAfterProjection, NoFinalNorm, NoAttentionResidual])
def test_planted_wiring_mistakes_fail_the_pin(broken):
    dense, qweight, scales, gains, embed, A, B = toy_inputs(0)
    want = np.array(brute_force_logits(dense, gains, embed, A, B, 3, 5))
    got = oracle_logits(broken, qweight, scales, gains, embed, A, B, 3, 5)
    assert not np.allclose(got, want, rtol=1e-6, atol=1e-8)


def test_brute_force_depends_on_every_piece():
    """The scalar reference itself reacts to each ingredient (a reference that ignored one could not pin it)."""
    dense, qweight, scales, gains, embed, A, B = toy_inputs(0)
    base = np.array(brute_force_logits(dense, gains, embed, A, B, 3, 5))
    for p in ref.PROJ:                                            # every adapter matters
        B2 = dict(B)
        B2[p] = np.zeros_like(B[p])
        assert not np.allclose(np.array(brute_force_logits(dense, gains, embed, A, B2, 3, 5)), base, rtol=1e-9)
    for g in ("attn", "ffn", "final"):                            # every gain matters
        g2 = dict(gains)
        g2[g] = [1.0] * D
        assert not np.allclose(np.array(brute_force_logits(dense, g2, embed, A, B, 3, 5)), base, rtol=1e-9)
    # the shared position matters (attention really mixes two rows)
    assert not np.allclose(np.array(brute_force_logits(dense, gains, embed, A, B, 4, 5)), base, rtol=1e-9)
