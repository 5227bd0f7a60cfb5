"""Pins for the CPU oracle: every check compares it with something other than itself --
values the paper prints, closed forms, library routines, brute force, or invariants that a
dropped term, wrong sign/index or transposed operand would break."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

import gen
from oracle import ref

TINY = gen.ModelCfg("tiny", 2, 64, 4, 2, 16, 96, 102, 32, 4, 127, 3, 3, 9)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def tiny_oracle(cfg=TINY, seed=1, n_adapters=None, b_std=0.05):
    m = gen.make_model(cfg, seed)
    o = ref.OracleModel.from_synth(m)
    for a in range(cfg.n_adapters if n_adapters is None else n_adapters):
        A, B = gen.make_adapter(cfg, a, seed, b_std=b_std)
        o.set_adapter(a, A, B, cfg.alpha)
    return m, o


# ------------------------------------------------------------------ INT4 unpack / dequant
def _fp16_rne(fr: Fraction) -> float:
    """Round an exact rational to IEEE binary16, ties to even, by integer arithmetic only."""
    if fr == 0:
        return 0.0
    sign = -1 if fr < 0 else 1
    a = abs(fr)
    e = 0
    while a >= 2:
        a /= 2
        e += 1
    while a < 1:
        a *= 2
        e -= 1
    e = max(e, -14)                      # subnormals share the exponent of the smallest normal
    ulp = Fraction(2) ** (e - 10)
    n = abs(fr) / ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    val = lo * ulp
    if val >= Fraction(65520):
        return sign * float("inf")
    return sign * float(val)


def test_unpack_hand_decoded_bytes():
    # byte 0x1F: low nibble 0xF -> q = 7 in the even column, high nibble 0x1 -> q = -7 in the odd one
    qb = np.array([[0x1F, 0x80], [0x08, 0xF0]], dtype=np.uint8)
    q = ref.unpack_int4(qb)
    assert q.tolist() == [[7, -7, -8, 0], [0, -8, -8, 7]]


def test_dequant_is_single_fp16_rounding():
    rng = np.random.default_rng(0)
    bits = np.concatenate([rng.integers(0, 0x7C00, 300), [0x0001, 0x03FF, 0x0400, 0x7BFF, 0x3C00, 0x3555]]).astype(np.uint16)
    scales = bits.view(np.float16)
    for sc in scales:
        for u in range(16):
            qb = np.array([[u | (u << 4)]], dtype=np.uint8)
            got = ref.dequant(qb, np.array([[sc, sc]], dtype=np.float16), 1)[0, 0]
            want = _fp16_rne(Fraction(u - 8) * Fraction(float(sc)))
            assert float(got) == want, (u, sc)


def test_dequant_group_and_column_indexing():
    # scale[k // G][n]: distinct powers of two per (group, column) make any index slip visible
    K, N, G = 8, 4, 4
    u = (np.arange(K * N).reshape(K, N) % 16).astype(np.uint8)
    sc = np.array([[1, 2, 4, 8], [16, 32, 64, 128]], dtype=np.float16)
    w = ref.dequant(gen.pack_nibbles(u), sc, G)
    for k in range(K):
        for n in range(N):
            assert w[k, n] == (int(u[k, n]) - 8) * float(sc[k // G, n])


def test_quantise_roundtrip_error_bound():
    rng = np.random.default_rng(3)
    w = rng.standard_normal((256, 32)).astype(np.float32) * 0.02
    qb, sc = gen.quantize_int4(w, 64)
    wd = ref.dequant(qb, sc, 64).astype(np.float64)
    s = np.repeat(sc.astype(np.float64), 64, axis=0)
    # |w - q*s| <= s/2 (rounding) + clipping slack from the fp16-rounded scale + fp16 rounding of q*s
    assert np.all(np.abs(w - wd) <= 0.5 * s * (1 + 2 ** -9) + np.abs(wd) * 2 ** -11 + 1e-12)


# ------------------------------------------------------------------ projections (Eq. 1-4)
def test_base_projection_is_matmul():
    rng = np.random.default_rng(1)
    W = rng.standard_normal((48, 20))
    h = rng.standard_normal((5, 48))
    A = [rng.standard_normal((4, 48))]
    B = [np.zeros((4, 20))]
    assert np.allclose(ref.linear_lora(h, W, [0] * 5, A, B, [4.0]), np.matmul(h, W), rtol=0, atol=1e-12)
    assert np.array_equal(ref.linear_lora(h, W, [-1] * 5, A, [np.ones((4, 20))], [4.0]), np.matmul(h, W))


def test_runtime_lora_equals_merged_and_onehot_masked():
    rng = np.random.default_rng(2)
    K, N, r, n_ad = 40, 24, 4, 3
    W = rng.standard_normal((K, N))
    h = rng.standard_normal((6, K))
    A = [rng.standard_normal((r, K)) for _ in range(n_ad)]
    B = [rng.standard_normal((r, N)) for _ in range(n_ad)]
    s = [16.0 / r, 0.5, 2.0]
    rows = [2, 0, 1, 1, -1, 2]
    y = ref.linear_lora(h, W, rows, A, B, s)
    for m, a in enumerate(rows):
        merged = W if a < 0 else W + s[a] * (A[a].T @ B[a])          # Y = X (W + s A B)
        assert np.allclose(y[m], h[m] @ merged, atol=1e-10)
        onehot = np.zeros(n_ad)
        if a >= 0:
            onehot[a] = 1.0
        masked = h[m] @ W + sum(onehot[i] * s[i] * (h[m] @ A[i].T) @ B[i] for i in range(n_ad))
        assert np.allclose(y[m], masked, atol=1e-10)                   # Sec. 3.2 approach (b)


def test_rank1_lora_closed_form():
    rng = np.random.default_rng(4)
    K, N = 16, 10
    h = rng.standard_normal((1, K))
    a, b = rng.standard_normal((1, K)), rng.standard_normal((1, N))
    y = ref.linear_lora(h, np.zeros((K, N)), [0], [a], [b], [3.0])
    assert np.allclose(y[0], 3.0 * float(h[0] @ a[0]) * b[0], atol=1e-12)


# ------------------------------------------------------------------ elementwise closed forms
def test_rope_closed_forms():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((3, 16))
    assert np.allclose(ref.rope(x, np.zeros(3, dtype=int), 1e4), x)
    y = ref.rope(x, np.array([7, 8, 9]), 1e4)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))
    q, k = rng.standard_normal(16), rng.standard_normal(16)
    d1 = ref.rope(q, 12, 1e4) @ ref.rope(k, 5, 1e4)
    d2 = ref.rope(q, 107, 1e4) @ ref.rope(k, 100, 1e4)
    assert np.isclose(d1, d2)
    # a 2-d head is one plane rotating by the position itself (theta^0 = 1): (1,0) -> (cos p, sin p)
    assert np.allclose(ref.rope(np.array([1.0, 0.0]), 3, 1e4), [np.cos(3.0), np.sin(3.0)])
    # pairing is (i, i + hd/2): with hd = 4 elements 0 and 2 form the first plane
    e0 = ref.rope(np.array([1.0, 0, 0, 0]), 2, 1e4)
    assert np.allclose(e0, [np.cos(2.0), 0, np.sin(2.0), 0])
    # second plane turns at theta^(-2/4) = 1/100 of the rate
    e1 = ref.rope(np.array([0, 1.0, 0, 0]), 50, 1e4)
    assert np.allclose(e1, [0, np.cos(0.5), 0, np.sin(0.5)])


def test_rmsnorm_and_silu_closed_forms():
    g = np.array([1.0, 2.0, -1.0, 0.5])
    assert np.allclose(ref.rmsnorm(np.full(4, -3.0), g, 0.0), -g)
    assert np.allclose(ref.rmsnorm(np.array([3.0, 4.0, 0.0, 0.0]), np.ones(4), 0.0), np.array([3, 4, 0, 0]) / 2.5)
    assert np.isclose(ref.rmsnorm(np.array([2.0]), np.ones(1), 5.0)[0], 2.0 / 3.0)    # eps inside the root
    x = np.linspace(-4, 4, 9)
    assert ref.silu(np.array([0.0]))[0] == 0.0
    assert np.allclose(ref.silu(x) - ref.silu(-x), x)
    assert np.isclose(ref.silu(np.array([1.0]))[0], 1.0 / (1.0 + np.exp(-1.0)))


# ------------------------------------------------------------------ attention
def test_attend_uniform_scores_give_mean_of_values():
    rng = np.random.default_rng(6)
    keys = np.repeat(rng.standard_normal((1, 2, 8)), 5, axis=0)
    vals = rng.standard_normal((5, 2, 8))
    q = rng.standard_normal((4, 8))
    out = ref.attend(q, keys, vals)
    for j in range(4):
        assert np.allclose(out[j], vals[:, j // 2, :].mean(axis=0))


def test_attend_matches_textbook_two_keys():
    # one head, two keys: weights are a logistic function of the scaled score gap
    q = np.array([[2.0, 0.0, 0.0, 0.0]])
    keys = np.array([[[1.0, 0, 0, 0]], [[0.0, 0, 0, 0]]])
    vals = np.array([[[1.0, 0, 0, 0]], [[0.0, 1, 0, 0]]])
    w0 = 1.0 / (1.0 + np.exp(-(2.0 / np.sqrt(4))))
    assert np.allclose(ref.attend(q, keys, vals)[0], [w0, 1 - w0, 0, 0])


def test_gqa_head_mapping():
    # query head j reads kv head j // group: make kv heads carry distinct constant values
    keys = np.zeros((3, 2, 4))
    vals = np.zeros((3, 2, 4))
    vals[:, 0, :] = 1.0
    vals[:, 1, :] = 2.0
    out = ref.attend(np.ones((4, 4)), keys, vals)
    assert np.allclose(out[:2], 1.0) and np.allclose(out[2:], 2.0)


def test_shared_prefix_decode_equals_causal_over_concatenation():
    """Prefill of P tokens then one base-weight decode step == last row of a (P+1)-token prefill."""
    m, o = tiny_oracle()
    ids = gen.make_prompt_ids(TINY, 0, 10)
    full = o.prefill_shared(ids)                       # logits after 10 tokens
    o.prefill_shared(ids[:9], n_streams=1)
    step = o.decode_step([-1], tokens=ids[9:10])
    assert np.allclose(step["logits"][0], full, atol=1e-9)
    # and the appended suffix KV is the KV that the longer prefill stored at position 9
    o2 = tiny_oracle()[1]
    o2.prefill_shared(ids)
    for l in range(TINY.n_layers):
        assert np.allclose(o.suf_k[l][0][0], o2.prefix_k[l][9], atol=1e-10)
        assert np.allclose(o.suf_v[l][0][0], o2.prefix_v[l][9], atol=1e-10)


def test_stream_isolation():
    """Stream i of an n-stream run equals a single-stream run with adapter i alone (App. A.1)."""
    m, o = tiny_oracle()
    ids = gen.make_prompt_ids(TINY, 0)
    o.prefill_shared(ids, n_streams=3)
    toks = np.array([[5, 17, 60], [33, 2, 8]])
    multi = [o.decode_step([0, 1, 2], tokens=toks[i]) for i in range(2)]
    for s in range(3):
        o1 = tiny_oracle()[1]
        o1.prefill_shared(ids, n_streams=1)
        for i in range(2):
            single = o1.decode_step([s], tokens=toks[i, s:s + 1])
            assert np.allclose(single["logits"][0], multi[i]["logits"][s], atol=1e-9)
    # adapters matter: the streams do differ from one another on identical tokens
    o.prefill_shared(ids, n_streams=3)
    same = o.decode_step([0, 1, 2], tokens=[5, 5, 5])["logits"]
    assert np.abs(same[0] - same[1]).max() > 1e-4


def test_zero_B_reproduces_base_model():
    m, o = tiny_oracle(b_std=0.0)
    ids = gen.make_prompt_ids(TINY, 0)
    o.prefill_shared(ids, n_streams=2)
    r = o.decode_step([0, -1], tokens=[7, 7])
    assert np.allclose(r["logits"][0], r["logits"][1], atol=1e-12)


def test_model_lora_equals_merged_weights():
    """The run-time adapter path equals a model whose dense weights are W + s A^T B."""
    m, o = tiny_oracle()
    ids = gen.make_prompt_ids(TINY, 0)
    o.prefill_shared(ids, n_streams=1)
    r = o.decode_step([1], tokens=[11])
    o2 = tiny_oracle(n_adapters=0)[1]
    o2.prefill_shared(ids, n_streams=1)                       # prefix is base-weight in both
    A, B = gen.make_adapter(TINY, 1, 1, b_std=0.05)
    s = TINY.alpha / TINY.lora_rank
    for idx in range(TINY.n_layers * 7):
        o2._W[idx] = o2.W(idx) + s * (A[idx].astype(np.float64).T @ B[idx].astype(np.float64))
    r2 = o2.decode_step([-1], tokens=[11])
    assert np.allclose(r["logits"], r2["logits"], atol=1e-9)


def test_every_root_path_of_a_tree_equals_sequential_decode():
    m, o = tiny_oracle()
    ids = gen.make_prompt_ids(TINY, 0)
    parent = gen.build_tree((2, 2, 1))
    T = len(parent)
    rng = np.random.default_rng(8)
    toks = rng.integers(0, TINY.vocab, size=(2, T))
    o.prefill_shared(ids, n_streams=2)
    o.decode_step([0, 2], tokens=[3, 4])                      # non-empty suffixes
    tree = o.verify_tree([0, 2], np.stack([parent, parent]), toks, commit=False)
    for s, a in enumerate([0, 2]):
        for t in range(T):
            path = ref.ancestors_and_self(parent, t)
            o1 = tiny_oracle()[1]
            o1.prefill_shared(ids, n_streams=1)
            o1.decode_step([a], tokens=[[3, 4][s]])
            for u in path:
                last = o1.decode_step([a], tokens=[toks[s, u]])
            assert np.allclose(last["logits"][0], tree["logits"][s * T + t], atol=1e-9), (s, t)


# ------------------------------------------------------------------ DS2D trees and acceptance (Sec. 3.5)
def _golden_rows():
    for line in open(os.path.join(GOLD, "ds2d_tree_counts.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        yield tuple(int(b) for b in f[0].split(",")), int(f[1]), int(f[2]), int(f[3]), int(f[4])


def test_tree_generator_matches_paper_counts():
    for branch, drafts, tokens, mfe, rows in _golden_rows():
        parent = gen.build_tree(branch)
        ref.check_parents(parent)
        assert len(parent) == tokens and len(parent) - 1 == drafts
        assert mfe == len(branch) and tokens * (1 + mfe) == rows and rows <= 32
        d = ref.depths(parent)
        for j, b in enumerate(branch):                         # every depth-j node has b_{j+1} children
            for node in [i for i in range(tokens) if d[i] == j]:
                assert sum(1 for p in parent if p == node) == b
    p = gen.build_tree((4, 2, 2), 16)
    assert np.bincount(gen.tree_depths(p)).tolist() == [1, 4, 8, 3]
    p = gen.build_tree((4, 4, 2), 32)
    assert np.bincount(gen.tree_depths(p)).tolist() == [1, 4, 16, 11]


def test_accept_walk_paper_example_shape():
    # the paper's "1-3-5": root (token 1) -> one depth-1 draft -> one depth-2 draft accepted
    parent = gen.build_tree((3, 2))
    tokens = [1, 2, 3, 4, 9, 9, 5, 6, 9, 9]                    # node 2 carries 3; its children 6,7 carry 5,6
    argmax = [3, 0, 5, 0, 0, 0, 8, 0, 0, 0]
    path, bonus = ref.accept_walk(tokens, parent, argmax)
    assert [tokens[i] for i in path] == [1, 3, 5] and path == [0, 2, 6] and bonus == 8


def _brute_force_accept(tokens, parent, argmax):
    """Longest root path valid under the first-match rule, by enumerating every root path."""
    best = [0]
    n = len(parent)
    for t in range(n):
        path = ref.ancestors_and_self(parent, t)
        ok = True
        for a, b in zip(path[:-1], path[1:]):
            if tokens[b] != argmax[a]:
                ok = False
                break
            if any(parent[u] == a and tokens[u] == argmax[a] for u in range(b)):   # an earlier sibling matches
                ok = False
                break
        if ok and len(path) > len(best):
            best = path
    return best, argmax[best[-1]]


def test_accept_walk_brute_force_small_trees():
    count = 0
    for n in range(1, 6):
        for parent in itertools.product(*[range(i) for i in range(1, n)]):
            parent = [-1] + list(parent)
            for toks in itertools.product(range(3), repeat=n - 1):
                tokens = [0] + list(toks)
                for argmax in itertools.product(range(3), repeat=n):
                    got = ref.accept_walk(tokens, parent, argmax)
                    want = _brute_force_accept(tokens, parent, list(argmax))
                    assert (got[0], got[1]) == (want[0], want[1])
                    count += 1
    assert count > 400000


def test_accept_walk_rejects_bad_parents():
    with pytest.raises(ValueError):
        ref.accept_walk([0, 1], [-1, 1], [0, 0])
    with pytest.raises(ValueError):
        ref.accept_walk([0, 1], [0, 0], [0, 0])


def _greedy(o, ids, adapters, first, steps):
    o.prefill_shared(ids, n_streams=len(adapters))
    out, cur = [], np.array(first)
    for _ in range(steps):
        cur = o.decode_step(adapters, tokens=cur)["next"]
        out.append(cur.copy())
    return np.array(out).T                                      # [stream][step]


def test_ds2d_tokens_equal_plain_greedy_decode():
    """Lossless speculation (Sec. 3.5): emitted tokens are those of plain greedy decoding, both
    with random drafts (nothing accepted) and with drafts that contain the true continuation."""
    m, o = tiny_oracle()
    ids = gen.make_prompt_ids(TINY, 0)
    adapters, first, steps = [0, 1, 2], [4, 9, 4], 12
    plain = _greedy(o, ids, adapters, first, steps)
    parent = gen.build_tree((2, 2), 6)
    rng = np.random.default_rng(9)
    for planted in (False, True):
        o.prefill_shared(ids, n_streams=3)
        emitted = [[] for _ in adapters]
        last = list(first)
        tokens_per_round = []
        while min(len(e) for e in emitted) < steps:
            toks = rng.integers(0, TINY.vocab, size=(3, len(parent)))
            toks[:, 0] = last
            if planted:
                for s in range(3):
                    # plant the true continuation on the last child at each level so that the
                    # first-match rule has to skip non-matching earlier siblings
                    done = len(emitted[s])
                    if done + 2 <= steps:
                        toks[s, 2] = plain[s, done]
                        toks[s, 5] = 0 if done + 1 >= steps else plain[s, done + 1]   # child of node 2
            r = o.verify_tree(adapters, np.stack([parent] * 3), toks)
            for s in range(3):
                L = int(r["accept_len"][s])
                acc = [int(toks[s, i]) for i in r["accept_idx"][s, 1:L]] + [int(r["next"][s])]
                emitted[s].extend(acc)
                last[s] = acc[-1]
                tokens_per_round.append(L)
        for s in range(3):
            assert emitted[s][:steps] == plain[s].tolist()[:steps]
        if planted:
            assert max(tokens_per_round) >= 2                   # the speculative branch was exercised
