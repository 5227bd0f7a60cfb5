"""Pins for DS2D draft generation in the oracle (Sec. 3.5, inference steps 1-2; App. A.2): forecast rows chained under
every token node, the next tree drafted from the forecast rows of the last accepted node."""
import os

import numpy as np
import pytest

import gen
from oracle import ref

TINY = gen.ModelCfg("tinyds2d", 2, 64, 2, 1, 32, 96, 50, 32, 4, 127, 2, 2, 6, b_std=0.05)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ds2d_tree_counts.txt")


def golden_rows():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = [x.strip() for x in line.split("|")]
        yield tuple(int(b) for b in f[0].split(",")), int(f[1]), int(f[2]), int(f[3]), int(f[4])


def test_template_row_counts_match_the_printed_example_and_budget():
    """Sec. 3.5: (3,2) with m = 2 gives 9 drafts, 10 tokens with the previous one, 20 forecast rows, 30 input rows; every
    configuration of Table 7 stays within the 32-row budget."""
    for branch, drafts, tokens, m, rows in golden_rows():
        t = gen.ds2d_template(branch)
        assert (t["T"] - 1, t["T"], t["m"], t["R"]) == (drafts, tokens, m, rows)
        assert t["R"] <= 32 and int((t["level"] < 0).sum()) == tokens * m
        assert list(t["widths"]) == list(branch)


def test_template_structure_by_explicit_walks():
    t = gen.ds2d_template((3, 2))
    par, lev = t["parent"], t["level"]
    for i in range(t["R"]):
        assert par[i] < i
        if lev[i] < 0:                                   # forecast row j: j steps up the chain reach its token node
            j, u = -lev[i], i
            for _ in range(j):
                u = par[u]
            assert lev[u] >= 0 and t["forecast_of"][u] + j - 1 == i
    # draft nodes: depth by walking to the root; ranks count the siblings before a node
    for i in range(1, t["T"]):
        d, u = 0, i
        while u:
            u, d = par[u], d + 1
        assert d == lev[i]
        assert t["rank"][i] == sum(1 for k in range(i) if par[k] == par[i])


def fresh(n_streams, with_forecast=True, planted=None, m_forecast=2):
    m = gen.make_model(TINY, 0)
    orc = ref.OracleModel.from_synth(m)
    for a in range(TINY.n_adapters):
        A, B = gen.make_adapter(TINY, a, 0)
        orc.set_adapter(a, A, B, TINY.alpha)
    if with_forecast:
        orc.set_forecast(gen.make_forecast(TINY, m_forecast, 0))
    last = orc.prefill_shared(gen.make_prompt_ids(TINY, 0), n_streams=n_streams)
    if planted is not None:                               # the forecast vectors as ordinary embedding rows (after the
        orc.embed = orc.embed.copy()                      # prefill, whose prompt may use those ids)
        for tok, vec in planted.items():
            orc.embed[tok] = vec
    return orc, last


def test_forecast_rows_are_tree_rows_fed_with_the_forecast_vectors():
    """A forecast row behaves as a tree node whose input row is the forecast vector: planting the two vectors at two
    ordinary token ids and asking for those ids instead gives the same logits everywhere."""
    t = gen.ds2d_template((2, 1))
    fc = gen.make_forecast(TINY, 2, 0)
    rng = np.random.default_rng(0)
    tt = rng.integers(0, 40, size=(2, t["R"])).astype(np.int32)
    tt[:, t["level"] < 0] = (TINY.vocab - np.minimum(t["level"], 0) - 1)[t["level"] < 0]
    orc, _ = fresh(2)
    a = orc.verify_tree([0, -1], np.stack([t["parent"]] * 2), tt, commit=False)["logits"]
    planted = {48: fc[0], 49: fc[1]}
    tt2 = tt.copy()
    tt2[tt == TINY.vocab] = 48
    tt2[tt == TINY.vocab + 1] = 49
    orc2, _ = fresh(2, with_forecast=False, planted=planted)
    b = orc2.verify_tree([0, -1], np.stack([t["parent"]] * 2), tt2, commit=False)["logits"]
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-12)
    # and the token nodes' logits do not depend on the forecast rows at all (they only hang below)
    orc3, _ = fresh(2)
    c = orc3.verify_tree([0, -1], np.stack([t["parent"][:t["T"]]] * 2), tt[:, :t["T"]], commit=False)["logits"]
    np.testing.assert_allclose(a.reshape(2, t["R"], -1)[:, :t["T"]], c.reshape(2, t["T"], -1), rtol=1e-10, atol=1e-12)


def test_drafts_sit_where_the_definition_puts_them():
    t = gen.ds2d_template((3, 2))
    orc, last = fresh(2)
    n, R, V = 2, t["R"], TINY.vocab
    rng = np.random.default_rng(1)
    tt = rng.integers(0, V, size=(n, R)).astype(np.int32)
    tt[:, 0] = ref.first_tokens(last, n)
    tt[:, t["level"] < 0] = (V - np.minimum(t["level"], 0) - 1)[t["level"] < 0]
    probe = orc.verify_tree([1, 0], np.stack([t["parent"]] * n), tt, commit=False)
    tt[0, 2] = probe["argmax"][0, 0]                      # stream 0 accepts node 2, then (planted below) node 6
    probe = orc.verify_tree([1, 0], np.stack([t["parent"]] * n), tt, commit=False)
    tt[0, 6] = probe["argmax"][0, 2]
    out = orc.ds2d_round([1, 0], t, tt)
    assert list(out["accept_idx"][0][:3]) == [0, 2, 6] and out["accept_len"][0] == 3 and out["accept_len"][1] >= 1
    lg = out["logits"].reshape(n, R, V)
    for s in range(n):
        leaf = int(out["accept_idx"][s][out["accept_len"][s] - 1])
        nxt = out["next_tree_tokens"][s]
        assert nxt[0] == np.argmax(lg[s, leaf])                       # bonus token at the root
        for i in range(1, t["T"]):
            d = int(t["level"][i])
            row = lg[s, t["forecast_of"][leaf] + d - 1]
            order = sorted(range(V), key=lambda v: (-row[v], v))      # falling logit, ties by rising id
            assert nxt[i] == order[int(t["rank"][i])]
        assert all(nxt[i] == V + (-t["level"][i]) - 1 for i in range(t["T"], R))
        # same depth and rank => same token, whatever the parent (product tree)
        assert nxt[4] == nxt[6] == nxt[8] and nxt[5] == nxt[7] == nxt[9]


@pytest.mark.parametrize("branch", [(3, 2), (2, 1, 1)])
def test_drafting_rounds_are_lossless(branch):
    """Whatever the drafts are, the emitted tokens are plain greedy decoding's (Sec. 3.5: the first token of every step is
    the frozen model's own)."""
    t = gen.ds2d_template(branch)
    n, V = 2, TINY.vocab
    ad = [0, -1]
    orc, last = fresh(n, m_forecast=len(branch))
    first = ref.first_tokens(last, n)
    plain, _ = fresh(n)
    want, _ = plain.generate(ad, first, 10)
    tt = np.zeros((n, t["R"]), dtype=np.int32)
    tt[:, 0] = first
    tt[:, t["level"] < 0] = (V - np.minimum(t["level"], 0) - 1)[t["level"] < 0]
    emitted = [[] for _ in range(n)]
    accepted_drafts = 0
    for rnd in range(6):
        if rnd:                                            # give the walk something to accept now and then
            probe = orc.verify_tree(ad, np.stack([t["parent"]] * n), tt, commit=False)
            tt[0, 1] = probe["argmax"][0, 0]
        out = orc.ds2d_round(ad, t, tt)
        for s in range(n):
            path = out["accept_idx"][s][:out["accept_len"][s]]
            emitted[s] += [int(tt[s, u]) for u in path[1:]] + [int(out["next"][s])]
            accepted_drafts += len(path) - 1
        tt = out["next_tree_tokens"].copy()
    assert accepted_drafts > 0
    for s in range(n):
        k = min(len(emitted[s]), 10)
        assert emitted[s][:k] == list(want[:k, s])
