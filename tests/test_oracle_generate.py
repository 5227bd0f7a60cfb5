"""Pins for the oracle's first-token sampler and its generation loop (App. A.1 flowsheet: one prefill, a sampler that
hands the n streams n distinct first tokens, then the n-fold model step after step)."""
import itertools

import numpy as np
import pytest

import gen
from oracle import ref

TINY = gen.ModelCfg("tinygen", 2, 64, 2, 1, 32, 96, 50, 32, 4, 127, 3, 3, 6, b_std=0.05)


def satisfies_definition(logits, picks):
    """The defining properties, checked one by one: distinct ids; listed by falling logit, equal logits by rising id;
    nothing left out ranks before the last pick."""
    picks = list(picks)
    if len(set(picks)) != len(picks):
        return False
    before = lambda a, b: logits[a] > logits[b] or (logits[a] == logits[b] and a < b)       # noqa: E731
    if any(not before(a, b) for a, b in zip(picks, picks[1:])):
        return False
    rest = [i for i in range(len(logits)) if i not in picks]
    return all(before(picks[-1], i) for i in rest)


def test_first_tokens_is_the_only_selection_that_satisfies_the_definition():
    """Every row of length 5 over three values (so ties abound), every n: among ALL ordered selections exactly one
    satisfies the definition, and it is the oracle's."""
    for row in itertools.product([0.0, 1.0, -2.5], repeat=5):
        for n in range(1, 6):
            good = [p for p in itertools.permutations(range(5), n) if satisfies_definition(row, p)]
            assert len(good) == 1
            assert list(ref.first_tokens(np.array(row), n)) == list(good[0])


@pytest.mark.parametrize("seed", range(4))
def test_first_tokens_against_library_routines(seed):
    rng = np.random.default_rng(seed)
    row = np.round(rng.standard_normal(300) * 3) / 4            # many exact ties
    assert ref.first_tokens(row, 1)[0] == np.argmax(row)         # numpy: first occurrence of the maximum
    assert np.array_equal(ref.first_tokens(row, 300), np.argsort(-row, kind="stable"))
    assert np.array_equal(ref.first_tokens(row, 17), np.argsort(-row, kind="stable")[:17])


def test_first_tokens_special_values():
    row = np.array([np.nan, -np.inf, 3.0, np.inf, 3.0, -0.0, 0.0, np.nan], dtype=np.float32)
    # +inf first, the two 3.0 by id, the two zeros (equal as numbers) by id, -inf, then the NaNs by id
    assert list(ref.first_tokens(row, 8)) == [3, 2, 4, 5, 6, 1, 0, 7]


def test_planted_tie_rule_mistake_fails():
    row = np.array([1.0, 2.0, 2.0, 0.0])
    wrong = sorted(range(4), key=lambda i: (-row[i], -i))[:2]    # ties by falling id
    assert not satisfies_definition(row, wrong)
    assert satisfies_definition(row, ref.first_tokens(row, 2))


def test_generation_is_each_stream_decoding_alone():
    """Stream isolation (Sec. 3.4) carried through a whole generation: the n-fold loop gives every stream the tokens it
    produces when it is the only stream."""
    m = gen.make_model(TINY, 0)
    ids = gen.make_prompt_ids(TINY, 0)
    ads = [gen.make_adapter(TINY, a, 0) for a in range(3)]

    def fresh(n_streams):
        orc = ref.OracleModel.from_synth(m)
        for a, (A, B) in enumerate(ads):
            orc.set_adapter(a, A, B, TINY.alpha)
        return orc, orc.prefill_shared(ids, n_streams=n_streams)

    orc, last = fresh(3)
    first = ref.first_tokens(last, 3)
    assert len(set(first.tolist())) == 3
    ad = [2, -1, 0]
    toks, logits = orc.generate(ad, first, 5)
    assert toks.shape == (5, 3) and logits.shape == (5, 3, TINY.vocab)
    assert np.array_equal(toks, np.argmax(logits, axis=2))
    for s in range(3):
        solo, _ = fresh(1)
        t, _ = solo.generate([ad[s]], first[s:s + 1], 5)
        assert np.array_equal(t[:, 0], toks[:, s])
    assert all(orc.suffix_len(s) == 5 for s in range(3))
