"""Parity at the full widths of the benchmark workloads, in the launch configuration bench.py times (CUDA-graph
replay on a side stream, persistent projection kernel for decode-sized passes): the ~1B model with all 16 layers
(decode steps of 8 streams and one 8 x 16-node verify pass), and a 2-layer cut of the ~3B model at its real
widths (head_dim 128, rank-32 adapters, 32-node trees).  The shared prompt is cut to 64 tokens so that the CPU
oracle's prefill stays within seconds; every weight matrix, adapter and projection has its full size."""
import numpy as np
import pytest

import gen
from oracle import ref
from tests.helpers import compare, check_argmax

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

PROMPT = 64


def build(cfg, max_tree, prompt=PROMPT, max_suffix=None):
    from tests.helpers import GpuModel
    m = gen.make_model(cfg, 0)
    orc = ref.OracleModel.from_synth(m, dtype=np.float32)
    gm = GpuModel(m, max_prefix=prompt, max_suffix=max_suffix or 8 + 3 * max_tree, max_tree=max_tree)
    for a in range(cfg.n_adapters):
        A, B = gen.make_adapter(cfg, a, 0)
        orc.set_adapter(a, A, B, cfg.alpha)
        gm.set_adapter(a, A, B, cfg.alpha)
    return m, orc, gm


def run_decode_and_verify(cfg, n_decode, branch, T, step_path=0):
    from paper_2604_18655_b200 import binding as mb
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    side = torch.cuda.Stream()                       # graph replay needs a capturable stream, as in bench.py
    with torch.cuda.stream(side):
        m, orc, gm = build(cfg, T)
        mb.mlora_debug_set(gm.ctx, 6, step_path)
        ids = gen.make_prompt_ids(cfg, 0, PROMPT)
        got_last = gm.prefill(ids)
        want_last = orc.prefill_shared(ids, n_streams=cfg.n_streams)
        compare(got_last, want_last, f"{cfg.name} prefill logits")
        n = cfg.n_streams
        ad = list(range(n - 1)) + [-1]               # seven adapters and one base-weight stream
        toks = np.argsort(-want_last)[:n].astype(np.int32)   # n distinct first tokens (App. A.1)
        for step in range(n_decode):
            nxt, logits = gm.decode(ad, toks)
            r = orc.decode_step(ad, tokens=toks)
            compare(logits, r["logits"], f"{cfg.name} decode logits step {step}")
            check_argmax(nxt, r["logits"], f"{cfg.name} decode step {step}")
            toks = nxt                               # follow the GPU's tokens
        # one verify pass: random drafts, with the true next token planted on the first child of the root
        parent = gen.build_tree(branch, T)
        rng = np.random.default_rng(5)
        tt = rng.integers(0, cfg.vocab, size=(n, T)).astype(np.int32)
        tt[:, 0] = toks
        probe = orc.verify_tree(ad, np.stack([parent] * n), tt, commit=False)
        tt[:, 1] = probe["argmax"][:, 0]             # the root's greedy continuation (root logits do not depend on drafts)
        res = gm.verify(ad, tt, np.stack([parent] * n))
        r = orc.verify_tree(ad, np.stack([parent] * n), tt, follow_argmax=np.argmax(res["logits"], axis=1).reshape(n, T))
        compare(res["logits"], r["logits"], f"{cfg.name} verify logits")
        check_argmax(np.argmax(res["logits"], axis=1), r["logits"], f"{cfg.name} verify rows")
        assert np.array_equal(res["accept_len"], r["accept_len"])          # integer work: exact
        assert np.array_equal(res["accept_idx"], r["accept_idx"])
        assert np.array_equal(res["next"], r["next"])
        assert (res["accept_len"] >= 2).all()        # the planted token was accepted
        for s in (0, n - 1):
            S = orc.suffix_len(s)
            got_s, k, v = gm.export_kv(cfg.n_layers - 1, s, 0, S)
            assert got_s == S
            compare(k, orc.suf_k[cfg.n_layers - 1][s], f"{cfg.name} suffix K stream {s}")
            compare(v, orc.suf_v[cfg.n_layers - 1][s], f"{cfg.name} suffix V stream {s}")
        mb.mlora_sync_status(gm.ctx)
        gm.close()


def test_llama1b_full_depth_decode_and_verify():
    run_decode_and_verify(gen.CFG1, n_decode=3, branch=(4, 2, 2), T=16)


def test_llama1b_full_depth_single_kernel_step():
    """The same workload with decode steps through the kernel that does a whole step in one launch."""
    run_decode_and_verify(gen.CFG1, n_decode=3, branch=(4, 2, 2), T=16, step_path=2)


@pytest.mark.parametrize("step_path", [1, 2, 3])
def test_llama1b_full_prompt_sixteen_steps(step_path):
    """The benchmark workload itself: the full 512-token shared prompt, 8 streams, 16 greedy decode steps in follow
    mode (the oracle walks on the GPU's tokens), logits of every step against the oracle, own-segment KV at the end."""
    from paper_2604_18655_b200 import binding as mb
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    cfg = gen.CFG1
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        m, orc, gm = build(cfg, 1, prompt=cfg.prompt_len, max_suffix=24)
        mb.mlora_debug_set(gm.ctx, 6, step_path)
        ids = gen.make_prompt_ids(cfg, 0)
        got_last = gm.prefill(ids)
        want_last = orc.prefill_shared(ids, n_streams=cfg.n_streams)
        compare(got_last, want_last, "llama1b prefill logits, 512 tokens")
        n = cfg.n_streams
        ad = list(range(n))
        toks = np.argsort(-want_last)[:n].astype(np.int32)
        first, produced = toks, []
        for step in range(16):
            nxt, logits = gm.decode(ad, toks)
            r = orc.decode_step(ad, tokens=toks)
            compare(logits, r["logits"], f"llama1b full-prompt decode logits step {step}")
            check_argmax(nxt, r["logits"], f"llama1b full-prompt decode step {step}")
            toks = nxt
            produced.append(nxt)
        for s in (0, n - 1):
            got_s, k, v = gm.export_kv(cfg.n_layers - 1, s, 0, 16)
            assert got_s == 16
            compare(k, orc.suf_k[cfg.n_layers - 1][s], f"suffix K stream {s}")
            compare(v, orc.suf_v[cfg.n_layers - 1][s], f"suffix V stream {s}")
        # the same generation as ONE call (one graph of 16 steps, tokens fed back on the device): the same tokens
        mb.mlora_reset_streams(gm.ctx)
        out = torch.empty(16, n, dtype=torch.int32, device="cuda")
        mb.mlora_generate(gm.ctx, torch.tensor(ad, dtype=torch.int32, device="cuda"), torch.from_numpy(first).cuda(), out)
        side.synchronize()
        assert np.array_equal(out.cpu().numpy(), np.stack(produced))
        mb.mlora_sync_status(gm.ctx)
        gm.close()


def test_llama3b_widths_two_layers_decode_and_verify():
    cfg = gen.CFG3.small(n_layers=2, name="llama3b-cut2L")
    run_decode_and_verify(cfg, n_decode=2, branch=(4, 4, 2), T=32)
