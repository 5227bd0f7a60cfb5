"""End-to-end parity of the decode / verify path on small models, through the C ABI, against the oracle."""
import numpy as np
import pytest

import gen
from oracle import ref
from tests.helpers import compare, check_argmax

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

# small model with a vocabulary: 2 layers, GQA 4/2 heads of 64, adapters on all seven projections
TINYV = gen.ModelCfg("tinyv", 2, 128, 4, 2, 64, 192, 160, 64, 4, 127, 3, 3, 70, b_std=0.05)


@pytest.fixture(scope="module")
def GpuModel():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from tests.helpers import GpuModel as G
    return G


# decode-step paths of the library (debug switch 6): per-layer kernels, or one kernel for the whole step
STEP_PATHS = [pytest.param(1, id="per_layer_kernels"), pytest.param(2, id="single_kernel_step"),
              pytest.param(3, id="kernel_per_projection")]


def make_pair(GpuModel, cfg, seed=0, step_path=0, **kw):
    from paper_2604_18655_b200 import binding as mb
    m = gen.make_model(cfg, seed)
    orc = ref.OracleModel.from_synth(m)
    gm = GpuModel(m, **kw)
    if step_path:
        mb.mlora_debug_set(gm.ctx, 6, step_path)
    for a in range(cfg.n_adapters):
        A, B = gen.make_adapter(cfg, a, seed)
        orc.set_adapter(a, A, B, cfg.alpha)
        gm.set_adapter(a, A, B, cfg.alpha)
    return m, orc, gm


def compare_kv(gm, orc, cfg, n_streams):
    from paper_2604_18655_b200 import binding as mb
    for l in range(cfg.n_layers):
        for s in range(n_streams):
            S = orc.suffix_len(s)
            got_s, k, v = gm.export_kv(l, s, 0, S)
            assert got_s == S
            if S:
                compare(k, orc.suf_k[l][s], f"suffix K l{l} s{s}")
                compare(v, orc.suf_v[l][s], f"suffix V l{l} s{s}")
    mb.mlora_sync_status(gm.ctx)


@pytest.mark.parametrize("step_path", STEP_PATHS)
def test_cfg0_hidden_state_decode(GpuModel, step_path):
    cfg = gen.CFG0
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=8, step_path=step_path)
    prompt = gen.make_hidden(cfg, cfg.prompt_len, 0, 0)
    want_last = orc.prefill_shared(hidden=prompt)
    got_last = gm.prefill_h(prompt)
    compare(got_last, want_last, "prefill last hidden")
    # shared segment KV
    _, pk, pv = gm.export_kv(0, -1, 0, cfg.prompt_len)
    compare(pk, orc.prefix_k[0], "prefix K")
    compare(pv, orc.prefix_v[0], "prefix V")
    ad = list(range(cfg.n_streams))
    for step in range(3):
        x = gen.make_hidden(cfg, cfg.n_streams, 0, 1 + step)
        want = orc.decode_step(ad, hidden=x)["hidden"]
        got = gm.decode_h(ad, x)
        compare(got, want, f"decode hidden step {step}")
    compare_kv(gm, orc, cfg, cfg.n_streams)
    gm.close()


def test_prefill_ragged_causal_chunks(GpuModel):
    """A prompt of 300 positions runs as one causal pass of 256 rows and one of 44 that also attends to the first:
    last hidden row and every position's K/V against the oracle."""
    cfg = gen.ModelCfg("tiny1L300", 1, 512, 8, 8, 64, 1408, 0, 64, 8, 15, 4, 4, 300)
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=8)
    prompt = gen.make_hidden(cfg, cfg.prompt_len, 0, 0)
    want_last = orc.prefill_shared(hidden=prompt)
    got_last = gm.prefill_h(prompt)
    compare(got_last, want_last, "prefill last hidden, 300 positions")
    _, pk, pv = gm.export_kv(0, -1, 0, cfg.prompt_len)
    compare(pk, orc.prefix_k[0], "prefix K")
    compare(pv, orc.prefix_v[0], "prefix V")
    gm.close()


@pytest.mark.parametrize("step_path", STEP_PATHS)
def test_prefill_logits_and_follow_mode_decode(GpuModel, step_path):
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=32, step_path=step_path)
    ids = gen.make_prompt_ids(cfg, 0)
    compare(gm.prefill(ids), orc.prefill_shared(ids), "prefill logits")
    ad = [0, 2, -1]
    toks = np.array([3, 50, 7], dtype=np.int32)
    ties = 0
    for step in range(8):
        nxt, logits = gm.decode(ad, toks)
        r = orc.decode_step(ad, tokens=toks)
        compare(logits, r["logits"], f"decode logits step {step}")
        ties += check_argmax(nxt, r["logits"], f"step {step}")
        assert np.array_equal(nxt, np.argmax(logits, axis=1))            # the GPU's argmax of its own logits
        toks = nxt                                                        # follow the GPU's tokens
    compare_kv(gm, orc, cfg, 3)
    gm.close()


@pytest.mark.parametrize("step_path", STEP_PATHS)
def test_decode_long_weight_streams(GpuModel, step_path):
    """A vocabulary and an FFN wide enough that one CTA's weight chunks of a projection wrap the shared-memory
    ring of the persistent kernel several times (the tiny models never do), 8 streams, rank-16 adapters."""
    from paper_2604_18655_b200 import binding as mb
    cfg = gen.ModelCfg("widev", 1, 256, 4, 2, 64, 2816, 32000, 128, 16, 127, 8, 8, 40, b_std=0.05)
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16, step_path=step_path)
    ids = gen.make_prompt_ids(cfg, 0)
    gm.prefill(ids)
    orc.prefill_shared(ids)
    ad = [0, 1, 2, 3, 4, 5, 6, -1]
    toks = np.arange(8, dtype=np.int32) * 101 + 7
    for step in range(3):
        nxt, logits = gm.decode(ad, toks)
        r = orc.decode_step(ad, tokens=toks)
        compare(logits, r["logits"], f"wide decode logits step {step}")
        check_argmax(nxt, r["logits"], f"wide step {step}")
        toks = nxt
    mb.mlora_sync_status(gm.ctx)
    compare_kv(gm, orc, cfg, 8)
    gm.close()


@pytest.mark.parametrize("step_path", STEP_PATHS)
def test_adapter_switch_without_recreate(GpuModel, step_path):
    """Adapters are run-time inputs: swapping a slot's tensors changes the next step, clearing gives the base."""
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=32, step_path=step_path)
    ids = gen.make_prompt_ids(cfg, 0)
    gm.prefill(ids)
    orc.prefill_shared(ids)
    A9, B9 = gen.make_adapter(cfg, 9, 0)
    gm.set_adapter(1, A9, B9, 8.0)
    orc.set_adapter(1, A9, B9, 8.0)
    gm.set_adapter(2, None, None, 0)
    orc.set_adapter(2, None, None, 0)
    _, logits = gm.decode([1, 2, -1], [5, 5, 5])
    r = orc.decode_step([1, 2, -1], tokens=[5, 5, 5])
    compare(logits, r["logits"], "after adapter switch")
    assert np.abs(logits[0] - logits[2]).max() > 1e-3                     # adapter visible
    compare(logits[1], logits[2], "cleared slot equals base")
    gm.close()


def planted_tree_tokens(rng, cfg, parent, last, truth):
    """Random drafts with the true continuation planted along one branch (deepest-first children)."""
    n, T = len(last), len(parent)
    toks = rng.integers(0, cfg.vocab, size=(n, T)).astype(np.int32)
    toks[:, 0] = last
    dep = gen.tree_depths(parent)
    for s in range(n):
        node = 0
        for d in range(len(truth[s])):
            kids = [u for u in range(T) if parent[u] == node]
            if not kids:
                break
            node = kids[-1]                                              # the last child carries the match
            toks[s, node] = truth[s][d]
    return toks


def test_verify_tree_follow_mode_accept_and_kv(GpuModel):
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=64, max_tree=16)
    ids = gen.make_prompt_ids(cfg, 0)
    gm.prefill(ids)
    orc.prefill_shared(ids)
    ad = [1, 0, 2]
    # plain greedy continuation from the oracle, used as the planted truth
    o2 = ref.OracleModel.from_synth(m)
    for a in range(cfg.n_adapters):
        A, B = gen.make_adapter(cfg, a, 0)
        o2.set_adapter(a, A, B, cfg.alpha)
    o2.prefill_shared(ids)
    first = np.array([11, 12, 13], dtype=np.int32)
    cur, truth = first.copy(), [[] for _ in ad]
    for _ in range(20):
        cur = o2.decode_step(ad, tokens=cur)["next"]
        for s in range(3):
            truth[s].append(int(cur[s]))
    parent = gen.build_tree((4, 2, 2), 16)
    rng = np.random.default_rng(4)
    last = first.copy()
    emitted = [[] for _ in ad]
    total_accept = 0
    for rnd in range(5):
        plant = [truth[s][len(emitted[s]):len(emitted[s]) + 2] for s in range(3)]
        toks = planted_tree_tokens(rng, cfg, parent, last, plant)
        par = np.stack([parent] * 3)
        g = gm.verify(ad, toks, par)
        gpu_argmax = np.argmax(g["logits"], axis=1).reshape(3, 16)
        r = orc.verify_tree(ad, par, toks, follow_argmax=gpu_argmax)
        compare(g["logits"], r["logits"], f"verify logits round {rnd}")
        check_argmax(gpu_argmax.reshape(-1), r["logits"], f"round {rnd}")
        # integer outputs are bit-exact against the oracle's walk on the same argmax
        assert np.array_equal(g["accept_len"], r["accept_len"])
        assert np.array_equal(g["accept_idx"], r["accept_idx"])
        assert np.array_equal(g["next"], r["next"])
        for s in range(3):
            L = int(g["accept_len"][s])
            acc = [int(toks[s, i]) for i in g["accept_idx"][s, 1:L]] + [int(g["next"][s])]
            emitted[s].extend(acc)
            last[s] = acc[-1]
            total_accept += L
    assert total_accept > 15                                             # drafts were accepted (more than 1/round)
    for s in range(3):
        assert orc.suffix_len(s) == gm.suffix_len(s)
    compare_kv(gm, orc, cfg, 3)
    gm.close()


def test_compaction_is_a_bit_exact_copy(GpuModel):
    """Same verify pass twice from the same state: once with compaction skipped.  Row suffix+j of the
    compacted cache must equal, bit for bit, tree row accept_idx[j] of the uncompacted one."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    ids = gen.make_prompt_ids(cfg, 0)
    parent = gen.build_tree((2, 2, 2), 12)
    par = np.stack([parent] * 2)
    outs = []
    for skip in (1, 0):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=32, max_tree=12)
        gm.prefill(ids)
        nxt, _ = gm.decode([0, 1], [4, 5])
        toks = np.zeros((2, 12), dtype=np.int32)
        toks[:, 0] = nxt
        # make every node match the argmax of its parent: chain of accepts down the first-child path
        g0 = gm.decode([0, 1], nxt)[0]
        mb.mlora_reset_streams(gm.ctx)
        gm.decode([0, 1], [4, 5])
        toks[:, 1] = g0
        toks[:, 2] = g0                                                   # duplicate sibling: lowest index must win
        mb.mlora_debug_set(gm.ctx, 1, skip)
        g = gm.verify([0, 1], toks, par)
        S0 = 1
        rows = [gm.export_kv(l, s, 0, S0 + 12)[1:] for l in range(cfg.n_layers) for s in range(2)]
        outs.append((g, rows, gm.suffix_len(0)))
        gm.close()
    (g_skip, rows_skip, s_skip), (g_cmp, rows_cmp, s_cmp) = outs
    assert np.array_equal(g_skip["accept_idx"], g_cmp["accept_idx"])
    assert s_skip == 1 and s_cmp == 1 + int(g_cmp["accept_len"][0])
    assert int(g_cmp["accept_len"][0]) >= 2 and g_cmp["accept_idx"][0, 1] == 1
    i = 0
    for l in range(cfg.n_layers):
        for s in range(2):
            L = int(g_cmp["accept_len"][s])
            for j in range(L):
                src = int(g_cmp["accept_idx"][s, j])
                for t in (0, 1):
                    assert np.array_equal(rows_cmp[i][t][1 + j].view(np.uint16), rows_skip[i][t][1 + src].view(np.uint16))
            i += 1


def test_stream_isolation_on_gpu(GpuModel):
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
    ids = gen.make_prompt_ids(cfg, 0)
    gm.prefill(ids)
    _, multi = gm.decode([0, 1, 2], [9, 9, 9])
    for s in range(3):
        m1, o1, g1 = make_pair(GpuModel, cfg, max_suffix=16, max_streams=1)
        g1.prefill(ids)
        _, single = g1.decode([s], [9])
        compare(multi[s], single[0], f"stream {s} alone")
        g1.close()
    gm.close()


def test_error_paths(GpuModel):
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=2, max_tree=4)
    with pytest.raises(mb.MloraError) as e:
        gm.decode([0], [1])
    assert e.value.code == -2                                            # no prefill yet
    with pytest.raises(mb.MloraError) as e:
        gm.prefill(np.zeros(cfg.prompt_len + 1, dtype=np.int32))
    assert e.value.code == -3
    gm.prefill(gen.make_prompt_ids(cfg, 0))
    with pytest.raises(mb.MloraError) as e:
        gm.decode([0, 0, 0, 0], [1, 1, 1, 1])
    assert e.value.code == -1                                            # more streams than max_streams
    with pytest.raises(mb.MloraError) as e:
        gm.verify([0], np.zeros((1, 5), dtype=np.int32), np.array([[-1, 0, 0, 0, 0]], dtype=np.int32))
    assert e.value.code == -3                                            # tree larger than max_tree
    with pytest.raises(mb.MloraError):
        gm.set_adapter(99, *gen.make_adapter(cfg, 0, 0), 16.0)
    # malformed tree: reported through the device status word, context stays usable
    gm.verify([0], np.zeros((1, 4), dtype=np.int32), np.array([[-1, 0, 2, 1]], dtype=np.int32))
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_sync_status(gm.ctx)
    assert e.value.code == -1
    mb.mlora_sync_status(gm.ctx)                                          # cleared
    # own segment capacity: max_suffix 2 (+ max_tree 4 rows of slack for tree rows)
    mb.mlora_reset_streams(gm.ctx)
    for _ in range(6):
        gm.decode([0], [1])
    with pytest.raises(mb.MloraError) as e:
        gm.decode([0], [1])
    assert e.value.code == -3
    gm.close()


def test_graph_replay_matches_direct_launches(GpuModel):
    """Steps of the multi-kernel path (debug switch 6: no single-kernel step) replayed from a CUDA graph give
    bit-identical logits to directly launched ones."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    res = []
    side = torch.cuda.Stream()                                            # the default stream cannot be captured
    for no_graph in (1, 0):
        with torch.cuda.stream(side):
            m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
            mb.mlora_debug_set(gm.ctx, 6, 1)                 # the multi-kernel path
            mb.mlora_debug_set(gm.ctx, 2, no_graph)
            gm.prefill(gen.make_prompt_ids(cfg, 0))
            dev = torch.device("cuda")
            ad = torch.tensor([0, 1, 2], dtype=torch.int32, device=dev)
            tok = torch.tensor([1, 2, 3], dtype=torch.int32, device=dev)
            nxt = torch.empty(3, dtype=torch.int32, device=dev)
            logits = torch.empty(3, cfg.vocab, dtype=torch.float32, device=dev)
            hist = []
            before = mb.mlora_launch_count(gm.ctx)
            for _ in range(5):
                mb.mlora_decode_step(gm.ctx, ad, tok, nxt, logits)
                tok.copy_(nxt)
                side.synchronize()
                hist.append(logits.cpu().numpy().copy())
            res.append(np.stack(hist))
            assert mb.mlora_launch_count(gm.ctx) - before >= 5 * 4
            gm.close()
    assert np.array_equal(res[0].view(np.uint32), res[1].view(np.uint32))


def test_step_kernel_is_one_launch_and_bit_reproducible(GpuModel):
    """A decode step is ONE kernel launch, and two runs of the same steps give bit-identical logits (the cross-CTA
    sums of the kernel are integer atomics on fixed-point values: the order of arrival cannot change them)."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    res = []
    for rep in range(2):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
        mb.mlora_debug_set(gm.ctx, 6, 2)                     # the single-kernel step
        gm.prefill(gen.make_prompt_ids(cfg, 0))
        toks = np.array([1, 2, 3], dtype=np.int32)
        hist = []
        before = mb.mlora_launch_count(gm.ctx)
        for _ in range(5):
            toks, logits = gm.decode([0, 1, -1], toks)
            hist.append(logits)
        assert mb.mlora_launch_count(gm.ctx) - before == 5
        res.append(np.stack(hist))
        mb.mlora_sync_status(gm.ctx)
        gm.close()
    assert np.array_equal(res[0].view(np.uint32), res[1].view(np.uint32))


def test_step_timeline_of_the_default_decode_path(GpuModel):
    """Debug switch 7 on the kernel-per-projection path: the traced instantiations give the same tokens and logits as
    the untraced kernels, and every stamped launch reads start <= wait returned <= main loop done <= end <= latest end
    of all its CTAs, the launches in step order."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    res = []
    for trace in (0, 1):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
        mb.mlora_debug_set(gm.ctx, 6, 3)
        mb.mlora_debug_set(gm.ctx, 7, trace)
        gm.prefill(gen.make_prompt_ids(cfg, 0))
        toks = np.array([1, 2, 3], dtype=np.int32)
        hist = []
        for _ in range(3):
            toks, logits = gm.decode([0, 1, -1], toks)
            hist.append(logits)
        res.append(np.stack(hist))
        if trace:
            tl = mb.mlora_step_timeline(gm.ctx)
            rows = [r for r in tl[0] if r[0]]
            assert len(rows) >= 5 * cfg.n_layers                  # q,k,v / attention / o / gate,up / down per layer (+ lm_head)
            prev = 0
            for r in rows:
                assert r[0] <= r[1] <= r[2] <= r[3] <= r[4], r
                assert r[4] >= prev                                   # a launch ends after the one before it
                prev = r[4]
        mb.mlora_sync_status(gm.ctx)
        gm.close()
    assert np.array_equal(res[0].view(np.uint32), res[1].view(np.uint32))


def test_switching_decode_paths_in_one_context(GpuModel):
    """Debug switch 6 in the middle of a context's life: steps of the single-kernel path that follow steps of the
    kernel-per-projection path give, bit for bit, what a context that only ever ran the single-kernel path gives (the
    step's accumulators are cleared at the switch)."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    res = []
    for warm_path in (2, 3):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
        gm.prefill(gen.make_prompt_ids(cfg, 0))
        mb.mlora_debug_set(gm.ctx, 6, warm_path)
        toks = np.array([1, 2, 3], dtype=np.int32)
        for _ in range(2):
            gm.decode([0, 1, -1], toks)
        mb.mlora_reset_streams(gm.ctx)
        mb.mlora_debug_set(gm.ctx, 6, 2)
        hist = []
        for _ in range(3):
            toks, logits = gm.decode([0, 1, -1], toks)
            hist.append(logits)
        res.append(np.stack(hist))
        mb.mlora_sync_status(gm.ctx)
        gm.close()
    assert np.array_equal(res[0].view(np.uint32), res[1].view(np.uint32))


def test_decode_paths_agree(GpuModel):
    """The single-kernel step against the per-layer persistent projection kernel (debug switch 6) and the
    one-kernel-per-projection form of the same arithmetic (debug switch 3): logits and KV within the parity tolerance."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    res = []
    for key, val in ((6, 2), (6, 1), (3, 1)):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
        mb.mlora_debug_set(gm.ctx, key, val)
        gm.prefill(gen.make_prompt_ids(cfg, 0))
        toks = np.array([1, 2, 3], dtype=np.int32)
        hist = []
        for _ in range(4):
            toks, logits = gm.decode([0, 1, -1], toks)
            hist.append(logits)
        _, k, v = gm.export_kv(1, 0, 0, 4)
        res.append((np.stack(hist), k, v))
        mb.mlora_sync_status(gm.ctx)
        gm.close()
    for i in (0, 1):
        compare(res[i][0], res[2][0], "logits across paths")
        compare(res[i][1], res[2][1], "K across paths")
        compare(res[i][2], res[2][2], "V across paths")


def test_debug_dequant_of_fused_projections_is_bit_exact(GpuModel):
    """The context's own weights -- q, k, v packed into one fused matrix, gate and up interleaved by tiles, and the
    plain ones -- unpacked by the kernels' dequantisation and compared bit for bit with the oracle's."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=8)
    for layer in (0, cfg.n_layers - 1):
        for p, name in enumerate(gen.PROJ_NAMES):
            K, N = gen.proj_shape(cfg, name)
            out = torch.empty(K, N, dtype=torch.float16, device="cuda")
            mb.mlora_debug_dequant(gm.ctx, layer, p, out)
            torch.cuda.synchronize()
            want = ref.dequant(m.qweight[layer * 7 + p], m.scales[layer * 7 + p], cfg.group_size)
            assert np.array_equal(out.cpu().numpy().view(np.uint16), want.view(np.uint16)), (layer, name)
    K, N = gen.proj_shape(cfg, "lm_head")
    out = torch.empty(K, N, dtype=torch.float16, device="cuda")
    mb.mlora_debug_dequant(gm.ctx, cfg.n_layers, 0, out)
    torch.cuda.synchronize()
    want = ref.dequant(m.qweight[cfg.n_layers * 7], m.scales[cfg.n_layers * 7], cfg.group_size)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), want.view(np.uint16))
    gm.close()


def test_export_state_gives_the_whole_own_segment(GpuModel):
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
    ids = gen.make_prompt_ids(cfg, 0)
    gm.prefill(ids)
    orc.prefill_shared(ids)
    toks = np.array([5, 6, 7], dtype=np.int32)
    for _ in range(3):
        toks, _ = gm.decode([0, 1, -1], toks)
    k = torch.zeros(17, cfg.n_kv_heads, cfg.head_dim, dtype=torch.float16, device="cuda")
    v = torch.zeros_like(k)
    S = mb.mlora_export_state(gm.ctx, 1, 2, k, v)
    assert S == 3
    _, k2, v2 = gm.export_kv(1, 2, 0, 3)
    assert np.array_equal(k.cpu().numpy()[:3], k2) and np.array_equal(v.cpu().numpy()[:3], v2)
    gm.close()


def test_decode_over_a_long_shared_prompt(GpuModel):
    """Decode steps over a 2100-token shared prompt: past the single-kernel attention's limit, so the layers' attention
    runs in the streaming kernel with q, k rotated on load and the new K/V row appended by it."""
    cfg = gen.ModelCfg("tinylong", 2, 128, 4, 2, 64, 192, 160, 64, 4, 127, 3, 3, 2100, b_std=0.05)
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=8)
    ids = gen.make_prompt_ids(cfg, 0)
    compare(gm.prefill(ids), orc.prefill_shared(ids, n_streams=3), "long prompt prefill logits")
    ad, toks = [0, -1, 2], np.array([3, 4, 5], dtype=np.int32)
    for step in range(4):
        nxt, logits = gm.decode(ad, toks)
        r = orc.decode_step(ad, tokens=toks)
        compare(logits, r["logits"], f"long prompt decode logits step {step}")
        check_argmax(nxt, r["logits"], f"long prompt step {step}")
        toks = nxt
    compare_kv(gm, orc, cfg, 3)
    gm.close()


def test_ds2d_rounds_verify_and_draft_on_the_device(GpuModel):
    """DS2D inference steps (Sec. 3.5, App. A.2): every pass verifies a (3,2) tree and drafts the next one from the
    forecast rows of the last accepted node, the drafted tokens staying on the device.  Follow mode: the oracle walks on
    the GPU's row argmax; accept results and the cache are exact, logits within tolerance, and the drafts are exactly
    the top ids of the GPU's own forecast logits (and near-maximal in the oracle's)."""
    from dataclasses import replace
    from paper_2604_18655_b200 import binding as mb
    # (adapters a few times the base projection, not TINYV's ten times: with random draft tokens at every node the
    # fp16 activations' rounding, amplified by the adapter branch, otherwise sits right at the logit tolerance)
    cfg = replace(TINYV, name="tinyds2d", b_std=0.02)
    t = gen.ds2d_template((3, 2))
    R, m, V, n = t["R"], t["m"], cfg.vocab, cfg.n_streams
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        mdl, orc, gm = make_pair(GpuModel, cfg, max_suffix=40, max_tree=R)
        fc = gen.make_forecast(cfg, m, 0)
        d_fc = torch.from_numpy(fc).cuda()
        mb.mlora_set_forecast(gm.ctx, d_fc)
        orc.set_forecast(fc)
        ids = gen.make_prompt_ids(cfg, 0)
        last = gm.prefill(ids)
        orc.prefill_shared(ids, n_streams=n)
        ad = [2, -1, 0]
        dv = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
        d_ad = dv(np.array(ad, dtype=np.int32))
        d_par = dv(np.stack([t["parent"]] * n))
        d_lvl, d_rank, d_fo, d_w = dv(t["level"]), dv(t["rank"]), dv(t["forecast_of"]), dv(t["widths"])
        tt = np.zeros((n, R), dtype=np.int32)
        tt[:, 0] = ref.first_tokens(last, n)
        tt[:, 1:t["T"]] = np.random.default_rng(0).integers(0, V, size=(n, t["T"] - 1))
        tt[:, t["level"] < 0] = (V - np.minimum(t["level"], 0) - 1)[t["level"] < 0]
        bufs = [dv(tt), torch.empty(n, R, dtype=torch.int32, device="cuda")]
        acc_len = torch.empty(n, dtype=torch.int32, device="cuda")
        acc_idx = torch.empty(n, R, dtype=torch.int32, device="cuda")
        nxt = torch.empty(n, dtype=torch.int32, device="cuda")
        logits = torch.empty(n * R, V, dtype=torch.float32, device="cuda")
        accepted = 0
        for rnd in range(5):
            cur, out = bufs[rnd & 1], bufs[(rnd + 1) & 1]
            h_tt = cur.cpu().numpy().copy()
            if rnd in (1, 3):                           # plant the true continuation on a draft node of stream 0 (and
                probe = orc.verify_tree(ad, np.stack([t["parent"]] * n), h_tt, commit=False)    # its child in round 3)
                h_tt[0, 2] = probe["argmax"][0, 0]
                if rnd == 3:
                    probe = orc.verify_tree(ad, np.stack([t["parent"]] * n), h_tt, commit=False)
                    h_tt[0, 7] = probe["argmax"][0, 2]
                cur.copy_(dv(h_tt))
            mb.mlora_ds2d_round(gm.ctx, d_ad, cur, d_par, d_lvl, d_rank, d_fo, d_w, int(t["widths"].max()),
                                acc_len, acc_idx, nxt, out, logits)
            side.synchronize()
            g_logits = logits.cpu().numpy()
            r = orc.ds2d_round(ad, t, h_tt, follow_argmax=np.argmax(g_logits, axis=1).reshape(n, R))
            compare(g_logits, r["logits"], f"ds2d round {rnd} logits")
            assert np.array_equal(acc_len.cpu().numpy(), r["accept_len"])
            assert np.array_equal(acc_idx.cpu().numpy(), r["accept_idx"])
            assert np.array_equal(nxt.cpu().numpy(), r["next"])
            accepted += int(r["accept_len"].sum()) - n
            g_next = out.cpu().numpy()
            o_lg = r["logits"].reshape(n, R, V)
            for s in range(n):
                leaf = int(r["accept_idx"][s][r["accept_len"][s] - 1])
                for i in range(R):
                    lv = int(t["level"][i])
                    if lv == 0:
                        assert g_next[s, i] == nxt[s].item()
                    elif lv < 0:
                        assert g_next[s, i] == V - lv - 1
                    else:
                        row = s * R + int(t["forecast_of"][leaf]) + lv - 1
                        want = ref.first_tokens(g_logits[row], int(t["widths"][lv - 1]))[int(t["rank"][i])]
                        assert g_next[s, i] == want, (rnd, s, i)
                        o_row = o_lg[s, int(t["forecast_of"][leaf]) + lv - 1]
                        kth = np.sort(o_row)[::-1][int(t["rank"][i])]
                        assert abs(o_row[g_next[s, i]] - kth) <= 1e-2       # the oracle's r-th best, up to near-ties
        assert accepted >= 3
        compare_kv(gm, orc, cfg, n)
        # the second call with the same arguments replays the captured graph: same outputs
        mb.mlora_sync_status(gm.ctx)
        mb.mlora_set_forecast(gm.ctx, None)
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_ds2d_round(gm.ctx, d_ad, bufs[1], d_par, d_lvl, d_rank, d_fo, d_w, 3, acc_len, acc_idx, nxt, bufs[0])
        assert e.value.code == -2
        gm.close()


def test_sample_first_matches_oracle(GpuModel):
    """The n distinct first tokens (App. A.1): integer work, exact -- with ties, infinities, signed zeros and NaN."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=8)
    rng = np.random.default_rng(3)
    rows = [np.round(rng.standard_normal(cfg.vocab) * 2) / 2, rng.standard_normal(cfg.vocab), np.zeros(cfg.vocab)]
    special = rng.standard_normal(cfg.vocab)
    special[[5, 9]] = np.nan
    special[[7, 70]] = np.inf
    special[[1, 100]] = -np.inf
    special[[30, 31]] = [-0.0, 0.0]
    rows.append(special)
    for row in rows:
        row = row.astype(np.float32)
        for n in (1, 3, 8, cfg.vocab):
            out = torch.full((n,), -7, dtype=torch.int32, device="cuda")
            mb.mlora_sample_first(gm.ctx, torch.from_numpy(row).cuda(), out)
            torch.cuda.synchronize()
            assert np.array_equal(out.cpu().numpy(), ref.first_tokens(row, n))
    with pytest.raises(mb.MloraError):
        mb.mlora_sample_first(gm.ctx, torch.zeros(cfg.vocab, device="cuda"), torch.zeros(cfg.vocab + 1, dtype=torch.int32, device="cuda"))
    gm.close()


@pytest.mark.parametrize("step_path", STEP_PATHS)
def test_generation_in_one_call_matches_step_by_step(GpuModel, step_path):
    """prefill -> sampler -> k steps with the tokens fed back on the device: the same tokens and the same cache, bit for
    bit, as k single-step calls; the tokens are the oracle's wherever its margin decides; twice (the second call
    replays the graph of the first)."""
    from paper_2604_18655_b200 import binding as mb
    cfg, k = TINYV, 12
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        m, orc, gm = make_pair(GpuModel, cfg, step_path=step_path, max_suffix=16)
        ids = gen.make_prompt_ids(cfg, 0)
        last = torch.from_numpy(gm.prefill(ids)).cuda()
        want_last = orc.prefill_shared(ids, n_streams=cfg.n_streams)
        n = cfg.n_streams
        first = torch.empty(n, dtype=torch.int32, device="cuda")
        mb.mlora_sample_first(gm.ctx, last, first)
        assert np.array_equal(first.cpu().numpy(), ref.first_tokens(last.cpu().numpy(), n))
        ad = [1, -1, 0]
        d_ad = torch.tensor(ad, dtype=torch.int32, device="cuda")
        # step by step
        toks, steps = first.cpu().numpy(), []
        for _ in range(k):
            toks, _ = gm.decode(ad, toks, want_logits=False)
            steps.append(toks)
        steps = np.stack(steps)
        kv = [gm.export_kv(l, s, 0, k) for l in range(cfg.n_layers) for s in range(n)]
        for rep in range(2):
            mb.mlora_reset_streams(gm.ctx)
            out = torch.full((k, n), -1, dtype=torch.int32, device="cuda")
            mb.mlora_generate(gm.ctx, d_ad, first, out)
            side.synchronize()
            assert np.array_equal(out.cpu().numpy(), steps), f"call {rep}"
            kv2 = [gm.export_kv(l, s, 0, k) for l in range(cfg.n_layers) for s in range(n)]
            for (s1, k1, v1), (s2, k2, v2) in zip(kv, kv2):
                assert s1 == s2 == k
                assert np.array_equal(k1.view(np.uint16), k2.view(np.uint16)) and np.array_equal(v1.view(np.uint16), v2.view(np.uint16))
        # host-array form
        mb.mlora_reset_streams(gm.ctx)
        h_out = torch.empty(k, n, dtype=torch.int32).pin_memory()
        mb.mlora_generate_host(gm.ctx, torch.tensor(ad, dtype=torch.int32), first.cpu(), h_out)
        assert np.array_equal(h_out.numpy(), steps)
        # the oracle, walked along the GPU's tokens
        toks = first.cpu().numpy()
        for j in range(k):
            r = orc.decode_step(ad, tokens=toks)
            check_argmax(steps[j], r["logits"], f"generation step {j}")
            toks = steps[j]
        # the own segments cannot take another k rows on top: CAPACITY, nothing enqueued
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_generate(gm.ctx, d_ad, first, out)
        assert e.value.code == -3
        mb.mlora_sync_status(gm.ctx)
        gm.close()


def test_host_buffer_step_matches_device_step(GpuModel):
    """mlora_decode_step_host (host arrays in and out) gives the tokens of mlora_decode_step."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    outs = []
    for host in (False, True):
        m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16)
        gm.prefill(gen.make_prompt_ids(cfg, 0))
        toks = np.array([4, 9, 11], dtype=np.int32)
        hist = []
        for _ in range(4):
            if host:
                h_ad = torch.tensor([0, 1, -1], dtype=torch.int32).pin_memory()
                h_tok = torch.from_numpy(toks.copy()).pin_memory()
                h_next = torch.empty(3, dtype=torch.int32).pin_memory()
                mb.mlora_decode_step_host(gm.ctx, h_ad, h_tok, h_next)
                toks = h_next.numpy().copy()
            else:
                toks, _ = gm.decode([0, 1, -1], toks, want_logits=False)
            hist.append(toks.copy())
        outs.append(np.stack(hist))
        mb.mlora_sync_status(gm.ctx)
        gm.close()
    assert np.array_equal(outs[0], outs[1])


@pytest.mark.parametrize("step_path", STEP_PATHS[:2])       # (the kernel-per-projection path has no device-side wait)
def test_bounded_wait_runs_out_and_context_recovers(GpuModel, step_path):
    """Failure detection without a fault: a grid barrier of the persistent kernel is made to wait (limit ~0.1 s) for an
    arrival nobody makes.  The kernel must return, the device status must say TIMEOUT and name the wait, and after
    mlora_sync_status the same context must compute the same logits as before."""
    from paper_2604_18655_b200 import binding as mb
    cfg = TINYV
    m, orc, gm = make_pair(GpuModel, cfg, max_suffix=16, step_path=step_path)
    ids = gen.make_prompt_ids(cfg, 0)
    toks = np.array([1, 2, 3], dtype=np.int32)
    gm.prefill(ids)
    _, want = gm.decode([0, 1, -1], toks)
    mb.mlora_sync_status(gm.ctx)
    gm.prefill(ids)
    mb.mlora_debug_set(gm.ctx, 5, 1)
    gm.decode([0, 1, -1], toks)                        # returns (with garbage) instead of hanging
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_sync_status(gm.ctx)
    assert e.value.code == -5 and "wait kind 5" in str(e.value)
    mb.mlora_sync_status(gm.ctx)                       # cleared
    gm.prefill(ids)
    _, got = gm.decode([0, 1, -1], toks)
    mb.mlora_sync_status(gm.ctx)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    gm.close()
