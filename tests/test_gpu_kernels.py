"""Kernel-level parity through the C ABI: INT4 unpack/dequant (bit-exact), fused INT4 GEMM + per-row LoRA,
shared-prefix / own-segment / tree-mask attention -- each against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

import gen
from oracle import ref
from tests.helpers import compare

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def mb():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_18655_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# ------------------------------------------------------------------ dequant
def test_dequant_bit_exact_all_scales_all_nibbles(mb):
    """16 nibbles x every finite fp16 scale pattern (both signs, subnormals included)."""
    bits = np.concatenate([np.arange(0, 0x7C00), np.arange(0x8000, 0xFC00)]).astype(np.uint16)
    N, K, G = len(bits), 64, 64
    assert N == 63488 and N % 16 == 0
    scales = bits.view(np.float16).reshape(1, N)
    u = np.broadcast_to((np.arange(K) % 16).astype(np.uint8)[:, None], (K, N))
    u = (u + (np.arange(N) % 16).astype(np.uint8)[None, :]) % 16        # every column sees all 16 nibbles
    qb = gen.pack_nibbles(np.ascontiguousarray(u.astype(np.uint8)))
    w = mb.mlora_weight_create(dev(qb), dev(scales), K, N, G)
    out = torch.empty(K, N, dtype=torch.float16, device="cuda")
    mb.mlora_weight_dequant(w, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint16)
    want = ref.dequant(qb, scales, G).view(np.uint16)
    mb.mlora_weight_destroy(w)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("K,N,G", [(128, 48, 64), (256, 1040, 128), (512, 64, 128)])
def test_dequant_bit_exact_random_weights(mb, K, N, G):
    rng = np.random.default_rng(K + N)
    qb, sc = gen.quantize_int4(rng.standard_normal((K, N)).astype(np.float32) * 0.02, G)
    w = mb.mlora_weight_create(dev(qb), dev(sc), K, N, G)
    out = torch.empty(K, N, dtype=torch.float16, device="cuda")
    mb.mlora_weight_dequant(w, out)
    torch.cuda.synchronize()
    mb.mlora_weight_destroy(w)
    assert np.array_equal(out.cpu().numpy().view(np.uint16), ref.dequant(qb, sc, G).view(np.uint16))


# ------------------------------------------------------------------ fused GEMM + LoRA
def run_linear(mb, K, N, G, M, n_ad, rank, seed, with_base_rows=True):
    rng = np.random.default_rng(seed)
    qb, sc = gen.quantize_int4(rng.standard_normal((K, N)).astype(np.float32) * 0.02, G)
    x = rng.standard_normal((M, K)).astype(np.float16)
    w = mb.mlora_weight_create(dev(qb), dev(sc), K, N, G)
    ws = torch.zeros(mb.mlora_linear_workspace_bytes(w, M, max(rank, 1)), dtype=torch.uint8, device="cuda")
    y = torch.empty(M, N, dtype=torch.float32, device="cuda")
    Wd = ref.dequant(qb, sc, G).astype(np.float64)
    xd = dev(x)
    if n_ad == 0:
        mb.mlora_linear(w, xd, y, ws)
        want = ref.linear_lora(x.astype(np.float64), Wd)
    else:
        A = [(rng.standard_normal((rank, K)) / rank).astype(np.float16) for _ in range(n_ad)]
        B = [(rng.standard_normal((rank, N)) * 0.05).astype(np.float16) for _ in range(n_ad)]
        scale = (16.0 / rank * (1 + 0.25 * np.arange(n_ad))).astype(np.float32)
        rows = rng.integers(-1 if with_base_rows else 0, n_ad, size=M).astype(np.int32)
        dA, dB = [dev(a) for a in A], [dev(b) for b in B]
        pa = torch.tensor([t.data_ptr() for t in dA], dtype=torch.int64, device="cuda")
        pb = torch.tensor([t.data_ptr() for t in dB], dtype=torch.int64, device="cuda")
        for _ in range(2):          # twice: the scratch (split counters) must be left ready for reuse
            mb.mlora_linear(w, xd, y, ws, dev(rows), pa, pb, dev(scale), rank)
        want = ref.linear_lora(x.astype(np.float64), Wd, rows, [a.astype(np.float64) for a in A],
                               [b.astype(np.float64) for b in B], scale.astype(np.float64))
    torch.cuda.synchronize()
    got = y.cpu().numpy()
    mb.mlora_weight_destroy(w)
    return got, want


@pytest.mark.parametrize("K,N,G", [(256, 192, 64), (512, 1040, 128), (2048, 512, 128), (1408, 512, 64)])
@pytest.mark.parametrize("M", [1, 3, 8, 20, 130])
def test_linear_base_matches_oracle(mb, K, N, G, M):
    got, want = run_linear(mb, K, N, G, M, 0, 0, seed=K * 7 + N + M)
    compare(got, want, f"linear base K{K} N{N} M{M}")


@pytest.mark.parametrize("K,N,G,M,n_ad,rank", [
    (256, 192, 64, 8, 1, 8), (512, 1040, 128, 8, 8, 16), (2048, 512, 128, 5, 3, 4), (512, 2048, 128, 32, 8, 32),
    (1024, 1024, 128, 130, 32, 16), (512, 512, 128, 16, 64, 64), (4096, 4096, 128, 8, 8, 16),
])
def test_linear_lora_matches_oracle(mb, K, N, G, M, n_ad, rank):
    got, want = run_linear(mb, K, N, G, M, n_ad, rank, seed=K + N + M + n_ad + rank)
    compare(got, want, f"linear lora K{K} N{N} M{M} ad{n_ad} r{rank}")


@pytest.mark.parametrize("K,N", [(14336, 4096), (4096, 14336)])
@pytest.mark.parametrize("M", [8, 256])
def test_linear_lora_at_the_sweep_shapes(mb, K, N, M):
    """The widest shapes of the single-projection workload (inputs or outputs of 14336 features), 8 adapters of rank 16
    picked per row at random: the few-row kernels and the tensor-core path with its widest row block."""
    got, want = run_linear(mb, K, N, 128, M, 8, 16, seed=K + M)
    compare(got, want, f"linear lora K{K} N{N} M{M}")


def test_linear_status_call_reports_nothing_after_clean_calls(mb):
    rng = np.random.default_rng(2)
    qb, sc = gen.quantize_int4(rng.standard_normal((256, 64)).astype(np.float32), 64)
    w = mb.mlora_weight_create(dev(qb), dev(sc), 256, 64, 64)
    x = dev(rng.standard_normal((4, 256)).astype(np.float16))
    y = torch.empty(4, 64, dtype=torch.float32, device="cuda")
    ws = torch.zeros(mb.mlora_linear_workspace_bytes(w, 4, 1), dtype=torch.uint8, device="cuda")
    mb.mlora_linear(w, x, y, ws)
    mb.mlora_linear_status(w, ws)                       # raises if the device status is set
    mb.mlora_linear_status(w, None)                     # the built-in array (possibly never used yet)
    with pytest.raises(mb.MloraError) as e:             # a misaligned input is refused on the host, not faulted on
        mb.mlora_linear(w, x.view(-1)[4:4 + 3 * 256].view(3, 256), y[:3], ws)
    assert e.value.code == -1
    mb.mlora_weight_destroy(w)


def test_linear_base_wide_ragged_output(mb):
    """Enough 16 x 32 output tiles for the warp-per-tile epilogue, with a width that is not a multiple of 32 and a row
    count that is not a multiple of 16: the ragged last tiles of both directions."""
    got, want = run_linear(mb, 256, 4112, 64, 168, 0, 0, seed=11)
    compare(got, want, "linear base K256 N4112 M168")


def test_linear_lora_visible_and_b_zero_is_base(mb):
    """The low-rank term changes the result, and adapter index -1 gives the base projection exactly."""
    got_l, _ = run_linear(mb, 512, 256, 128, 8, 4, 16, seed=5, with_base_rows=False)
    got_b, want_b = run_linear(mb, 512, 256, 128, 8, 0, 0, seed=5)
    assert np.abs(got_l - got_b).max() > 1e-3 * np.abs(got_b).max()
    compare(got_b, want_b, "base")


def test_linear_rejects_bad_arguments(mb):
    rng = np.random.default_rng(0)
    qb, sc = gen.quantize_int4(rng.standard_normal((128, 64)).astype(np.float32), 64)
    with pytest.raises(mb.MloraError):
        mb.mlora_weight_create(dev(qb), dev(sc), 100, 64, 64)            # K not a multiple of 64
    w = mb.mlora_weight_create(dev(qb), dev(sc), 128, 64, 64)
    x = torch.zeros(4, 128, dtype=torch.float16, device="cuda")
    y = torch.zeros(4, 64, dtype=torch.float32, device="cuda")
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_linear(w, x, y, torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == -3
    mb.mlora_weight_destroy(w)


# ------------------------------------------------------------------ attention
def run_attention(mb, n, T, Hq, Hkv, hd, P, suf, branch, seed, cap=None):
    rng = np.random.default_rng(seed)
    cap = cap or (max(suf) + T + 3)
    q = rng.standard_normal((n * T, Hq, hd)).astype(np.float16)
    pk = rng.standard_normal((Hkv, max(P, 1), hd)).astype(np.float16)
    pv = rng.standard_normal((Hkv, max(P, 1), hd)).astype(np.float16)
    ok = rng.standard_normal((n, Hkv, cap, hd)).astype(np.float16)
    ov = rng.standard_normal((n, Hkv, cap, hd)).astype(np.float16)
    parent = gen.build_tree(branch, T) if T > 1 else np.array([-1], dtype=np.int32)
    parents = np.stack([parent] * n).astype(np.int32)
    out = torch.empty(n * T, Hq, hd, dtype=torch.float16, device="cuda")
    ws = torch.empty(mb.mlora_attention_workspace_bytes(n, T, Hq, Hkv, hd, P, cap), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mb.mlora_attention(dev(q), dev(pk[:, :P]) if P else None, dev(pv[:, :P]) if P else None, dev(ok), dev(ov),
                       dev(np.asarray(suf, dtype=np.int32)), int(max(suf)), dev(parents), out, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    f = np.float64
    suf_k = [ok[s, :, :suf[s]].transpose(1, 0, 2).astype(f) for s in range(n)]
    suf_v = [ov[s, :, :suf[s]].transpose(1, 0, 2).astype(f) for s in range(n)]
    tree_k = np.concatenate([ok[s, :, suf[s]:suf[s] + T].transpose(1, 0, 2) for s in range(n)]).astype(f)
    tree_v = np.concatenate([ov[s, :, suf[s]:suf[s] + T].transpose(1, 0, 2) for s in range(n)]).astype(f)
    want = ref.tree_attention(q.astype(f), pk[:, :P].transpose(1, 0, 2).astype(f), pv[:, :P].transpose(1, 0, 2).astype(f),
                              suf_k, suf_v, tree_k, tree_v, [list(parent)] * n)
    return out.cpu().numpy(), want


@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("n,T,branch,P,suf", [
    (4, 1, (), 128, [0, 0, 0, 0]),
    (3, 1, (), 100, [0, 5, 70]),
    (8, 1, (), 512, [3, 64, 65, 1, 127, 128, 129, 200]),
    (2, 6, (2, 2), 77, [9, 0]),
    (3, 16, (4, 2, 2), 300, [0, 63, 130]),
    (2, 64, (4, 4, 4), 65, [1, 40]),
    (2, 10, (3, 2), 0, [4, 0]),
    (3, 1, (), 0, [0, 33, 64]),          # no shared prefix: one CTA of a decode cluster may have no tile at all
    (2, 1, (), 31, [0, 1]),              # a prefix shorter than one tile
    (2, 1, (), 1500, [100, 7]),          # the longest context the single-pass kernel takes
])
def test_attention_matches_oracle(mb, hd, n, T, branch, P, suf):
    got, want = run_attention(mb, n, T, 8, 2, hd, P, suf, branch, seed=hd + n + T + P)
    compare(got, want, f"attention hd{hd} n{n} T{T} P{P}")


@pytest.mark.parametrize("n,T,branch,P,suf", [
    (2, 32, (4, 4, 2), 2048, [64, 5]),       # the 3B verify shape: 32-node trees over a 2048-token prompt
    (2, 16, (4, 2, 2), 8192, [64, 0]),       # the longest prefix of the attention sweep
])
def test_attention_tree_passes_at_long_prefixes(mb, n, T, branch, P, suf):
    got, want = run_attention(mb, n, T, 32, 8, 128, P, suf, branch, seed=P + T)
    compare(got, want, f"attention hd128 32q/8kv n{n} T{T} P{P}")


def test_attention_workspace_covers_every_suffix_bound(mb):
    """The documented workspace size must do for any suffix bound the capacity allows (the chunking, and with it the
    scratch, is not monotone in the bound): capacity 129 with bound 127 once needed more than the size planned at 128."""
    got, want = run_attention(mb, 8, 1, 32, 8, 64, 512, [127, 0, 5, 64, 100, 127, 1, 90], (), seed=9, cap=129)
    compare(got, want, "attention cap129 bound127")


@pytest.mark.parametrize("n,Hq,Hkv,hd,P,suf", [
    (8, 32, 8, 128, 8192, [0, 63, 64, 65, 200, 1, 17, 128]),     # the sweep's longest prefix: 18 chunks per kv head
    (8, 32, 8, 64, 2048, [5, 0, 64, 100, 127, 128, 129, 300]),   # two tiles per chunk at most
    (3, 24, 8, 128, 2100, [0, 40, 90]),                          # three query heads per kv head, ragged last tile
    (1, 8, 2, 64, 4099, [7]),                                    # one stream; 65 tiles on 65 chunks
    (5, 8, 8, 128, 1990, [100, 3, 64, 0, 77]),                   # just past the single-kernel limit, one head per group
    (8, 32, 8, 64, 2500, [1000, 0, 1, 2, 3, 4, 5, 6]),           # a long own segment: 16 tiles of it on one CTA
])
def test_attention_one_row_per_stream_over_long_prefix(mb, n, Hq, Hkv, hd, P, suf):
    """One decode row per stream over a prefix too long for the single-kernel path: the streaming kernel (prefix chunks
    shared by all streams' rows, tiled TMA copies) plus the merge."""
    got, want = run_attention(mb, n, 1, Hq, Hkv, hd, P, suf, (), seed=P + n)
    compare(got, want, f"attention stream hd{hd} {Hq}q/{Hkv}kv n{n} P{P}")


@pytest.mark.parametrize("K,N", [(2048, 2048), (4096, 4096), (5632, 2048), (14336, 4096), (256, 16)])
@pytest.mark.parametrize("M", [1, 3, 8, 9, 16, 31, 64])
def test_w4a8_projection_is_bit_exact(mb, K, N, M):
    """The paper's own regime (Sec. 3.3): per-channel INT4 weights x per-tensor INT8 activations.  Integer contraction and
    float32 scaling in a fixed order on both sides: compared bit for bit, the activation quantiser too."""
    rng = np.random.default_rng(K + N + M)
    qb, sc = gen.quantize_int4_per_channel(rng.standard_normal((K, N)).astype(np.float32) * 0.02)
    x = rng.standard_normal((M, K)).astype(np.float16)
    sx = float(np.float32(np.abs(x.astype(np.float32)).max() / np.float32(127)))
    d_qx = torch.empty(M, K, dtype=torch.int8, device="cuda")
    mb.mlora_quantize_act_int8(dev(x), sx, d_qx)
    qx = ref.quantize_act_int8(x, sx)
    assert np.array_equal(d_qx.cpu().numpy(), qx)
    y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    mb.mlora_linear_w4a8(dev(qb), dev(sc), d_qx, sx, y)
    torch.cuda.synchronize()
    want = ref.linear_w4a8(qx, sx, qb, sc)
    assert np.array_equal(y.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_w4a8_extreme_values_and_limits(mb):
    """Every product at its largest magnitude (-8 x -127 and -8 x 127 over K = 14336 inputs stays inside 32 bits), and
    the shapes outside the kernel's limits are refused on the host."""
    K, N, M = 14336, 16, 2
    qb = np.zeros((N, K // 2), dtype=np.uint8)                       # nibble 0 = q -8 everywhere
    sc = np.full(N, 1.0, dtype=np.float16)
    qx = np.stack([np.full(K, -127, dtype=np.int8), np.full(K, 127, dtype=np.int8)])
    y = torch.empty(M, N, dtype=torch.float32, device="cuda")
    mb.mlora_linear_w4a8(dev(qb), dev(sc), dev(qx), 1.0, y)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), ref.linear_w4a8(qx, 1.0, qb, sc))
    assert y[0, 0].item() == float(np.float32(8 * 127 * K))
    for bad in [(65, 256, 16), (1, 300, 16), (1, 256, 24)]:
        Mb, Kb, Nb = bad
        with pytest.raises(mb.MloraError) as e:
            mb.mlora_linear_w4a8(torch.zeros(Nb, Kb // 2, dtype=torch.uint8, device="cuda"), torch.ones(Nb, dtype=torch.float16, device="cuda"),
                                 torch.zeros(Mb, Kb, dtype=torch.int8, device="cuda"), 1.0, torch.empty(Mb, Nb, device="cuda"))
        assert e.value.code == -6


def test_attention_long_prefix_split(mb):
    got, want = run_attention(mb, 2, 1, 8, 2, 128, 3000, [64, 10], (), seed=3)
    compare(got, want, "attention P3000")


def test_attention_reports_malformed_tree(mb):
    n, T, Hq, Hkv, hd, P, cap = 1, 4, 4, 2, 64, 16, 16
    z = lambda *s: torch.zeros(*s, dtype=torch.float16, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(mb.mlora_attention_workspace_bytes(n, T, Hq, Hkv, hd, P, cap), dtype=torch.uint8, device="cuda")
    bad = dev(np.array([[-1, 0, 2, 1]], dtype=np.int32))                  # parent[2] = 2 is not < 2
    mb.mlora_attention(z(n * T, Hq, hd), z(Hkv, P, hd), z(Hkv, P, hd), z(n, Hkv, cap, hd), z(n, Hkv, cap, hd),
                       dev(np.zeros(1, dtype=np.int32)), 0, bad, z(n * T, Hq, hd), ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == -1
