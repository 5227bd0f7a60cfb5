"""The allocation-free projection entry point (collected last on purpose: every other test has run by then).

mlora_linear_noalloc serves callers that must not allocate device memory at the moment they issue work -- a
serving loop that reserved its memory up front, code without an allocator at hand.  It must give what
mlora_linear gives on the same inputs, also on a second call in a row (the built-in scratch is shared by all
calls and keeps the previous call's contents).  Both are also held against the CPU oracle's projection."""
import numpy as np
import pytest

import gen
from oracle import ref
from tests.helpers import compare

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_noalloc_linear_matches_linear_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2604_18655_b200 import binding as mb
    mb.lib()
    K, N, G, M, n_ad, rank = 2048, 1040, 128, 8, 5, 16
    rng = np.random.default_rng(11)
    qb, sc = gen.quantize_int4(rng.standard_normal((K, N)).astype(np.float32) * 0.02, G)
    w = mb.mlora_weight_create(dev(qb), dev(sc), K, N, G)
    hA = [(rng.standard_normal((rank, K)) / rank).astype(np.float16) for _ in range(n_ad)]
    hB = [(rng.standard_normal((rank, N)) * 0.05).astype(np.float16) for _ in range(n_ad)]
    A, B = [dev(a) for a in hA], [dev(b) for b in hB]
    Wd = ref.dequant(qb, sc, G).astype(np.float64)
    hscale = (16.0 / rank * (1 + 0.25 * np.arange(n_ad))).astype(np.float32)
    pa = torch.tensor([t.data_ptr() for t in A], dtype=torch.int64, device="cuda")
    pb = torch.tensor([t.data_ptr() for t in B], dtype=torch.int64, device="cuda")
    scale = dev((16.0 / rank * (1 + 0.25 * np.arange(n_ad))).astype(np.float32))
    ws = torch.zeros(mb.mlora_linear_workspace_bytes(w, M, rank), dtype=torch.uint8, device="cuda")
    for call in range(2):
        hx = rng.standard_normal((M, K)).astype(np.float16)
        hrows = rng.integers(-1, n_ad, size=M).astype(np.int32)
        x, rows = dev(hx), dev(hrows)
        want = torch.empty(M, N, dtype=torch.float32, device="cuda")
        got = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
        mb.mlora_linear(w, x, want, ws, rows, pa, pb, scale, rank)
        mb.mlora_linear_noalloc(w, x, got, rows, pa, pb, scale, rank)
        torch.cuda.synchronize()
        compare(got.cpu().numpy(), want.cpu().numpy(), f"noalloc call {call}")
        oracle = ref.linear_lora(hx.astype(np.float64), Wd, hrows, [a.astype(np.float64) for a in hA],
                                 [b.astype(np.float64) for b in hB], hscale.astype(np.float64))
        compare(got.cpu().numpy(), oracle, f"noalloc call {call} against the oracle")
        mb.mlora_linear_status(w, None)                  # no bounded wait ran out
    # base projection (no adapters) and the size limit
    x = dev(rng.standard_normal((3, K)).astype(np.float16))
    want = torch.empty(3, N, dtype=torch.float32, device="cuda")
    got = torch.empty(3, N, dtype=torch.float32, device="cuda")
    mb.mlora_linear(w, x, want, ws)
    mb.mlora_linear_noalloc(w, x, got)
    torch.cuda.synchronize()
    compare(got.cpu().numpy(), want.cpu().numpy(), "noalloc base")
    with pytest.raises(mb.MloraError) as e:
        mb.mlora_linear_noalloc(w, dev(np.zeros((9, K), dtype=np.float16)), torch.empty(9, N, dtype=torch.float32, device="cuda"))
    assert e.value.code == -3
    mb.mlora_weight_destroy(w)
