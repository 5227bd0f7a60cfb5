"""Pins for the oracle's INT4 x INT8 projection (Sec. 3.3 "LLM Quantization": activations per-tensor to Int8, weights
per-channel to Int4)."""
from fractions import Fraction

import numpy as np

import gen
from oracle import ref


def test_per_channel_packing_by_hand():
    """Two channels, four inputs: w[:, 0] = (7, -7, 3.5, 0) -> scale 1, q = (7, -7, 4, 0) (3.5 rounds to even 4);
    w[:, 1] = 0 -> scale 1, q = 0.  Bytes are channel-major, even k in the low nibble, nibble = q + 8."""
    w = np.array([[7.0, 0.0], [-7.0, 0.0], [3.5, 0.0], [0.0, 0.0]], dtype=np.float32)
    qb, sc = gen.quantize_int4_per_channel(w)
    assert qb.shape == (2, 2) and sc.shape == (2,)
    assert list(sc) == [1.0, 1.0]
    assert list(qb[0]) == [(7 + 8) | ((-7 + 8) << 4), (4 + 8) | ((0 + 8) << 4)]
    assert list(qb[1]) == [0x88, 0x88]


def test_activation_quantiser_rounding_and_clipping():
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 126.6, 127.4, 200.0, -300.0, 0.49], dtype=np.float16)
    assert list(ref.quantize_act_int8(x, 1.0)) == [0, 2, 2, 0, -2, 127, 127, 127, -127, 0]      # half to even, +-127
    assert list(ref.quantize_act_int8(np.array([1.0, -3.0], dtype=np.float16), 0.5)) == [2, -6]


def test_projection_against_python_integers():
    """Every product and sum in arbitrary-precision Python integers, the scaling as exact fractions, then ONE rounding
    to float32 per factor as the definition says."""
    rng = np.random.default_rng(0)
    K, N, M = 16, 6, 3
    qb, sc = gen.quantize_int4_per_channel(rng.standard_normal((K, N)).astype(np.float32))
    qx = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
    sx = 0.0371
    got = ref.linear_w4a8(qx, sx, qb, sc)
    assert got.dtype == np.float32
    for m in range(M):
        for n in range(N):
            acc = 0
            for k in range(K):
                byte = int(qb[n, k // 2])
                q = ((byte >> 4) if k % 2 else (byte & 15)) - 8
                acc += int(qx[m, k]) * q
            f = np.float32(sx) * np.float32(sc[n])                      # float32 product of the two scales
            want = np.float32(acc) * f
            assert got[m, n] == want
            exact = Fraction(acc) * Fraction(float(np.float32(sx))) * Fraction(float(sc[n]))
            assert abs(Fraction(float(got[m, n])) - exact) <= abs(exact) * Fraction(1, 2 ** 22)   # two float32 roundings


def test_projection_is_the_product_of_the_dequantised_operands():
    rng = np.random.default_rng(1)
    K, N, M = 256, 48, 5
    w = rng.standard_normal((K, N)).astype(np.float32) * 0.02
    qb, sc = gen.quantize_int4_per_channel(w)
    x = rng.standard_normal((M, K)).astype(np.float16)
    sx = float(np.abs(x.astype(np.float32)).max() / 127)
    qx = ref.quantize_act_int8(x, sx)
    y = ref.linear_w4a8(qx, sx, qb, sc)
    wd = (ref.unpack_int4(qb).astype(np.float64) * sc.astype(np.float64)[:, None]).T          # [K][N]
    xd = qx.astype(np.float64) * float(np.float32(sx))
    np.testing.assert_allclose(y, xd @ wd, rtol=1e-6, atol=1e-9)
    # and it approximates the unquantised product within the quantisers' error bound:
    # |x - xd| <= sx / 2, |w - wd| <= scale / 2 per element
    exact = x.astype(np.float64) @ w.astype(np.float64)
    bound = (np.abs(x.astype(np.float64)) @ np.tile(sc.astype(np.float64) / 2, (K, 1))
             + (sx / 2) * np.abs(wd).sum(axis=0)[None, :] + 1e-6)
    assert np.all(np.abs(y - exact) <= bound)


def test_planted_mistakes_fail():
    rng = np.random.default_rng(2)
    K, N, M = 32, 8, 2
    qb, sc = gen.quantize_int4_per_channel(rng.standard_normal((K, N)).astype(np.float32))
    qx = rng.integers(-127, 128, size=(M, K)).astype(np.int8)
    y = ref.linear_w4a8(qx, 0.1, qb, sc)
    swapped = ((qb & 15) << 4) | (qb >> 4)                            # nibbles in the wrong order
    assert not np.allclose(ref.linear_w4a8(qx, 0.1, swapped, sc), y)
    assert not np.allclose(ref.linear_w4a8(qx, 0.1, qb, sc[::-1].copy()), y)     # scales applied to the wrong channels
