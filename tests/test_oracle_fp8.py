"""Pins of the reduced-precision (E4M3) oracle: the code table, the rounding rule, saturation,
the row-wise scaling - each against something that is not the oracle's own formula."""
import itertools

import numpy as np
import torch

from oracle import fp8_oracle as f8
from oracle import mt_oracle as orc


def scalar_decode(code: int) -> float:
    """E4M3 as its definition reads: sign, 4 exponent bits (bias 7), 3 mantissa bits, subnormals."""
    s = -1.0 if code & 0x80 else 1.0
    e, m = (code >> 3) & 0xF, code & 7
    if e == 15 and m == 7:
        return float("nan")
    return s * (m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))


def brute_force_encode(y: float) -> int:
    """Nearest finite code by exhaustive search; ties to the even mantissa; beyond 448 the largest."""
    best, best_d = None, None
    for code in range(0x7F):                      # non-negative finite codes
        d = abs(abs(y) - scalar_decode(code))
        if best is None or d < best_d or (d == best_d and code % 2 == 0 and best % 2 == 1):
            best, best_d = code, d
    return best | (0x80 if np.signbit(np.float32(y)) else 0)


def test_code_table_matches_the_format_definition():
    codes = np.arange(256, dtype=np.uint8)
    got = f8.e4m3_decode(codes)
    want = np.array([scalar_decode(int(c)) for c in codes])
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[~np.isnan(got)], want[~np.isnan(want)])
    # values anyone can check by hand
    assert f8.e4m3_decode(np.uint8(0x38)) == 1.0
    assert f8.e4m3_decode(np.uint8(0x7E)) == 448.0            # largest finite
    assert f8.e4m3_decode(np.uint8(0x08)) == 2.0 ** -6        # smallest normal
    assert f8.e4m3_decode(np.uint8(0x01)) == 2.0 ** -9        # smallest subnormal
    assert f8.e4m3_decode(np.uint8(0xC0)) == -2.0
    assert np.isnan(f8.e4m3_decode(np.uint8(0x7F))) and np.isnan(f8.e4m3_decode(np.uint8(0xFF)))


def test_every_finite_code_round_trips():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = f8.e4m3_decode(codes).astype(np.float32)
    assert np.array_equal(f8.e4m3_encode(vals), codes)       # -0.0 keeps its sign bit


def test_midpoints_round_to_the_even_mantissa_and_large_values_saturate():
    pos = [scalar_decode(c) for c in range(0x7F)]
    for lo, hi in zip(range(0x7E), range(1, 0x7F)):
        mid = np.float32((pos[lo] + pos[hi]) / 2.0)           # exact in float32
        want = lo if lo % 2 == 0 else hi
        assert int(f8.e4m3_encode(mid)) == want, (lo, hi)
        assert int(f8.e4m3_encode(-mid)) == (want | 0x80)
        assert int(f8.e4m3_encode(np.nextafter(mid, np.float32(0)))) == lo
        assert int(f8.e4m3_encode(np.nextafter(mid, np.float32(1e9)))) == hi
    for big in (448.0, 449.0, 464.0, 480.0, 1e4, 3e38):
        assert int(f8.e4m3_encode(np.float32(big))) == 0x7E
        assert int(f8.e4m3_encode(np.float32(-big))) == 0xFE
    assert int(f8.e4m3_encode(np.float32(0.0))) == 0 and int(f8.e4m3_encode(np.float32(-0.0))) == 0x80
    assert int(f8.e4m3_encode(np.float32(2.0 ** -10))) == 0   # half the smallest subnormal: tie to even (zero)
    assert int(f8.e4m3_encode(np.float32(2.0 ** -10 * 1.01))) == 1


def test_encoder_against_exhaustive_search_and_a_library_cast():
    rng = np.random.default_rng(5)
    y = np.concatenate([rng.standard_normal(300) * s for s in (1e-3, 0.02, 1.0, 40.0, 300.0)]).astype(np.float32)
    got = f8.e4m3_encode(y)
    want = np.array([brute_force_encode(float(v)) for v in y], dtype=np.uint8)
    assert np.array_equal(got, want)
    # inside the finite range torch's float8_e4m3fn cast is the same rounding
    big = np.clip((rng.standard_normal(200000) * 120.0).astype(np.float32), -448.0, 448.0)
    lib = torch.from_numpy(big).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(f8.e4m3_encode(big), lib)


def test_row_scaling_maps_the_largest_magnitude_to_448_and_bounds_the_error():
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((64, 768)) * rng.uniform(0.01, 30.0, (64, 1))).astype(np.float32)
    x[3] = 0.0                                                # a row of zeros: scale 1, codes 0
    codes, scale = f8.quantize_rows(x)
    assert codes.dtype == np.uint8 and scale.dtype == np.float32
    amax_pos = np.argmax(np.abs(x), axis=1)
    for r in range(64):
        if r == 3:
            assert scale[r] == 1.0 and not codes[r].any()
            continue
        assert (int(codes[r, amax_pos[r]]) & 0x7F) == 0x7E
        assert scale[r] == np.float32(np.abs(x[r]).max()) * np.float32(1.0 / 448.0)
    back = f8.dequantize_rows(codes, scale)
    # relative spacing of E4M3 is 2^-3 within a binade: half of it bounds the rounding error of normal values,
    # the subnormal step (2^-9 of the scale) the rest
    bound = np.abs(x) * 2.0 ** -4 + scale[:, None].astype(np.float64) * 2.0 ** -10
    assert np.all(np.abs(back - x) <= bound * (1 + 1e-6))
    # scaling a row by a power of two scales the scale and leaves the codes alone
    codes2, scale2 = f8.quantize_rows(x * np.float32(4.0))
    assert np.array_equal(codes2, codes) and np.array_equal(scale2[np.arange(64) != 3], scale[np.arange(64) != 3] * 4)


def test_fp8_linear_is_the_product_of_the_decoded_operands_and_close_to_the_exact_one():
    rng = np.random.default_rng(9)
    x = rng.standard_normal((5, 64))
    w = rng.standard_normal((7, 64)) * 0.05
    b = rng.standard_normal(7) * 0.1
    got = f8.linear_fp8(x, w, b)
    xq, sx = f8.quantize_rows(x)
    wq, sw = f8.quantize_rows(w)
    want = np.zeros((5, 7))
    for i, j in itertools.product(range(5), range(7)):        # scalar loops, decoded values by the table
        acc = 0.0
        for k in range(64):
            acc += scalar_decode(int(xq[i, k])) * scalar_decode(int(wq[j, k]))
        want[i, j] = acc * float(sx[i]) * float(sw[j]) + b[j]
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    exact = orc.linear(x, w, b)
    assert np.linalg.norm(got - exact) / np.linalg.norm(exact) < 0.06     # two operands at 2^-4 each, at most


def test_fp8_layer_stays_close_to_the_exact_layer():
    rng = np.random.default_rng(11)
    H, F, n = 128, 256, 9

    def mat(*shape):
        return rng.standard_normal(shape) * 0.05

    layer = {"wq": mat(H, H), "wk": mat(H, H), "wv": mat(H, H), "bq": mat(H), "bk": mat(H), "bv": mat(H),
             "wo": mat(H, H), "bo": mat(H), "ln1_g": 1 + mat(H), "ln1_b": mat(H), "w1": mat(F, H), "b1": mat(F),
             "w2": mat(H, F), "b2": mat(H), "ln2_g": 1 + mat(H), "ln2_b": mat(H)}
    h = rng.standard_normal((n, H))
    exact = orc.encoder_layer(h, layer, 2, 1e-12)
    low = f8.encoder_layer_fp8(h, layer, 2, 1e-12)
    err = np.linalg.norm(low - exact) / np.linalg.norm(exact)
    assert 0 < err < 0.05
