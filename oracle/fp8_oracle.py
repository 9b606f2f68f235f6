"""CPU oracle of the reduced-precision (FP8) variant of the encoder layer's linear maps.

TEST INFRASTRUCTURE ONLY, like mt_oracle.py: plain numpy, no code shared with the CUDA path, never
called from the product path.

The paper's production model ran at reduced precision (Appendix E: half precision with a fast
transformer library on its GPUs); it prints no quantisation recipe.  The reading taken here for the
8-bit path:

* format E4M3 ("fn" flavour: 1 sign, 4 exponent bits with bias 7, 3 mantissa bits, subnormals,
  no infinities, largest finite value 448, the all-ones pattern is NaN);
* what is quantised: both operands of the Q/K/V projection, of the FFN-up projection and of the
  FFN-down projection.  The attention-output projection, attention itself, LayerNorm, the residual
  stream, pooler and heads stay as they are;
* granularity: one scale per ROW of each operand - per token for activations [rows, K], per output
  channel for weights [N, K] - so a product is  (sum_k a_q w_q) * s_a[row] * s_w[col];
* scale = amax * (1 / 448) (a row of zeros gets scale 1), value / scale rounded to the nearest E4M3
  value, ties to the even mantissa, saturating at +-448.  These three steps are DECISIONS that produce
  integer codes, so they are taken in float32, the precision the kernels take them in; everything after
  them (the products and sums of the decoded values) is float64.

Pins (tests/test_oracle_fp8.py): every finite code decodes and re-encodes to itself; table values
(1.0, 448, the smallest normal and subnormal); midpoints go to the even neighbour; saturation; the
vectorised encoder against a scalar brute-force search over all 256 codes; agreement with torch's own
float8_e4m3fn cast inside the finite range; the largest magnitude of a row always maps to +-448.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np

from . import mt_oracle as base

E4M3_MAX = 448.0


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 E4M3 codes -> float64 values (NaN for the two all-ones patterns)."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    exp = (c >> 3) & 0xF
    man = (c & 0x7).astype(np.float64)
    normal = (1.0 + man / 8.0) * np.exp2(exp.astype(np.float64) - 7.0)
    sub = (man / 8.0) * 2.0 ** -6
    val = np.where(exp == 0, sub, normal)
    val = np.where((c & 0x7F) == 0x7F, np.nan, val)
    return sign * val


def e4m3_encode(y: np.ndarray) -> np.ndarray:
    """float32 values -> uint8 E4M3 codes: nearest representable value, ties to the even mantissa,
    magnitudes beyond 448 saturate to 448.  The sign of zero is kept."""
    y = np.asarray(y, dtype=np.float32)
    a = np.abs(y).astype(np.float64)                     # float32 values are exact in float64
    neg = np.signbit(y)
    # spacing of the E4M3 grid around a: 2^(e - 3) in the binade 2^e, never finer than the subnormal step 2^-9
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -20)))
    e = np.clip(e, -6.0, 8.0)
    step = np.exp2(e - 3.0)
    q = np.rint(a / step) * step                         # np.rint rounds halves to even, a / step is exact
    q = np.minimum(q, E4M3_MAX)
    # value -> code
    qe = np.floor(np.log2(np.maximum(q, 2.0 ** -20)))
    is_sub = q < 2.0 ** -6
    man_sub = np.rint(q / 2.0 ** -9)
    man_nor = np.rint(q / np.exp2(np.clip(qe, -6.0, 8.0) - 3.0)) - 8.0
    code = np.where(is_sub, man_sub, (np.clip(qe, -6.0, 8.0) + 7.0) * 8.0 + man_nor)
    code = np.where(q == 0.0, 0.0, code).astype(np.int64)
    return (code | np.where(neg, 0x80, 0)).astype(np.uint8)


def quantize_rows(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """One scale per row of ``x`` [rows, K]: returns (codes uint8 [rows, K], scale float32 [rows]).
    All three decisions in float32: amax, scale = amax * (1/448), code = encode(x / scale)."""
    x32 = np.asarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=-1)
    scale = (amax * np.float32(1.0 / 448.0)).astype(np.float32)
    scale = np.where(amax == 0, np.float32(1.0), scale).astype(np.float32)
    y = (x32 / scale[..., None]).astype(np.float32)
    return e4m3_encode(y), scale


def dequantize_rows(codes: np.ndarray, scale: np.ndarray) -> np.ndarray:
    return e4m3_decode(codes) * np.asarray(scale, dtype=np.float64)[..., None]


def linear_fp8(x: np.ndarray, w: np.ndarray, b: np.ndarray) -> np.ndarray:
    """y = Q(x) Q(W)^T + b with both operands quantised row by row (x per token, W per output channel)."""
    xq, sx = quantize_rows(x)
    wq, sw = quantize_rows(w)
    return dequantize_rows(xq, sx) @ dequantize_rows(wq, sw).T + b


def attention_fp8(h: np.ndarray, layer: Dict[str, np.ndarray], heads: int) -> np.ndarray:
    """Self-attention whose Q/K/V projection is the 8-bit one (one activation scale per token, shared by
    the three projections since they read the same operand); the attention arithmetic itself is unchanged."""
    n, H = h.shape
    dh = H // heads
    q = linear_fp8(h, layer["wq"], layer["bq"])
    k = linear_fp8(h, layer["wk"], layer["bk"])
    v = linear_fp8(h, layer["wv"], layer["bv"])
    ctx = np.empty((n, H), dtype=np.float64)
    for a in range(heads):
        cols = slice(a * dh, (a + 1) * dh)
        scores = (q[:, cols] @ k[:, cols].T) / np.sqrt(float(dh))
        ctx[:, cols] = base.softmax_rows(scores) @ v[:, cols]
    return ctx


def encoder_layer_fp8(h: np.ndarray, layer: Dict[str, np.ndarray], heads: int, eps: float) -> np.ndarray:
    """The post-LN encoder layer with the 8-bit Q/K/V, FFN-up and FFN-down projections."""
    ctx = attention_fp8(h, layer, heads)
    h1 = base.layer_norm(h + base.linear(ctx, layer["wo"], layer["bo"]), layer["ln1_g"], layer["ln1_b"], eps)
    f = base.gelu(linear_fp8(h1, layer["w1"], layer["b1"]))
    return base.layer_norm(h1 + linear_fp8(f, layer["w2"], layer["b2"]), layer["ln2_g"], layer["ln2_b"], eps)
