"""Rotary position embedding of cached keys (oracle, test infrastructure).

Paper basis: Methodology, "Migration-Stable Quantization": keys are kept in the pre-RoPE domain together with
their absolute positions, and the rotation is applied again after dequantization.  The paper does not restate
the rotation itself; it is the standard one of the models it evaluates (Llama, Qwen):

    theta_i = base^(-2 i / d),  i = 0 .. d/2 - 1
    (x_i, y_i) = (k[i], k[i + d/2])          the "rotate-half" pairing of those models
    x_i' = x_i cos(p theta_i) - y_i sin(p theta_i)
    y_i' = y_i cos(p theta_i) + x_i sin(p theta_i)

for a key at absolute position p.

Readings taken where the paper is silent:
  * every stored key, full precision or low-bit, is pre-RoPE (a window must be quantizable at any routing event, and
    a promoted window holds the dequantized pre-RoPE approximation); the rotation is applied whenever attention
    reads a key; queries arrive already rotated; values are never rotated;
  * the position of slot j of window w is w * W + j (windows are contiguous and the sequence starts at 0);
  * the arithmetic is that of the models' own implementation in the execution datatype T: cos and sin are rounded
    to T, and each product and each sum of the two formulas is rounded to T on its own
    (x' = RN(RN(x c) - RN(y s)), y' = RN(RN(y c) + RN(x s))).

`rotate_exact` is the definition in float64 without any rounding; the tests pin it against complex
multiplication and the relative-position identity, and pin `apply_rope` to it within the rounding bound.
"""

import numpy as np

from .numerics import round_to_dtype


def rope_frequencies(head_dim, base):
    """theta_i = base^(-2 i / d), i < d / 2 (float64)."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    return np.power(float(base), -2.0 * i / head_dim)


def rotate_exact(k, positions, base):
    """The rotation in float64, no rounding.  k [..., n, d], positions [n] -> [..., n, d]."""
    k = np.asarray(k, dtype=np.float64)
    d = k.shape[-1]
    ang = np.outer(np.asarray(positions, dtype=np.float64), rope_frequencies(d, base))  # [n, d/2]
    c, s = np.cos(ang), np.sin(ang)
    x, y = k[..., : d // 2], k[..., d // 2 :]
    return np.concatenate([x * c - y * s, y * c + x * s], axis=-1)


def apply_rope(k, positions, base, dtype):
    """The rotation as a model computes it in the execution datatype: tables and every operation rounded to it.
    k [..., n, d] (values of `dtype` held as float64), positions [n] -> [..., n, d] (values of `dtype`)."""
    k = np.asarray(k, dtype=np.float64)
    d = k.shape[-1]
    ang = np.outer(np.asarray(positions, dtype=np.float64), rope_frequencies(d, base))
    c = round_to_dtype(np.cos(ang), dtype)
    s = round_to_dtype(np.sin(ang), dtype)
    x, y = k[..., : d // 2], k[..., d // 2 :]
    rn = lambda a: round_to_dtype(a, dtype)  # noqa: E731
    xr = rn(rn(x * c) - rn(y * s))
    yr = rn(rn(y * c) + rn(x * s))
    return np.concatenate([xr, yr], axis=-1)
