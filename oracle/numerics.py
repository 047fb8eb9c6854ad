"""Rounding of float64 values to the model's execution datatype (oracle, test infrastructure).

The paper stores full-precision windows "in the model's execution datatype"
(Methodology, Migration-Stable Quantization) without fixing it; the workloads
use fp16 and bf16.  The oracle carries every tensor as float64 holding values
that are exactly representable in that datatype, and rounds with the function
below wherever the method produces a value in the execution datatype.

The rounding is done from first principles (scale to the unit in the last place,
round half to even, scale back), directly from float64, so that no intermediate
float32 rounding can occur.
"""

import numpy as np

# name -> (significand bits including the implicit one, exponent of the smallest normal, largest finite)
DTYPES = {
    "fp16": (11, -14, 65504.0),
    "bf16": (8, -126, float.fromhex("0x1.fep127")),
}


def round_to_dtype(x, dtype):
    """Round-to-nearest-even of float64 `x` to `dtype` ("fp16" or "bf16"); result is float64.

    Subnormals of the target type are kept (fixed quantum below the smallest
    normal); magnitudes that round past the largest finite value become inf.
    """
    sig_bits, emin, fmax = DTYPES[dtype]
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)  # x = m * 2**e with 0.5 <= |m| < 1, so the leading bit has weight 2**(e-1)
    lead = np.maximum(e - 1, emin)  # exponent of the binade (clamped: subnormal range)
    quantum_exp = lead - (sig_bits - 1)
    scaled = np.ldexp(x, -quantum_exp)  # exact: power-of-two scaling
    r = np.ldexp(np.rint(scaled), quantum_exp)  # np.rint rounds half to even
    r = np.where(np.abs(r) > fmax, np.copysign(np.inf, r), r)
    r = np.where(np.isfinite(x), r, x)
    return r
