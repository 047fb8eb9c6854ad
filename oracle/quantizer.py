"""Asymmetric low-bit window quantizer (oracle, test infrastructure).

Paper basis (Methodology, "Migration-Stable Quantization"): a window entering
the quantized tier is quantized asymmetrically at low bit width; keys per
channel across the token dimension, values per token across the channel
dimension; promotion reconstructs the same low-bit approximation in the
execution datatype.  The paper does not state group size, parameter storage or
rounding; the readings taken here:

  * a group is `g` consecutive elements along the grouped axis (tokens for K,
    channels for V), always inside one window;
  * parameters are the pair (scale s, zero z) stored in the execution datatype:
    z = min of the group, s = RNE_T((max - min) / qmax) with the subtraction and
    the division done in IEEE float32;
  * code = clamp(rint((x - z) / s), 0, qmax), subtraction and division in IEEE
    float32, rint = round half to even;
  * a group whose scale is not a positive finite number gets s = 1 and all
    codes 0;
  * the dequantized value is x~ = RNE_T(code * s + z), the product and sum taken
    exactly before the single rounding.

All tensors are float64 arrays holding values representable in the execution
datatype; codes are uint8.
"""

import numpy as np

from .numerics import round_to_dtype


def quantize_groups(x, bits, dtype):
    """Quantize groups laid along the last axis of `x`.

    Returns (codes uint8 same shape as x, s float64 [...], z float64 [...]).
    """
    x = np.asarray(x, dtype=np.float64)
    qmax = (1 << bits) - 1
    mn = x.min(axis=-1)
    mx = x.max(axis=-1)
    r32 = mx.astype(np.float32) - mn.astype(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        s32 = r32 / np.float32(qmax)
    s = round_to_dtype(s32.astype(np.float64), dtype)
    z = mn.copy()
    bad = ~(s > 0) | ~np.isfinite(s)
    s = np.where(bad, 1.0, s)
    x32 = x.astype(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        t = (x32 - z.astype(np.float32)[..., None]) / s.astype(np.float32)[..., None]
    c = np.clip(np.rint(t), 0, qmax)
    c = np.where(bad[..., None], 0, c)
    return c.astype(np.uint8), s, z


def dequantize_exact(codes, s, z):
    """Exact dequantized value code*s + z along the last axis groups (no rounding to the datatype)."""
    return codes.astype(np.float64) * np.asarray(s)[..., None] + np.asarray(z)[..., None]


def dequantize(codes, s, z, dtype):
    """x~ = RNE_T(code*s + z): the value attention uses and promotion writes."""
    return round_to_dtype(dequantize_exact(codes, s, z), dtype)


def quantize_window(k, v, bits, group, dtype):
    """Quantize one window.  k, v: [H_kv, W, d].

    Keys: one group per (head, channel, block of `group` tokens).
    Values: one group per (head, token, block of `group` channels).
    Returns a dict with
      k_codes, v_codes : uint8 [H_kv, W, d]
      k_s, k_z         : float64 [H_kv, W/group, d]
      v_s, v_z         : float64 [H_kv, W, d/group]
    """
    h, w, d = k.shape
    assert w % group == 0 and d % group == 0
    # keys: bring the token axis last, split into blocks of `group` tokens
    kt = np.transpose(k, (0, 2, 1)).reshape(h, d, w // group, group)  # [h, d, blocks, g]
    kc, ks, kz = quantize_groups(kt, bits, dtype)
    k_codes = np.transpose(kc.reshape(h, d, w), (0, 2, 1))
    k_s = np.transpose(ks, (0, 2, 1))  # [h, blocks, d]
    k_z = np.transpose(kz, (0, 2, 1))
    # values: channel axis already last
    vt = v.reshape(h, w, d // group, group)
    vc, vs, vz = quantize_groups(vt, bits, dtype)
    v_codes = vc.reshape(h, w, d)
    return {
        "k_codes": np.ascontiguousarray(k_codes),
        "k_s": np.ascontiguousarray(k_s),
        "k_z": np.ascontiguousarray(k_z),
        "v_codes": np.ascontiguousarray(v_codes),
        "v_s": vs,
        "v_z": vz,
    }


def dequantize_window(entry, group, dtype):
    """Inverse of quantize_window: returns (k~, v~) as [H_kv, W, d] in the execution datatype."""
    k_codes, v_codes = entry["k_codes"], entry["v_codes"]
    h, w, d = k_codes.shape
    kc = np.transpose(k_codes, (0, 2, 1)).reshape(h, d, w // group, group)
    ks = np.transpose(entry["k_s"], (0, 2, 1))
    kz = np.transpose(entry["k_z"], (0, 2, 1))
    k = dequantize(kc, ks, kz, dtype).reshape(h, d, w)
    k = np.ascontiguousarray(np.transpose(k, (0, 2, 1)))
    vc = v_codes.reshape(h, w, d // group, group)
    v = dequantize(vc, entry["v_s"], entry["v_z"], dtype).reshape(h, w, d)
    return k, v
