"""Pins for the oracle's rounding and quantizer: closed forms, hand-computed examples, library
routines used as independent references, and the half-step error bound."""

import os

import numpy as np
import pytest
import torch

from oracle import (
    dequantize,
    dequantize_exact,
    dequantize_window,
    quantize_groups,
    quantize_window,
    round_to_dtype,
)
from oracle.cache import OracleConfig, window_bytes

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- rounding
def test_round_fp16_matches_numpy_cast():
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(20000) * 10.0 ** rng.integers(-8, 5, 20000),
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e-8, 5.96e-8, 2.98e-8, 2.9802322387695312e-8]),
    ])
    ref = x.astype(np.float16).astype(np.float64)  # numpy rounds float64 -> float16 directly
    got = round_to_dtype(x, "fp16")
    assert np.array_equal(ref, got)


def test_round_bf16_matches_torch_on_float32_inputs():
    # torch converts float32 -> bfloat16 with round-to-nearest-even; float32 inputs avoid the
    # double -> float -> bfloat16 double rounding that a float64 source would go through.
    rng = np.random.default_rng(2)
    x32 = (rng.standard_normal(50000) * 10.0 ** rng.integers(-30, 30, 50000)).astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = round_to_dtype(x32.astype(np.float64), "bf16")
    assert np.array_equal(ref, got)


def test_round_ties_to_even_and_direct_from_double():
    # bf16 has 8 significand bits: spacing in [1, 2) is 2^-7
    u = 2.0 ** -7
    assert round_to_dtype(1.0 + u / 2, "bf16") == 1.0  # tie -> even significand
    assert round_to_dtype(1.0 + 3 * u / 2, "bf16") == 1.0 + 2 * u
    # a value just above a tie that float32 would first round onto the tie
    x = 1.0 + u / 2 + 2.0 ** -40
    assert round_to_dtype(x, "bf16") == 1.0 + u
    # fp16: 11 significand bits, spacing 2^-10 in [1, 2)
    v = 2.0 ** -10
    assert round_to_dtype(1.0 + v / 2, "fp16") == 1.0
    assert round_to_dtype(1.0 + v / 2 + 2.0 ** -40, "fp16") == 1.0 + v
    # subnormal quantum of fp16 is 2^-24
    assert round_to_dtype(1.4 * 2.0 ** -24, "fp16") == 2.0 ** -24
    assert round_to_dtype(0.5 * 2.0 ** -24, "fp16") == 0.0


# --------------------------------------------------------------------------- hand examples
def _read_examples():
    out = []
    with open(os.path.join(GOLDEN, "quant_hand_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, xs, s, z, codes, deq = [p.strip() for p in line.split("|")]
            dtype, bits = head.split()
            out.append((dtype, int(bits), np.array(xs.split(), float), float(s), float(z),
                        np.array(codes.split(), int), np.array(deq.split(), float)))
    return out


@pytest.mark.parametrize("ex", _read_examples())
def test_hand_computed_examples(ex):
    dtype, bits, x, s_ref, z_ref, codes_ref, deq_ref = ex
    codes, s, z = quantize_groups(x[None, :], bits, dtype)
    assert s[0] == s_ref and z[0] == z_ref
    assert np.array_equal(codes[0], codes_ref)
    assert np.array_equal(dequantize(codes, s, z, dtype)[0], deq_ref)


# ------------------------------------------------------------------------------ properties
def _rand_T(rng, shape, dtype, scale=1.0):
    return round_to_dtype(rng.standard_normal(shape) * scale, dtype)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [2, 4])
def test_half_step_error_bound(dtype, bits):
    rng = np.random.default_rng(3)
    for scale in (1.0, 8.0, 1e-3, 300.0):
        x = _rand_T(rng, (4000, 32), dtype, scale)
        codes, s, z = quantize_groups(x, bits, dtype)
        xhat = dequantize_exact(codes, s, z)
        err = np.abs(x - xhat)
        assert np.all(err <= (s[:, None] / 2) * (1 + 2.0 ** -20))
        assert codes.max() <= (1 << bits) - 1
        # end points: the minimum always maps to code 0, the maximum to qmax
        assert np.all(np.take_along_axis(codes, x.argmin(-1)[:, None], -1) == 0)
        assert np.all(np.take_along_axis(codes, x.argmax(-1)[:, None], -1) == (1 << bits) - 1)
        # codes are monotone in x inside a group
        order = np.argsort(x, axis=-1, kind="stable")
        assert np.all(np.diff(np.take_along_axis(codes.astype(int), order, -1), axis=-1) >= 0)
        # the value in the execution datatype is within half an ulp of the exact one
        xt = dequantize(codes, s, z, dtype)
        assert np.array_equal(xt, round_to_dtype(xhat, dtype))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [2, 4])
def test_lattice_groups_are_lossless(dtype, bits):
    rng = np.random.default_rng(4)
    qmax = (1 << bits) - 1
    for _ in range(200):
        s = 2.0 ** rng.integers(-6, 3)  # power of two: representable, and qmax*s/qmax is exact
        z = float(rng.integers(-8, 8)) * s
        j = rng.integers(0, qmax + 1, 32)
        j[0], j[1] = 0, qmax
        x = z + j * s
        codes, s_out, z_out = quantize_groups(x[None], bits, dtype)
        assert s_out[0] == s and z_out[0] == z
        assert np.array_equal(codes[0], j)
        assert np.array_equal(dequantize(codes, s_out, z_out, dtype)[0], x)


def test_two_valued_group_uses_end_codes():
    x = np.array([[0.5, -2.0, 0.5, 0.5, -2.0, -2.0, 0.5, -2.0]])
    for bits in (2, 4):
        codes, s, z = quantize_groups(x, bits, "bf16")
        assert set(np.unique(codes)) == {0, (1 << bits) - 1}


def test_degenerate_groups():
    x = np.full((3, 32), -7.25)
    codes, s, z = quantize_groups(x, 4, "fp16")
    assert np.all(codes == 0) and np.all(s == 1.0) and np.all(z == -7.25)
    assert np.array_equal(dequantize(codes, s, z, "fp16"), x)
    # a range so small that the scale underflows to zero in fp16
    tiny = np.array([[0.0, 2.0 ** -24] * 16])
    codes, s, z = quantize_groups(tiny, 4, "fp16")
    assert np.all(codes == 0) and s[0] == 1.0


# ------------------------------------------------------------------- window axes (K vs V)
def test_key_groups_run_over_tokens_value_groups_over_channels():
    """Keys: per channel across tokens; values: per token across channels (Methodology).
    A key tensor that is constant along tokens and a value tensor that is constant along channels are
    both reproduced exactly; swapping the axes in either would not be."""
    rng = np.random.default_rng(5)
    h, w, d, g = 2, 32, 64, 32
    per_channel = _rand_T(rng, (h, 1, d), "bf16", 4.0)
    per_token = _rand_T(rng, (h, w, 1), "bf16", 4.0)
    k = np.broadcast_to(per_channel, (h, w, d)).copy()
    v = np.broadcast_to(per_token, (h, w, d)).copy()
    e = quantize_window(k, v, 2, g, "bf16")
    assert e["k_s"].shape == (h, w // g, d) and e["v_s"].shape == (h, w, d // g)
    assert np.all(e["k_codes"] == 0) and np.all(e["v_codes"] == 0)
    kk, vv = dequantize_window(e, g, "bf16")
    assert np.array_equal(kk, k) and np.array_equal(vv, v)
    # the swapped tensors are not constant inside their groups, so they are lossy at 2 bits
    e2 = quantize_window(v, k, 2, g, "bf16")
    kk2, vv2 = dequantize_window(e2, g, "bf16")
    assert not np.array_equal(kk2, v) and not np.array_equal(vv2, k)


def test_window_roundtrip_matches_per_group_definition():
    """quantize_window must equal the per-group routine applied group by group with explicit loops."""
    rng = np.random.default_rng(6)
    h, w, d, g, bits = 2, 64, 64, 32, 4
    k = _rand_T(rng, (h, w, d), "fp16")
    v = _rand_T(rng, (h, w, d), "fp16")
    e = quantize_window(k, v, bits, g, "fp16")
    for hh in range(h):
        for blk in range(w // g):
            for c in range(0, d, 7):
                codes, s, z = quantize_groups(k[hh, blk * g:(blk + 1) * g, c][None], bits, "fp16")
                assert np.array_equal(codes[0], e["k_codes"][hh, blk * g:(blk + 1) * g, c])
                assert s[0] == e["k_s"][hh, blk, c] and z[0] == e["k_z"][hh, blk, c]
        for t in range(0, w, 5):
            for blk in range(d // g):
                codes, s, z = quantize_groups(v[hh, t, blk * g:(blk + 1) * g][None], bits, "fp16")
                assert np.array_equal(codes[0], e["v_codes"][hh, t, blk * g:(blk + 1) * g])
                assert s[0] == e["v_s"][hh, t, blk] and z[0] == e["v_z"][hh, t, blk]


# ------------------------------------------------------------------------ byte accounting
def test_int2_window_costs_three_sixteenths_of_fp16_paper_operating_points():
    """The paper's conditions R3 and R4 are two complete operating points at one measured budget; they
    are consistent with each other only if an INT2 window costs 3/16 of a 16-bit window."""
    pts = {}
    with open(os.path.join(GOLDEN, "paper_operating_points.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, w, kf, kq, sink, prefill, frac = line.split()
                pts[name] = (int(w), int(kf), int(kq), int(sink), int(prefill), float(frac))
    cfg = OracleConfig(32, 8, 128, "fp16", 32, 2, 32, 1, 1, 4096)
    m_f, m_q = window_bytes(cfg)
    assert m_q * 16 == m_f * 3
    totals = []
    for w, kf, kq, sink, prefill, frac in pts.values():
        totals.append(kf * w + kq * w * m_q / m_f + sink)  # in full-precision token equivalents
        assert abs(totals[-1] - np.ceil(frac * prefill)) < 1e-9
    assert totals[0] == totals[1]
