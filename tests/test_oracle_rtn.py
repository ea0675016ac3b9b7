"""Pins for the oracle's group quantizer and packed format (CPU only).

None of these re-types the oracle's formula: they check the quantizer against
an exhaustive nearest-level search, against structural identities, and
against bounds that follow from the definition.
"""
import os

import numpy as np
import pytest

from oracle import adadim_oracle as O

RNG = np.random.default_rng(1234)


def _levels(s, z, bits):
    return [float(s) * (c - float(z)) for c in range(2 ** bits)]


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_codes_are_the_nearest_level_brute_force(bits, dim):
    g = 4
    W = (RNG.standard_normal((8, 12)) * 0.02).astype(np.float32)
    r = O.quantize_rtn(W, bits, g, dim)
    S = r["scales"].astype(np.float64)
    Z = r["zeros"].astype(np.float64)
    for o in range(8):
        for i in range(12):
            s, z = (S[o, i // g], Z[o, i // g]) if dim == "oc" else (S[o // g, i], Z[o // g, i])
            lv = _levels(s, z, bits)
            best = min(range(2 ** bits), key=lambda c: abs(float(W[o, i]) - lv[c]))
            assert r["codes"][o, i] == best
            assert r["Q"][o, i] == np.float32(lv[best])


@pytest.mark.parametrize("bits", [3, 4])
def test_group_parameters_cover_the_range(bits):
    maxq = 2 ** bits - 1
    W = (RNG.standard_normal((16, 256)) * 0.05).astype(np.float32)
    r = O.quantize_rtn(W, bits, 64, "oc")
    G = W.reshape(16, 4, 64).astype(np.float64)
    lo = np.minimum(G.min(2), 0.0)
    hi = np.maximum(G.max(2), 0.0)
    s = r["scales"].astype(np.float64)
    z = r["zeros"].astype(np.float64)
    # the stored scale is the fp16 rounding of range / maxq
    assert np.all(np.abs(s * maxq - (hi - lo)) <= (hi - lo) * 2.0 ** -11 * 1.0001)
    # zero point is an integer in range, and the grid origin sits within half a step of lo
    assert np.all(z == np.round(z)) and z.min() >= 0 and z.max() <= maxq
    assert np.all(np.abs(-z * s - lo) <= 0.5 * s * 1.0001)
    # a weight equal to zero is reproduced exactly
    W0 = W.copy()
    W0[:, ::7] = 0.0
    r0 = O.quantize_rtn(W0, bits, 64, "oc")
    assert np.all(r0["Q"][:, ::7] == 0.0)


@pytest.mark.parametrize("bits,group", [(3, 128), (4, 128), (3, 64), (4, 32)])
def test_transpose_identity(bits, group):
    """Per-IC quantization of W is per-OC quantization of W^T, transposed (Section 3.2)."""
    W = (RNG.standard_normal((256, 384)) * 0.02).astype(np.float32)
    W[3, :] *= 20.0
    W[:, 5] *= 30.0
    a = O.quantize_rtn(W, bits, group, "ic")
    b = O.quantize_rtn(np.ascontiguousarray(W.T), bits, group, "oc")
    assert np.array_equal(a["codes"], b["codes"].T)
    assert np.array_equal(a["scales"].view(np.uint16), b["scales"].T.view(np.uint16))
    assert np.array_equal(a["zeros"].view(np.uint16), b["zeros"].T.view(np.uint16))
    assert np.array_equal(a["Q"], b["Q"].T)


@pytest.mark.parametrize("bits", [3, 4])
@pytest.mark.parametrize("dim", ["oc", "ic"])
def test_error_bound(bits, dim):
    """|w - q| <= s (1/2 + maxq 2^-11): half a step, plus what the fp16 rounding of the
    scale and the integer rounding of the zero point can clip at the top of the range."""
    maxq = 2 ** bits - 1
    W = (RNG.standard_normal((256, 256)) * 0.02).astype(np.float32)
    W[RNG.integers(0, 256, 50), RNG.integers(0, 256, 50)] *= 40.0
    r = O.quantize_rtn(W, bits, 128, dim)
    s = np.repeat(r["scales"].astype(np.float64), 128, axis=1 if dim == "oc" else 0)
    err = np.abs(W.astype(np.float64) - r["Q"].astype(np.float64))
    assert np.all(err <= s * (0.5 + maxq * 2.0 ** -11) * (1 + 1e-6))
    assert err.max() > 0.25 * s.min()     # not trivially zero


@pytest.mark.parametrize("bits", [3, 4])
def test_on_grid_weights_are_reproduced(bits):
    maxq = 2 ** bits - 1
    s0 = np.float32(np.float16(0.0123))
    for z0 in [0, 2, maxq]:
        c = RNG.integers(0, maxq + 1, size=(4, 128)).astype(np.uint8)
        c[:, 0], c[:, 1] = 0, maxq
        W = (s0 * (c.astype(np.float32) - np.float32(z0))).astype(np.float32)
        r = O.quantize_rtn(W, bits, 128, "oc")
        assert np.array_equal(r["codes"], c)
        assert np.all(r["scales"] == np.float16(s0)) and np.all(r["zeros"] == z0)
        assert np.array_equal(r["Q"], W)


def test_one_signed_and_degenerate_groups():
    # all-positive group: the range is extended down to zero, zero point 0
    W = np.linspace(0.5, 1.2, 128, dtype=np.float32)[None, :]
    r = O.quantize_rtn(W, 3, 128, "oc")
    assert r["zeros"][0, 0] == 0 and r["zeros"].view(np.uint16)[0, 0] == 0      # +0, never -0
    assert abs(float(r["scales"][0, 0]) * 7 - 1.2) < 1.2 * 2.0 ** -10
    # all-negative group: zero point is maxq
    r = O.quantize_rtn(-W, 3, 128, "oc")
    assert r["zeros"][0, 0] == 7
    # all-zero group: scale 1, zero 0, codes 0
    r = O.quantize_rtn(np.zeros((2, 128), np.float32), 4, 128, "oc")
    assert np.all(r["scales"] == 1) and np.all(r["zeros"] == 0) and not r["codes"].any()
    # range underflows fp16: same fallback
    r = O.quantize_rtn(np.full((1, 128), 1e-9, np.float32), 4, 128, "oc")
    assert r["scales"][0, 0] == 1 and r["zeros"][0, 0] == 0 and not r["codes"].any()
    # range overflows fp16: same fallback
    r = O.quantize_rtn(np.full((1, 128), 1e7, np.float32), 3, 128, "oc")
    assert r["scales"][0, 0] == 1 and not r["codes"].any()


def test_rounding_is_ties_to_even():
    # step exactly 1 (range 7 over 7 levels): values at .5 go to the even code
    W = np.zeros((1, 128), np.float32)
    W[0, 0], W[0, 1] = -3.0, 4.0
    W[0, 2:6] = [0.5, 1.5, 2.5, -0.5]
    r = O.quantize_rtn(W, 3, 128, "oc")
    assert r["scales"][0, 0] == 1 and r["zeros"][0, 0] == 3
    assert list(r["codes"][0, 2:6]) == [3, 5, 5, 3]


@pytest.mark.parametrize("bits", [3, 4])
def test_packing_matches_bigint_bitstream(bits):
    codes = RNG.integers(0, 2 ** bits, size=(5, 96)).astype(np.uint8)
    packed = O.pack_codes(codes, bits)
    assert packed.dtype == np.uint32 and packed.shape == (5, 96 * bits // 32)
    for o in range(5):
        big = 0
        for k in range(96):
            big |= int(codes[o, k]) << (k * bits)
        words = [(big >> (32 * j)) & 0xFFFFFFFF for j in range(96 * bits // 32)]
        assert [int(v) for v in packed[o]] == words
    assert np.array_equal(O.unpack_codes(packed, 96, bits), codes)


def test_average_bits_matches_the_papers_tables():
    path = os.path.join(os.path.dirname(__file__), "golden", "average_bits.txt")
    rows = [ln.split() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 4
    for b, g, avg in rows:
        assert O.average_bits(int(b), int(g)) == pytest.approx(float(avg), abs=1e-12)


def test_dequantize_round_trip():
    W = (RNG.standard_normal((128, 256)) * 0.02).astype(np.float32)
    for dim in ("oc", "ic"):
        r = O.quantize_rtn(W, 3, 128, dim)
        assert np.array_equal(O.dequantize(r["codes"], r["scales"], r["zeros"], 128, dim), r["Q"])
