"""The fp16 quantizer kernel forms rint(w / s) without a division: p = fma(w, rcp(s), 192) snaps the
product to a multiple of 2^-16, and adding 1.5 * 2^23 - 192 rounds that to an integer.  This file
replays those two roundings on the CPU (exact rational arithmetic, then nearest binary32) and
compares with rint of the correctly rounded binary32 quotient, over positive fp16 scales
against random and worst-case (exact tie, nearest-to-tie) fp16 weights."""
from fractions import Fraction

import numpy as np

F32 = np.float32


def _rn32(fr: Fraction) -> float:
    """Nearest binary32 (normal range) to an exact rational, ties to even, as a Python float."""
    if fr == 0:
        return 0.0
    sign = -1.0 if fr < 0 else 1.0
    a = abs(fr)
    e = 0
    while a >= 2 ** 24:
        a /= 2
        e += 1
    while a < 2 ** 23:
        a *= 2
        e -= 1
    n = a.numerator // a.denominator
    rem = a - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return sign * float(n) * 2.0 ** e


def _kernel_rint(w: float, s: float) -> int:
    r = _rn32(Fraction(1) / Fraction(s))                                  # correctly rounded reciprocal
    t = _rn32(Fraction(w) * Fraction(r) + 192)                            # one fma
    t = _rn32(Fraction(t) + Fraction(12582912 - 192))                     # one add
    return int(np.array(t, F32).view(np.int32)) - 0x4B400000


def _reference_rint(w: float, s: float) -> int:
    return int(np.rint(F32(_rn32(Fraction(w) / Fraction(s)))))


def test_snap_rounding_exact_cases():
    rng = np.random.default_rng(77)
    scales = np.arange(1, 0x7C00, dtype=np.uint16).view(np.float16)      # every positive finite fp16
    pick = rng.choice(len(scales), 400, replace=False)
    checked = ties = 0
    for s16 in scales[pick]:
        s = float(s16)
        cands = []
        for m in range(0, 16):                                            # exact ties and their fp16 neighbours
            with np.errstate(over="ignore"):
                t = np.float16((m + 0.5) * s)
            bits = int(t.view(np.uint16))
            for u in (-1, 0, 1):
                if 0 < bits + u < 0x7C00:
                    cands.append(float(np.uint16(bits + u).view(np.float16)))
        with np.errstate(over="ignore"):
            cands += [float(np.float16(x * s)) for x in rng.uniform(-15.9, 15.9, 12)]
        for w in cands:
            if not np.isfinite(w) or abs(w / s) > 16.0:
                continue
            for ww in (w, -w):
                assert _kernel_rint(ww, s) == _reference_rint(ww, s), (ww, s)
                checked += 1
                ties += (Fraction(ww) / Fraction(s) * 2) % 2 == 1
    assert checked > 20000 and ties > 2000


def test_snap_rounding_bulk_float64_replay():
    """Same comparison over about 4e6 (w, s) pairs with the fma replayed in float64 (the product of
    an 11-bit and a 24-bit significand is exact there; adding 192 rounds once more, far below the
    2^-16 grid that decides)."""
    rng = np.random.default_rng(78)
    s = rng.integers(1, 0x7C00, 4_000_000).astype(np.uint16).view(np.float16).astype(np.float64)
    k = rng.integers(-31, 32, s.size)                                     # half of the draws aim at multiples of s/2
    with np.errstate(over="ignore"):
        w = (k * 0.5 * s).astype(np.float16).astype(np.float64)
        rnd = rng.random(s.size) < 0.5
        w = np.where(rnd, (rng.uniform(-15.9, 15.9, s.size) * s).astype(np.float16).astype(np.float64), w)
    good = np.isfinite(w) & (np.abs(w / s) <= 16.0)
    w, s = w[good], s[good]
    r = (1.0 / s).astype(F32)
    t = (w * r.astype(np.float64) + 192.0).astype(F32)
    t = (t.astype(np.float64) + (12582912.0 - 192.0)).astype(F32)
    got = t.view(np.int32).astype(np.int64) - 0x4B400000
    ref = np.rint((w / s).astype(F32)).astype(np.int64)
    assert got.size > 3_000_000 and np.array_equal(got, ref)
