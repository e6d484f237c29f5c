"""The three-instruction quotient of the CUDA kernels (product with the rounded reciprocal, exact residual by
FMA, one correction) against IEEE float32 division, emulated instruction by instruction in numpy.

For a bfloat16-valued numerator (8 significant bits) and ANY float32 divisor the two agree bit for bit: scaling
either operand by a power of two scales every intermediate exactly, so the 128 numerator significands times
the 2^23 divisor significands are all the cases there are.  The default run covers a spread of 8 numerator
significands (6.7e7 cases, a few seconds); MREM_EXHAUSTIVE=1 runs all 1.07e9 (about 90 s on one core; passed
with 0 mismatches when the kernel started to rely on it).  The float64 emulation of the last FMA rounds twice;
the few thousand cases per significand where that could matter are re-done in exact rational arithmetic."""
import os
from fractions import Fraction

import numpy as np

f32 = np.float32


def _mismatches(x_sig, s_lo=0, s_hi=1 << 23, chunk=1 << 22):
    x = f32(1.0 + x_sig / 128.0)
    bad = total = 0
    for a in range(s_lo, s_hi, chunk):
        sm = np.arange(a, min(a + chunk, s_hi), dtype=np.uint32)
        s = (sm | np.uint32(0x3F800000)).view(np.float32)                  # every float32 in [1, 2)
        ref = (x / s).astype(np.float32)                                   # IEEE division
        r = (f32(1.0) / s).astype(np.float32)                              # rcp.rn
        z0 = (x * r).astype(np.float32)                                    # mul.rn
        e = (np.float64(x) - z0.astype(np.float64) * s.astype(np.float64)).astype(np.float32)   # fma.rn(-z0, s, x): exact in float64
        v = z0.astype(np.float64) + e.astype(np.float64) * r.astype(np.float64)                 # fma.rn(e, r, z0), rounded to 53 bits first
        z = v.astype(np.float32)
        up = np.nextafter(z, f32(np.inf)).astype(np.float64)
        dn = np.nextafter(z, f32(-np.inf)).astype(np.float64)
        zd = z.astype(np.float64)
        near = (np.abs(v - (zd + up) / 2) < np.abs(v) * 2.0 ** -40) | (np.abs(v - (zd + dn) / 2) < np.abs(v) * 2.0 ** -40)
        for i in np.nonzero(near)[0]:                                      # double rounding possible: decide exactly
            exact = Fraction(float(z0[i])) + Fraction(float(e[i])) * Fraction(float(r[i]))
            cands = [float(dn[i]), float(z[i]), float(up[i])]
            z[i] = f32(min(cands, key=lambda c: (abs(Fraction(c) - exact), int(np.float32(c).view(np.uint32)) & 1)))
        bad += int((z != ref).sum())
        total += len(sm)
    return bad, total


def test_quotient_equals_ieee_division_for_bf16_numerators():
    sigs = range(128) if os.environ.get("MREM_EXHAUSTIVE") else (0, 1, 37, 63, 64, 90, 126, 127)
    for x_sig in sigs:
        bad, total = _mismatches(x_sig)
        assert bad == 0 and total == 1 << 23, (x_sig, bad)


def test_quotient_on_float32_numerators_is_within_one_ulp_and_almost_always_exact():
    # general float32 numerators (the straight-through factors of float32 tensors): not guaranteed exact
    rng = np.random.default_rng(0)
    n = 4_000_000
    x = (rng.standard_normal(n) * 0.05).astype(np.float32)
    s = (np.abs(rng.standard_normal(n)) * 0.01 + 1e-3).astype(np.float32)
    ref = (x / s).astype(np.float32)
    r = (f32(1.0) / s).astype(np.float32)
    z0 = (x * r).astype(np.float32)
    e = (x.astype(np.float64) - z0.astype(np.float64) * s.astype(np.float64)).astype(np.float32)
    z = (z0.astype(np.float64) + e.astype(np.float64) * r.astype(np.float64)).astype(np.float32)
    diff = np.abs(z.view(np.int32).astype(np.int64) - ref.view(np.int32).astype(np.int64))
    assert diff.max() <= 1
    assert (diff != 0).mean() < 1e-5


def _code_fast(n, s, lo, hi, exact_quotient):
    """numpy emulation, instruction by instruction, of the kernels' code path: first product kept inside
    [lo - 1, hi + 1], residual by FMA, correction, clip, nearest integer by adding and subtracting 1.5 * 2^23, and (unless
    the quotient is known to be exact) a second look by IEEE division for values within 2^-10 of a half-integer."""
    magic = f32(12582912.0)
    r = (f32(1.0) / s).astype(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        z0 = np.clip((n * r).astype(np.float32), f32(lo - 1), f32(hi + 1))
        e = (n.astype(np.float64) - z0.astype(np.float64) * s.astype(np.float64)).astype(np.float32)
        z = (z0.astype(np.float64) + e.astype(np.float64) * r.astype(np.float64)).astype(np.float32)
    zc = np.clip(z, f32(lo), f32(hi))
    t = (zc + magic).astype(np.float32)
    q = (t - magic).astype(np.float32)
    low_byte = t.view(np.uint32) & np.uint32(0xFF)
    if not exact_quotient:
        again = np.abs(np.abs(zc - q) - f32(0.5)) < f32(2.0 ** -10)
        with np.errstate(over="ignore"):
            zd = np.clip((n / s).astype(np.float32), f32(lo), f32(hi))
        t2 = (zd + magic).astype(np.float32)
        q = np.where(again, (t2 - magic).astype(np.float32), q)
        low_byte = np.where(again, t2.view(np.uint32) & np.uint32(0xFF), low_byte)
    return q.astype(np.int64), low_byte.astype(np.int64)


def test_fast_codes_equal_division_codes():
    """The codes the kernels emit without the division instruction against Eq. 1 computed with IEEE division: random
    float32 numerators (the fix-up path), bfloat16 numerators (no fix-up), numerators placed within a few ulps of every
    rounding boundary k + 1/2, and numerators so large that the first product overflows; signed and unsigned ranges;
    the low byte of the rounding word is the two's-complement code."""
    rng = np.random.default_rng(1)
    for lo, hi in ((-127, 127), (0, 255), (-7, 7)):
        s = (np.abs(rng.standard_normal(2_000_000)) * 0.02 + 1e-4).astype(np.float32)
        cases = [(rng.standard_normal(s.size) * 2.0).astype(np.float32)]
        k = rng.integers(lo - 1, hi + 1, s.size).astype(np.float64) + 0.5
        ulps = rng.integers(-3, 4, s.size)
        near = (k * s.astype(np.float64)).astype(np.float32)
        cases.append((near.view(np.int32) + ulps.astype(np.int32)).view(np.float32))         # a few ulps around the boundary
        cases.append(np.where(rng.random(s.size) < 0.5, f32(3e38), f32(-3e38)) * rng.random(s.size).astype(np.float32))
        for n in cases:
            with np.errstate(over="ignore"):
                ref = np.rint(np.clip((n / s).astype(np.float32), lo, hi)).astype(np.int64)
            q, byte = _code_fast(n, s, lo, hi, exact_quotient=False)
            assert np.array_equal(q, ref)
            assert np.array_equal(byte, ref & 0xFF)
        # bfloat16 numerators: no second look
        nb = (cases[0].view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
        ref = np.rint(np.clip((nb / s).astype(np.float32), lo, hi)).astype(np.int64)
        q, byte = _code_fast(nb, s, lo, hi, exact_quotient=True)
        assert np.array_equal(q, ref) and np.array_equal(byte, ref & 0xFF)
        nb = (cases[1].view(np.uint32) & np.uint32(0xFFFF0000)).view(np.float32)
        ref = np.rint(np.clip((nb / s).astype(np.float32), lo, hi)).astype(np.int64)
        assert np.array_equal(_code_fast(nb, s, lo, hi, exact_quotient=True)[0], ref)
