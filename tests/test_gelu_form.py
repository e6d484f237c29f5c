"""The GELU the CUDA kernels evaluate, restated step by step in float32 numpy and held against the definition
u * Phi(u) with the exact error function (math.erf in float64).

The kernels compute  tail = Phi(-|u|) = (a1' t + ... + a5' t^5) exp(-u^2 / 2),  t = 1 / (1 + (p / sqrt 2) |u|),
with the coefficients of Abramowitz & Stegun 7.1.26 halved, and  GELU(u) = max(u, 0) - |u| tail,
GELU'(u) = Phi(u) + u exp(-u^2 / 2) / sqrt(2 pi).  The published bound of the erf formula is 1.5e-7 (absolute); a
wrong or un-halved coefficient, a wrong constant in the exponent or in t, or a wrong sign in the recombination
moves the result by 1e-3 or more somewhere on the grid below.  (The device uses ex2.approx and rcp.approx, each
good to about 2 ulp; numpy's correctly rounded exp2 and division stand in for them here, so the figures below are
those of the formula, not of the approximate instructions.)"""
import math

import numpy as np

f32 = np.float32
HALF_A = [f32(0.127414796), f32(-0.142248368), f32(0.7107068705), f32(-0.7265760135), f32(0.5307027145)]
P_OVER_SQRT2 = f32(0.23164189)
NEG_HALF_LOG2E = f32(-0.72134752044448170)
INV_SQRT_2PI = f32(0.39894228040143268)


def _parts(u):
    u = u.astype(np.float32)
    au = np.abs(u)
    ex = np.exp2((u * u).astype(np.float32) * NEG_HALF_LOG2E).astype(np.float32)
    t = (f32(1.0) / (P_OVER_SQRT2 * au + f32(1.0)).astype(np.float32)).astype(np.float32)
    poly = (HALF_A[4] * t + HALF_A[3]).astype(np.float32)
    for a in (HALF_A[2], HALF_A[1], HALF_A[0]):
        poly = (poly * t + a).astype(np.float32)
    tail = ((poly * t).astype(np.float32) * ex).astype(np.float32)
    return au, tail, ex


def gelu_kernel_form(u):
    au, tail, _ = _parts(u)
    return (np.maximum(u, f32(0.0)) - au * tail).astype(np.float32)


def gelu_grad_kernel_form(u):
    _, tail, ex = _parts(u)
    cdf = np.where(u >= 0, f32(1.0) - tail, tail).astype(np.float32)
    return (u * (ex * INV_SQRT_2PI).astype(np.float32) + cdf).astype(np.float32)


def _grid():
    return np.concatenate([np.linspace(-12.0, 12.0, 48001), np.array([0.0, -0.0, 1e-8, -1e-8, 30.0, -30.0])]).astype(np.float32)


def test_halved_coefficients_are_the_published_ones():
    published = [0.254829592, -0.284496736, 1.421413741, -1.453152027, 1.061405429]
    assert [float(a) for a in HALF_A] == [float(f32(c) / f32(2.0)) for c in published]
    assert abs(float(P_OVER_SQRT2) - 0.3275911 / math.sqrt(2.0)) < 2e-8
    assert abs(float(NEG_HALF_LOG2E) + 0.5 * math.log2(math.e)) < 1e-7


def test_gelu_form_against_the_definition():
    u = _grid()
    ref = np.array([x * 0.5 * (1.0 + math.erf(x / math.sqrt(2.0))) for x in u.astype(np.float64)])
    got = gelu_kernel_form(u).astype(np.float64)
    err = np.abs(got - ref)
    # |u| * (error of the erf formula, 1.5e-7 / 2 on Phi) + float32 rounding of the few operations
    bound = np.abs(u.astype(np.float64)) * 1.0e-7 + 4e-7 + 2e-7 * np.abs(ref)
    assert (err <= bound).all(), (float(err.max()), float(u[np.argmax(err - bound)]))
    assert got[u == 30.0][0] == 30.0 and got[u == -30.0][0] == 0.0          # the tails are exact
    assert (got[u == 0.0] == 0.0).all()


def test_gelu_derivative_form_against_the_definition():
    u = _grid()
    x = u.astype(np.float64)
    ref = 0.5 * (1.0 + np.array([math.erf(v / math.sqrt(2.0)) for v in x])) + x * np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)
    got = gelu_grad_kernel_form(u).astype(np.float64)
    assert np.abs(got - ref).max() < 5e-7, float(np.abs(got - ref).max())


def test_a_wrong_coefficient_or_sign_is_seen():
    u = _grid()
    ref = np.array([x * 0.5 * (1.0 + math.erf(x / math.sqrt(2.0))) for x in u.astype(np.float64)])
    good = float(np.abs(gelu_kernel_form(u) - ref).max())
    global HALF_A
    saved = list(HALF_A)
    try:
        HALF_A = [saved[0] * f32(2.0)] + saved[1:]                           # a coefficient left un-halved
        assert float(np.abs(gelu_kernel_form(u) - ref).max()) > 1000 * good
        HALF_A = saved[:3] + [-saved[3]] + saved[4:]                          # a sign lost
        assert float(np.abs(gelu_kernel_form(u) - ref).max()) > 1000 * good
    finally:
        HALF_A = saved
