"""The tensor-core kernels evaluate GeLU's Phi through Abramowitz & Stegun's rational approximation 7.1.28 of erfc,
erfc(z) = (1 + a1 z + ... + a6 z^6)^-16 with |error| <= 3e-7.  This restates that arithmetic in numpy float32 (same
constants, same order of operations) and holds it against scipy's erf: the claim behind using it in place of erff is
that its error is far below the bf16 rounding of the result (2^-9 relative)."""
import numpy as np
from scipy.special import erf

A = [np.float32(v) for v in (0.0705230784, 0.0422820123, 0.0092705272, 0.0001520143, 0.0002765672, 0.0000430638)]


def gelu_rational_f32(v: np.ndarray) -> np.ndarray:
    v = v.astype(np.float32)
    z = np.abs(v) * np.float32(0.70710678118654752440)
    p = z * A[5] + A[4]
    for a in (A[3], A[2], A[1], A[0]):
        p = z * p + a
    p = z * p + np.float32(1)
    q = np.float32(1) / p
    for _ in range(4):
        q = q * q
    tail = np.float32(0.5) * q                      # Phi(-|v|)
    return v * np.where(v < 0, tail, np.float32(1) - tail)


def test_rational_gelu_against_exact_erf():
    v = np.linspace(-12.0, 12.0, 2_000_001).astype(np.float32)
    got = gelu_rational_f32(v).astype(np.float64)
    ref = 0.5 * v.astype(np.float64) * (1.0 + erf(v.astype(np.float64) / np.sqrt(2.0)))
    err = np.abs(got - ref)
    assert err.max() <= 1.0e-6                                   # absolute, over the whole range
    big = np.abs(ref) >= 1e-3
    assert (err[big] / np.abs(ref[big])).max() <= 6e-4            # an eighth of a bf16 ulp (2^-8 relative spacing)
    # the formula itself, in exact arithmetic, within the bound its source states
    z = np.abs(v.astype(np.float64)) / np.sqrt(2.0)
    poly = 1.0 + sum(float(a) * z ** (k + 1) for k, a in enumerate(A))
    assert np.abs(poly ** -16 - (1.0 - erf(z))).max() <= 3.1e-7


def test_rational_gelu_special_values():
    v = np.array([0.0, -0.0, 1e-30, -1e-30, 40.0, -40.0, np.inf], dtype=np.float32)
    g = gelu_rational_f32(v)
    assert g[0] == 0.0 and g[1] == 0.0 and abs(g[2]) < 1e-29 and abs(g[3]) < 1e-29
    assert g[4] == np.float32(40.0) and g[5] == 0.0 and g[6] == np.inf
