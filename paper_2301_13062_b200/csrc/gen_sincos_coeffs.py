"""Derive the float32 polynomial coefficients of the range-restricted sine and cosine
used by the kernels (cartpole_device.cuh, `sin_cos_small`), and measure their error.

    python paper_2301_13062_b200/csrc/gen_sincos_coeffs.py

For |x| <= 0.22 (every angle an episode can hold is below 0.2095), with z = x*x:
    sin(x) ~= x + x*z*(S0 + z*S1)
    cos(x) ~= 1 + z*(-1/2 + z*(C0 + z*C1))
(one more coefficient each lowers the largest error by 0.01 ulp at most: the error is the
rounding of the evaluation, not the truncation)
The coefficients are the weighted minimax fit (Lawson iteration on Chebyshev nodes, float64)
of the two remainder functions, rounded to float32. The script then evaluates the float32
evaluation order the kernels use (fused multiply-adds emulated with exactly rounded float64
products) on every 5th float in (2^-14, 0.22] and prints the largest error in ulps against
mpmath-free float64 sin/cos. The exhaustive check over every float runs on the GPU
(cp_selftest_sincos_accuracy).
"""
from __future__ import annotations

import numpy as np

LIMIT = np.float32(0.22)  # episodes only ever take sin/cos of |theta| <= 12 degrees = 0.2095 rad


def lawson_fit(g, weight, deg, zmax, iters=60, nodes=4000):
    k = np.arange(nodes)
    z = 0.5 * zmax * (1 - np.cos(np.pi * (k + 0.5) / nodes))
    A = np.vander(z, deg + 1, increasing=True)
    y = g(z)
    w = np.ones(nodes)
    wt = weight(z)
    coef = None
    for _ in range(iters):
        sw = np.sqrt(w) * wt
        coef, *_ = np.linalg.lstsq(A * sw[:, None], y * sw, rcond=None)
        err = np.abs((A @ coef - y) * wt)
        w = w * (err + 1e-300)
        w /= w.sum()
    return coef


def sin_remainder(z):
    x = np.sqrt(np.maximum(z, 1e-30))
    # (sin(x)/x - 1)/z, series for tiny z to avoid cancellation
    series = -1.0 / 6 + z / 120 - z * z / 5040 + z ** 3 / 362880
    direct = (np.sin(x) / x - 1.0) / np.maximum(z, 1e-30)
    return np.where(z < 1e-3, series, direct)


def cos_remainder(z):
    x = np.sqrt(np.maximum(z, 1e-30))
    series = 1.0 / 24 - z / 720 + z * z / 40320 - z ** 3 / 3628800
    direct = (np.cos(x) - 1.0 + 0.5 * z) / np.maximum(z * z, 1e-60)
    return np.where(z < 1e-2, series, direct)


def f32(v):
    return np.asarray(v, np.float64).astype(np.float32)


def fma32(a, b, c):
    """float32 fused multiply-add: the float64 product of two float32 values is exact."""
    return (a.astype(np.float64) * b.astype(np.float64) + c.astype(np.float64)).astype(np.float32)


def mul32(a, b):
    return (a.astype(np.float64) * b.astype(np.float64)).astype(np.float32)


def eval_sin(x, S):
    z = mul32(x, x)
    p = fma32(np.full_like(x, S[1]), z, np.full_like(x, S[0]))
    w = mul32(p, z)
    return fma32(w, x, x)


def eval_cos(x, C):
    z = mul32(x, x)
    q = fma32(np.full_like(x, C[1]), z, np.full_like(x, C[0]))
    q = fma32(q, z, np.full_like(x, np.float32(-0.5)))
    return fma32(q, z, np.full_like(x, np.float32(1.0)))


def ulp_error(approx32, exact64):
    ulp = np.spacing(np.abs(exact64).astype(np.float32)).astype(np.float64)
    return np.abs(approx32.astype(np.float64) - exact64) / ulp


def main():
    zmax = float(LIMIT) ** 2
    # relative error of sin is z*(p - g) (to first order), of cos is z^2*(q - g)/cos
    S = f32(lawson_fit(sin_remainder, lambda z: z, 1, zmax))
    C = f32(lawson_fit(cos_remainder, lambda z: z * z, 1, zmax))
    print("sin S0,S1 =", [f"{float(v):.9e}" for v in S], [hex(int(v.view(np.uint32))) for v in S])
    print("cos C0,C1 =", [f"{float(v):.9e}" for v in C], [hex(int(v.view(np.uint32))) for v in C])
    lo = int(np.float32(2.0 ** -14).view(np.uint32))
    hi = int(LIMIT.view(np.uint32))
    worst_s = worst_c = 0.0
    for start in range(lo, hi + 1, 1 << 24):
        bits = np.arange(start, min(hi + 1, start + (1 << 24)), 5, dtype=np.uint32)
        x = bits.view(np.float32)
        xs = x.astype(np.float64)
        worst_s = max(worst_s, float(ulp_error(eval_sin(x, S), np.sin(xs)).max()))
        worst_c = max(worst_c, float(ulp_error(eval_cos(x, C), np.cos(xs)).max()))
    print(f"max error on the sample: sin {worst_s:.4f} ulp, cos {worst_c:.4f} ulp")


if __name__ == "__main__":
    main()
