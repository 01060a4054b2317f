"""Generator of the polynomial in gelu_erf_fast (common.cuh).  Run: python fit_gelu_poly.py

erf(z) for z >= 0 is evaluated as 1 - 2^p(z) with p a degree-7 polynomial without constant term that
approximates log2(erfc(z)) on [0, 4] (z is clamped to 4, where erfc < 2e-8).  The fit is an iteratively
re-weighted least-squares fit on Chebyshev nodes that levels the ABSOLUTE error of erfc; the script
prints the coefficients and the maximum absolute error of the fp32 evaluation against scipy's erf.
One exp2 (MUFU) and seven FMAs replace the division + exponential of the classical rational forms.
"""
import numpy as np
from scipy.special import erf, erfc

ZMAX, DEG = 4.0, 7


def fit():
    n = 4000
    z = np.cos(np.pi * (np.arange(n) + 0.5) / n) * ZMAX / 2 + ZMAX / 2
    target = np.log2(erfc(z))
    A = np.stack([z ** k for k in range(1, DEG + 1)], axis=1)
    w = erfc(z)
    ww = w.copy()
    for _ in range(60):
        coef, *_ = np.linalg.lstsq(A * ww[:, None], target * ww, rcond=None)
        err = (A @ coef - target) * w
        ww = ww * (1 + 0.3 * np.abs(err) / np.abs(err).max())
    return coef


def max_error_fp32(coef):
    zz = np.linspace(0, 6, 200001)
    c32 = coef.astype(np.float32)
    z32 = np.minimum(zz, ZMAX).astype(np.float32)
    acc = np.zeros_like(z32)
    for c in c32[::-1]:
        acc = (acc + c) * z32
    return float(np.abs((1 - np.exp2(acc)).astype(np.float64) - erf(zz)).max())


if __name__ == "__main__":
    c = fit()
    for k, v in enumerate(c, 1):
        print(f"c{k} = {np.float32(v)!r}")
    print("max |erf error| (fp32 evaluation):", max_error_fp32(c))
