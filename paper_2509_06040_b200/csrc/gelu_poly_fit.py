"""Derives the bf16 coefficients of the packed GELU polynomial in mlp_velocity.cu.

    python paper_2509_06040_b200/csrc/gelu_poly_fit.py

2 GELU(x) = x + x erf(x / sqrt 2) = x + s Q(s), s = x^2.  Q (degree 2 in s) is fitted to erf(x / sqrt 2) / x on
|x| <= 1 so that the largest error of s Q(s) is smallest (weighted least squares with Lawson's reweighting); the
kernel evaluates in bf16, so the coefficients are rounded to bf16 one after the other, each time refitting the ones
not yet fixed.  Prints the coefficients, their bf16 bit patterns and the largest error of the rounded polynomial.
"""
import numpy as np
from scipy.special import erf

RANGE, DEGREE = 1.0, 2


def to_bf16(x):
    u = np.asarray(x, dtype=np.float32).reshape(1).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return float(u.astype(np.uint32).view(np.float32)[0])


def fit():
    x = RANGE * np.cos(np.linspace(0.0, np.pi / 2, 4000))
    s = x * x
    target = np.where(x > 1e-9, erf(x / np.sqrt(2.0)) / np.maximum(x, 1e-9), np.sqrt(2.0 / np.pi))
    fixed = {}
    for _ in range(DEGREE + 1):
        free = [j for j in range(DEGREE + 1) if j not in fixed]
        basis = np.stack([s ** j for j in free], axis=1)
        rest = target - sum(fixed[j] * s ** j for j in fixed)
        weight = np.ones_like(x)
        for _ in range(60):
            coef, *_ = np.linalg.lstsq(basis * (s * weight)[:, None], rest * s * weight, rcond=None)
            err = np.abs((basis @ coef - rest) * s)
            weight *= 0.5 + err / err.max()
            weight /= weight.max()
        fixed[free[0]] = to_bf16(coef[0])
    return [fixed[j] for j in range(DEGREE + 1)]


if __name__ == "__main__":
    q = fit()
    x = np.linspace(-RANGE, RANGE, 400001)
    s = x * x
    approx = x + s * sum(q[k] * s ** k for k in range(DEGREE + 1))
    exact = x * (1.0 + erf(x / np.sqrt(2.0)))
    for k, c in enumerate(q):
        print(f"Q{k} = {c!r}  bf16 bits 0x{int(np.float32(c).view(np.uint32)) >> 16:04x}")
    print("largest |x + s Q(s) - 2 GELU(x)| on |x| <= %.2f: %.3g" % (RANGE, np.abs(approx - exact).max()))
