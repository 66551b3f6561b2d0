"""Derives the polynomial coefficients used by csrc/sparse_zo.cu for ln(1+s) and cos(pi b), and
checks the fp32 evaluation of the whole Gaussian draw against fp64.

    python paper_2406_02913_b200/csrc/fit_gauss_polys.py

ln: u = f * 2^e with f in [sqrt(1/2), sqrt(2)), s = f - 1:  ln(1+s) = s - s^2/2 + s^3 P(s).
cos: b in [0, 1/2], t = b^2:  cos(pi b) = C(t).
Both P and C are least-squares fits on Chebyshev nodes in fp64 (close to minimax on these ranges).
"""
import numpy as np


def cheb_nodes(a, b, n):
    k = np.arange(n)
    return 0.5 * (a + b) + 0.5 * (b - a) * np.cos(np.pi * (k + 0.5) / n)


def fit_log(deg=7):
    s = cheb_nodes(np.sqrt(0.5) - 1, np.sqrt(2) - 1, 4000)
    target = (np.log1p(s) - s + 0.5 * s * s) / s ** 3
    return np.polynomial.polynomial.polyfit(s, target, deg)          # ascending powers


def fit_cos(deg=6):
    t = cheb_nodes(0.0, 0.25, 4000)
    return np.polynomial.polynomial.polyfit(t, np.cos(np.pi * np.sqrt(t)), deg)


def f32(x):
    return np.asarray(x, dtype=np.float32)


def eval_gauss_f32(r0, r1, PL, PC):
    """fp32 emulation of the kernel's arithmetic (fma modelled by fp64 product-sum rounded once)."""
    fma = lambda a, b, c: f32(a.astype(np.float64) * b.astype(np.float64) + c.astype(np.float64))
    u1 = f32(((r0 >> 8) + 1).astype(np.float64)) * f32(2.0 ** -24)
    bits = u1.view(np.int32)
    e = (bits - np.int32(0x3F3504F3)) >> 23
    f = (bits - (e << 23)).view(np.float32)
    s = f - f32(1.0)
    p = np.full_like(s, f32(PL[-1]))
    for c in PL[-2::-1]:
        p = fma(p, s, np.full_like(s, f32(c)))
    s2 = s * s
    lg = fma(s2 * s, p, fma(f32(-0.5) * s2, np.ones_like(s), s))        # s - s^2/2 + s^3 P
    L = fma(e.astype(np.float32), np.full_like(s, f32(0.6931471805599453)), lg)
    rad = np.sqrt(f32(-2.0) * L)
    x = f32((r1 >> 8).astype(np.float64)) * f32(2.0 ** -23)               # 2 u2 in [0, 2)
    a = np.abs(x - f32(1.0))
    b = np.minimum(a, f32(1.0) - a)
    t = b * b
    c = np.full_like(t, f32(PC[-1]))
    for k in PC[-2::-1]:
        c = fma(c, t, np.full_like(t, f32(k)))
    c = np.where(a > f32(0.5), c, -c)
    return rad * c


def main():
    PL, PC = fit_log(), fit_cos()
    print("ln P coefficients (ascending):", ", ".join(f"{c:.9e}f" for c in PL))
    print("cos C coefficients (ascending):", ", ".join(f"{c:.9e}f" for c in PC))
    g = np.random.default_rng(0)
    r0 = g.integers(0, 2 ** 32, 4_000_000, dtype=np.uint64)
    r1 = g.integers(0, 2 ** 32, 4_000_000, dtype=np.uint64)
    r0[:1000] = (np.arange(1000, dtype=np.uint64) << 8)                    # u1 near 2^-24
    r0[1000:2000] = ((2 ** 24 - 1 - np.arange(1000, dtype=np.uint64)) << 8)  # u1 near 1
    r1[2000:3000] = ((2 ** 22 + np.arange(1000, dtype=np.uint64) - 500) << 8)  # cos near 0
    z = eval_gauss_f32(r0, r1, PL, PC).astype(np.float64)
    u1 = ((r0 >> 8) + 1).astype(np.float64) * 2.0 ** -24
    u2 = (r1 >> 8).astype(np.float64) * 2.0 ** -24
    ref = np.sqrt(-2 * np.log(u1)) * np.cos(2 * np.pi * u2)
    err = np.abs(z - ref) / np.maximum(1.0, np.abs(ref))
    print("max |z - z_ref| / max(1, |z_ref|) =", err.max(), "(bound 1e-6)")


if __name__ == "__main__":
    main()
