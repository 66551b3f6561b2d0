"""The polynomial ln and cos of the Gaussian draw in csrc/sparse_zo.cu, checked on the CPU: the
coefficients are read out of the kernel source, compared with a fresh least-squares fit, and the
kernel's fp32 arithmetic (emulated step by step in numpy, every fma as an exactly rounded fp64
product-sum) is held to |z - z_fp64| <= 5e-7 max(1, |z|) against Box-Muller in fp64, the bound that the
z tolerance of the GPU parity tests (1e-6) relies on.

ln: u = f 2^e with f in [sqrt(1/2), sqrt(2)), s = f - 1:  ln(1+s) = s - s^2/2 + s^3 P(s), P of degree 7.
cos: b in [0, 1/2], t = b^2:  cos(pi b) = C(t), C of degree 6.
"""
import os
import re

import numpy as np

SRC = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "paper_2406_02913_b200", "csrc",
                   "sparse_zo.cu")


def kernel_coefficients():
    """(P ascending, C ascending) as written in gaussian_from_words."""
    text = open(SRC).read()
    body = text[text.index("gaussian_from_words("):]
    body = body[:body.index("__device__ __forceinline__ float z_of")]
    num = r"(-?\d\.\d+e[+-]\d+)f"
    p = [float(re.search(r"float p = " + num, body).group(1))] + [float(v) for v in re.findall(r"p = fmaf\(p, s, " + num, body)]
    c = [float(re.search(r"float c = " + num, body).group(1))] + [float(v) for v in re.findall(r"c = fmaf\(c, t, " + num, body)]
    c.append(1.0)                                         # the last step adds the constant 1.0f
    assert len(p) == 8 and len(c) == 7, (len(p), len(c))
    return np.array(p[::-1]), np.array(c[::-1])


def cheb_nodes(a, b, n):
    k = np.arange(n)
    return 0.5 * (a + b) + 0.5 * (b - a) * np.cos(np.pi * (k + 0.5) / n)


def f32(x):
    return np.asarray(x, dtype=np.float32)


def kernel_gaussian_f32(r0, r1, PL, PC):
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
    lg = fma(s2 * s, p, fma(f32(-0.5) * s2, np.ones_like(s), s))
    L = fma(e.astype(np.float32), np.full_like(s, f32(0.6931471805599453)), lg)
    rad = np.sqrt(f32(-2.0) * L)
    x = f32((r1 >> 8).astype(np.float64)) * f32(2.0 ** -23)
    a = np.abs(x - f32(1.0))
    b = np.minimum(a, f32(1.0) - a)
    t = b * b
    c = np.full_like(t, f32(PC[-1]))
    for k in PC[-2::-1]:
        c = fma(c, t, np.full_like(t, f32(k)))
    return np.where(a > f32(0.5), rad * c, -(rad * c))


def test_coefficients_are_the_least_squares_fits():
    PL, PC = kernel_coefficients()
    s = cheb_nodes(np.sqrt(0.5) - 1, np.sqrt(2) - 1, 4000)
    fit_l = np.polynomial.polynomial.polyfit(s, (np.log1p(s) - s + 0.5 * s * s) / s ** 3, 7)
    t = cheb_nodes(0.0, 0.25, 4000)
    fit_c = np.polynomial.polynomial.polyfit(t, np.cos(np.pi * np.sqrt(t)), 6)
    assert np.allclose(PL, fit_l, rtol=2e-6, atol=0) and np.allclose(PC, fit_c, rtol=2e-6, atol=1e-9)
    # and the polynomials themselves are accurate on their ranges
    assert np.max(np.abs(np.polynomial.polynomial.polyval(s, PL) * s ** 3 + s - 0.5 * s * s - np.log1p(s))) < 2e-8
    assert np.max(np.abs(np.polynomial.polynomial.polyval(t, PC) - np.cos(np.pi * np.sqrt(t)))) < 2e-8


def test_fp32_gaussian_of_the_kernel_is_within_5e7_of_fp64():
    PL, PC = kernel_coefficients()
    g = np.random.default_rng(0)
    n = 1_000_000
    r0 = g.integers(0, 2 ** 32, n, dtype=np.uint64)
    r1 = g.integers(0, 2 ** 32, n, dtype=np.uint64)
    r0[:1000] = np.arange(1000, dtype=np.uint64) << 8                          # u1 near 2^-24
    r0[1000:2000] = (2 ** 24 - 1 - np.arange(1000, dtype=np.uint64)) << 8      # u1 near 1
    r1[2000:3000] = (2 ** 22 + np.arange(1000, dtype=np.uint64) - 500) << 8    # cosine near 0
    z = kernel_gaussian_f32(r0, r1, PL, PC).astype(np.float64)
    u1 = ((r0 >> 8) + 1).astype(np.float64) * 2.0 ** -24
    u2 = (r1 >> 8).astype(np.float64) * 2.0 ** -24
    ref = np.sqrt(-2 * np.log(u1)) * np.cos(2 * np.pi * u2)
    assert np.max(np.abs(z - ref) / np.maximum(1.0, np.abs(ref))) <= 5e-7
