"""Pins for oracle/szo_oracle.py: every function is checked against something other than
itself: published known answers, closed forms, brute force, libm, statistical laws."""
import ctypes
import ctypes.util
import itertools
import os

import numpy as np
import pytest
from scipy import stats

from oracle import szo_oracle as so

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox4x32-10
def _kat():
    rows = []
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[:4], w[4:6], w[6:]))
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        got = so.philox4x32_10(*ctr, *key)
        assert [int(g) for g in got] == out


def _philox_bigint(ctr, key):
    """Second, independent statement with Python integers (no numpy)."""
    c = list(ctr)
    k = list(key)
    for r in range(10):
        if r:
            k = [(k[0] + 0x9E3779B9) % 2**32, (k[1] + 0xBB67AE85) % 2**32]
        p0 = 0xD2511F53 * c[0]
        p1 = 0xCD9E8D57 * c[2]
        c = [(p1 // 2**32) ^ c[1] ^ k[0], p1 % 2**32, (p0 // 2**32) ^ c[3] ^ k[1], p0 % 2**32]
    return c


def test_philox_matches_bigint_statement():
    g = np.random.default_rng(1)
    words = g.integers(0, 2**32, (200, 6), dtype=np.uint64)
    got = so.philox4x32_10(*[words[:, i] for i in range(6)])
    for j in range(200):
        ref = _philox_bigint([int(x) for x in words[j, :4]], [int(x) for x in words[j, 4:]])
        assert [int(got[i][j]) for i in range(4)] == ref


def test_philox_is_a_bijection_on_a_counter_slice():
    n = 1 << 14
    out = so.philox4x32_10(np.arange(n), 7, 9, 11, 123, 456)
    packed = np.stack(out, 1)
    assert len(np.unique(packed, axis=0)) == n


def test_philox_words_layout():
    # counter = (gidx_lo, gidx_hi, step_lo, step_hi), key = (seed_lo, seed_hi)
    gidx = np.array([5, 2**32 + 5, 2**40 + 17], dtype=np.uint64)
    seed, step = 0x1122334455667788, 0x99AABBCCDDEEFF00
    got = so.philox_words(seed, step, gidx)
    for j, gi in enumerate(gidx):
        gi = int(gi)
        ref = _philox_bigint([gi % 2**32, gi // 2**32, step % 2**32, step // 2**32],
                             [seed % 2**32, seed // 2**32])
        assert [int(got[i][j]) for i in range(4)] == ref


def test_philox_avalanche():
    # flipping one counter bit flips about half of the 128 output bits
    a = np.stack(so.philox4x32_10(np.arange(4096), 0, 3, 0, 1234, 0), 1)
    b = np.stack(so.philox4x32_10(np.arange(4096) ^ 1, 0, 3, 0, 1234, 0), 1)
    flips = np.unpackbits((a ^ b).view(np.uint8), axis=1).sum(1)
    assert abs(flips.mean() - 64) < 1.0


# ------------------------------------------------------------------ Gaussian z
def test_gaussian_moments_and_ks():
    z = so.gaussian(1234, 3, np.arange(2_000_000)).astype(np.float64)
    n = z.size
    assert abs(z.mean()) < 4 / np.sqrt(n)
    assert abs(z.var() - 1) < 4 * np.sqrt(2 / n)
    assert abs(stats.skew(z)) < 4 * np.sqrt(6 / n)
    assert abs(stats.kurtosis(z)) < 4 * np.sqrt(24 / n)
    assert stats.kstest(z[:200_000], "norm").pvalue > 1e-3
    assert np.isfinite(z).all()


def test_gaussian_box_muller_formula_on_chosen_words():
    # u1 = 2^-24 * ((r0 >> 8) + 1), u2 = 2^-24 * (r1 >> 8): check the extremes by hand.
    r0 = np.array([0xFFFFFFFF, 0x00000000, 0x7FFFFF00], dtype=np.uint32)
    r1 = np.array([0x00000000, 0x80000000, 0x40000000], dtype=np.uint32)
    u1, u2 = so.uniforms_from_words(r0, r1)
    assert u1[0] == 1.0 and u1[1] == 2.0 ** -24 and u1[2] == 0.5
    assert u2[0] == 0.0 and u2[1] == 0.5 and u2[2] == 0.25
    # u1 = 1 -> z = 0; u1 = 2^-24, u2 = 1/2 -> z = -sqrt(48 ln 2)
    assert np.sqrt(-2 * np.log(u1[0])) == 0.0
    assert np.isclose(np.sqrt(-2 * np.log(u1[1])) * np.cos(2 * np.pi * u2[1]), -np.sqrt(48 * np.log(2)))


def test_gaussian_is_keyed_by_index_not_by_mask_position():
    idx_a = np.array([3, 10, 500, 2**33 + 1])
    idx_b = np.array([10, 2**33 + 1])
    za = so.gaussian(7, 2, idx_a)
    zb = so.gaussian(7, 2, idx_b)
    assert za[1] == zb[0] and za[3] == zb[1]
    assert not np.array_equal(so.gaussian(7, 3, idx_a), za)      # new step, new draw
    assert not np.array_equal(so.gaussian(8, 2, idx_a), za)      # new seed, new draw


def test_gaussian_uncorrelated_across_steps_and_neighbours():
    i = np.arange(400_000)
    z0 = so.gaussian(1, 0, i).astype(np.float64)
    z1 = so.gaussian(1, 1, i).astype(np.float64)
    bound = 4 / np.sqrt(i.size)
    assert abs(np.mean(z0 * z1)) < bound
    assert abs(np.mean(z0[:-1] * z0[1:])) < bound


# ------------------------------------------------------------------ fp32 fma
def test_fmaf32_matches_libm():
    libm = ctypes.CDLL(ctypes.util.find_library("m"))
    libm.fmaf.restype = ctypes.c_float
    libm.fmaf.argtypes = [ctypes.c_float] * 3
    g = np.random.default_rng(0)
    a = (g.standard_normal(20000) * 10.0 ** g.integers(-6, 3, 20000)).astype(np.float32)
    b = g.standard_normal(20000).astype(np.float32)
    c = (g.standard_normal(20000) * 10.0 ** g.integers(-6, 3, 20000)).astype(np.float32)
    # near-cancellation cases stress the single rounding
    c[:5000] = -(a[:5000] * b[:5000]).astype(np.float32)
    got = so.fmaf32(a, b, c)
    ref = np.array([libm.fmaf(float(x), float(y), float(z)) for x, y, z in zip(a, b, c)], np.float32)
    assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    # and it differs from the twice-rounded a*b+c somewhere (so the test can tell them apart)
    twice = (a * b + c).astype(np.float32)
    assert (twice != ref).any()


# ------------------------------------------------------------------ quantizer
@pytest.mark.parametrize("fmt,G", [("bf16", 128), ("f16", 64), ("bf16", 32)])
def test_quantize_invariants(fmt, G):
    g = np.random.default_rng(2)
    W = g.normal(0, 0.02, (24, 4 * G)).astype(np.float32)
    W[3, :G] = 0.0125                       # a constant group
    codes, s_bits, z_bits = so.quantize_int4(W, G, fmt)
    q = so.unpack_codes(codes)
    assert codes.shape == (24, 2 * G) and q.min() >= 0 and q.max() <= 15
    s = so.bits16_to_f32(s_bits, fmt).astype(np.float64)
    z0 = so.bits16_to_f32(z_bits, fmt).astype(np.float64)
    deq = so.dequantize(codes, s_bits, z_bits, G, fmt)
    Wg = W.reshape(24, 4, G).astype(np.float64)
    mn = Wg.min(2)
    # constant group: scale 0, all codes 0, dequantises to the rounded minimum
    assert s[3, 0] == 0 and (q[3, :G] == 0).all() and (deq[3, :G] == z0[3, 0]).all()
    # scale and zero are the 16-bit roundings of (max-min)/15 and min
    rel = 2.0 ** -8 if fmt == "bf16" else 2.0 ** -11
    assert np.all(np.abs(s - (Wg.max(2) - mn) / 15) <= rel * np.abs((Wg.max(2) - mn) / 15) * 1.01 + 1e-12)
    assert np.all(np.abs(z0 - mn) <= rel * np.abs(mn) * 1.01)
    # error bound where the code was not clamped: |w - deq| <= s/2 (+ fp32 rounding of the quotient)
    qg = q.reshape(24, 4, G)
    err = np.abs(Wg - deq.reshape(24, 4, G))
    inner = (qg > 0) & (qg < 15)
    assert np.all(err[inner] <= (0.5 + 1e-5) * np.broadcast_to(s[:, :, None], err.shape)[inner] + 1e-12)
    # brute force: the chosen level is the nearest of the 16 levels (ties aside)
    levels = z0[:, :, None, None] + s[:, :, None, None] * np.arange(16)[None, None, None, :]
    dist = np.abs(Wg[..., None] - levels)
    best = dist.min(-1)
    chosen = np.take_along_axis(dist, qg[..., None].astype(np.int64), -1)[..., 0]
    nz = np.broadcast_to(s[:, :, None] > 0, chosen.shape)
    assert np.all(chosen[nz] <= best[nz] + 1e-6 * np.broadcast_to(s[:, :, None], chosen.shape)[nz])


def test_quantize_reproduces_exact_levels_and_rounds_half_to_even():
    # zero = 0.5, scale = 0.25 are exact in both 16-bit formats; levels 0.5 + 0.25 q
    G = 16
    q_true = np.arange(16)
    W = (0.5 + 0.25 * q_true).astype(np.float32)[None, :]
    for fmt in ("bf16", "f16"):
        codes, s_bits, z_bits = so.quantize_int4(W, G, fmt)
        assert np.array_equal(so.unpack_codes(codes)[0], q_true)
        assert so.bits16_to_f32(s_bits, fmt)[0, 0] == 0.25 and so.bits16_to_f32(z_bits, fmt)[0, 0] == 0.5
        assert np.array_equal(so.dequantize(codes, s_bits, z_bits, G, fmt)[0], W[0].astype(np.float64))
    # half-way points: (w - zero)/scale = 0.5, 1.5, 2.5, ... -> 0, 2, 2, 4, 4 ...
    Wh = W.copy()
    Wh[0, 1:15] = (0.5 + 0.25 * (np.arange(1, 15) - 0.5)).astype(np.float32)
    codes, _, _ = so.quantize_int4(Wh, G, "bf16")
    expect = np.rint(np.arange(1, 15) - 0.5).astype(int)      # numpy rint is half-to-even
    assert np.array_equal(so.unpack_codes(codes)[0, 1:15], expect)
    assert list(expect[:4]) == [0, 2, 2, 4]


def test_quantize_packing_order():
    W = np.zeros((1, 16), np.float32)
    W[0, :] = np.linspace(0, 15, 16)
    codes, _, _ = so.quantize_int4(W, 16, "bf16")
    assert codes[0, 0] == (0 | (1 << 4)) and codes[0, 7] == (14 | (15 << 4))


def test_quantize_rejects_bad_input():
    with pytest.raises(ValueError):
        so.quantize_int4(np.zeros((2, 100), np.float32), 64, "bf16")
    W = np.zeros((2, 64), np.float32)
    W[0, 3] = np.nan
    with pytest.raises(ValueError):
        so.quantize_int4(W, 64, "bf16")


# ------------------------------------------------------------------ sensitive mask
def test_dequantize_lut_hand_values_and_reduction_to_the_uniform_format():
    """Non-uniform 4-bit format (a code selects one of 16 per-row values).  Pinned by values written
    out by hand (nibble order: low nibble = even column; the table is per row) and by the special case
    of an arithmetic table j*s + z, where the look-up must equal the uniform format with one group
    per row, which the quantizer tests pin."""
    codes = np.array([[0x21, 0x43], [0xF0, 0x0F]], np.uint8)            # q = [1,2,3,4], [0,15,15,0]
    lut = np.stack([10.0 + np.arange(16), -np.arange(16) / 4.0]).astype(np.float32)
    for fmt in ("f16", "bf16"):
        bits, vals = so.round_to_16(lut, fmt)
        assert np.array_equal(vals, lut)                                   # representable in both formats
        W = so.dequantize_lut(codes, bits, fmt)
        assert np.array_equal(W, np.array([[11.0, 12.0, 13.0, 14.0], [0.0, -3.75, -3.75, 0.0]]))
    r = np.random.default_rng(5)
    N, K = 6, 64
    codes = r.integers(0, 256, (N, K // 2), dtype=np.uint8)
    s = (2.0 ** -r.integers(4, 8, N)).astype(np.float32)                   # powers of two: j*s + z is exact
    z = (-8.0 * s).astype(np.float32)
    lut = (np.arange(16, dtype=np.float32)[None, :] * s[:, None] + z[:, None]).astype(np.float32)
    for fmt in ("f16", "bf16"):
        lb, lv = so.round_to_16(lut, fmt)
        assert np.array_equal(lv, lut)
        sb, _ = so.round_to_16(s[:, None], fmt)
        zb, _ = so.round_to_16(z[:, None], fmt)
        assert np.array_equal(so.dequantize_lut(codes, lb, fmt), so.dequantize(codes, sb, zb, K, fmt))
    # a table that is not arithmetic: every element is one of its row's 16 values, chosen by its code
    lut = np.sort(r.normal(0, 0.02, (N, 16)).astype(np.float32), axis=1)
    lb, lv = so.round_to_16(lut, "f16")
    W = so.dequantize_lut(codes, lb, "f16")
    q = so.unpack_codes(codes)
    for n in range(N):
        assert set(np.unique(W[n])) <= set(lv[n].astype(np.float64))
        assert np.all(np.diff(W[n][np.argsort(q[n], kind="stable")]) >= 0)   # ascending table: monotone in the code


def test_select_mask_brute_force_subsets():
    g = np.random.default_rng(3)
    for trial in range(30):
        n = int(g.integers(4, 13))
        k = int(g.integers(0, n + 1))
        grad = g.standard_normal(n).astype(np.float32)
        if trial % 3 == 0:                       # force ties
            grad = np.round(grad)
        scores = grad * grad
        best, best_set = -1.0, None
        for sub in itertools.combinations(range(n), k):       # lexicographic order
            v = float(np.sum(scores[list(sub)].astype(np.float64)))
            if v > best:                                     # strict: first (lowest) set wins ties
                best, best_set = v, sub
        got = so.select_mask(scores, k)
        assert float(np.sum(scores[got].astype(np.float64))) == best
        assert tuple(got) == tuple(best_set if best_set is not None else ())


def test_select_mask_ties_and_order():
    assert list(so.select_mask(np.ones(10, np.float32), 4)) == [0, 1, 2, 3]
    s = np.array([1, 5, 3, 5, 3, 3, 0], np.float32)
    assert list(so.select_mask(s, 3)) == [1, 2, 3]           # threshold 3 is tied: lowest index
    assert list(so.select_mask(s, 4)) == [1, 2, 3, 4]
    assert list(so.select_mask(s, 0)) == []
    assert list(so.select_mask(np.array([0.0, -0.0, 0.0], np.float32), 2)) == [0, 1]
    with pytest.raises(ValueError):
        so.select_mask(np.array([1.0, np.nan], np.float32), 1)


def test_select_mask_matches_full_sort_large():
    g = np.random.default_rng(4)
    scores = np.square(g.standard_t(3, 300_000).astype(np.float32))
    k = 300
    got = so.select_mask(scores, k)
    order = sorted(range(scores.size), key=lambda i: (-float(scores[i]), i))[:k]
    assert list(got) == sorted(order)


def test_decompose_reconstructs_w():
    g = np.random.default_rng(5)
    W = g.normal(0, 0.02, (16, 32)).astype(np.float32)
    idx = np.sort(g.choice(W.size, 20, replace=False))
    S, Wd = so.decompose(W, idx)
    assert (Wd.ravel()[idx] == 0).all()
    back = Wd.copy()
    back.ravel()[idx] += S
    assert np.array_equal(back, W)                           # w = w_sparse + w_dense, bit-exact


# ------------------------------------------------------------------ linear layer
def test_linear_special_cases():
    g = np.random.default_rng(6)
    N, K, M, G = 16, 64, 5, 32
    W = g.normal(0, 0.02, (N, K)).astype(np.float32)
    idx = np.sort(g.choice(N * K, 12, replace=False))
    S, Wd = so.decompose(W, idx)
    codes, sb, zb = so.quantize_int4(Wd, G, "bf16")
    deq = so.dequantize(codes, sb, zb, G, "bf16")
    x = g.standard_normal((M, K))
    # nnz = 0: plain matmul with the dequantised weight
    assert np.allclose(so.linear_fwd(x, deq, [], []), x @ deq.T, rtol=0, atol=1e-13)
    # x = I returns W_eff^T
    Weff = so.effective_weight(deq, idx, S)
    assert np.array_equal(so.linear_fwd(np.eye(K), deq, idx, S), Weff.T)
    assert np.allclose(Weff.ravel()[idx], deq.ravel()[idx] + S.astype(np.float64), rtol=0, atol=0)
    off = np.setdiff1d(np.arange(N * K), idx)
    assert np.array_equal(Weff.ravel()[off], deq.ravel()[off])
    # zero dense part: only the sparse term remains
    y = so.linear_fwd(x, np.zeros((N, K)), idx, S)
    ref = np.zeros((M, N))
    for e, v in zip(idx, S):
        ref[:, e // K] += float(v) * x[:, e % K]
    assert np.allclose(y, ref, rtol=0, atol=1e-14)
    # the two evaluation orders of the appendix agree
    b = g.standard_normal(N)
    assert np.allclose(so.linear_fwd(x, deq, idx, S, b), so.linear_fwd_sparse_addmm(x, deq, idx, S, b),
                       rtol=0, atol=1e-13)
    # dequantised weights stay close to the dense part
    assert np.max(np.abs(deq - Wd)) <= 0.51 * so.bits16_to_f32(sb, "bf16").max() + 1e-4


# ------------------------------------------------------------------ SPSA / ZO-SGD
def _quad_problem(d=64, k=16, seed=7):
    g = np.random.default_rng(seed)
    A = g.standard_normal((d, d))
    A = A + A.T
    w = g.normal(0, 0.05, d).astype(np.float32)
    idx = np.sort(g.choice(d, k, replace=False)).astype(np.int64)
    return A, w, idx


def test_spsa_exact_on_quadratic_and_linear():
    A, w, idx = _quad_problem()
    d = w.size
    gidx = idx + 1000                                         # flat index with a tensor base

    def full(S):
        v = w.astype(np.float64).copy()
        v[idx] = S.astype(np.float64)
        return v

    eps = np.float32(1e-3)
    for step in range(5):
        z = np.zeros(d)
        z[idx] = so.gaussian(11, step, gidx).astype(np.float64)
        # f = 1/2 w^T A w  ->  (f+ - f-)/(2 eps) = zbar^T A w
        S1, fp, fm, gq = so.zo_sgd_step(lambda S: 0.5 * full(S) @ A @ full(S), w[idx], gidx, 11, step, eps, 0.0)
        assert np.isclose(gq, z @ A @ w.astype(np.float64), rtol=2e-5, atol=1e-7)
        # f = a^T w -> g = zbar^T a
        a = A[0]
        _, _, _, gl = so.zo_sgd_step(lambda S: a @ full(S), w[idx], gidx, 11, step, eps, 0.0)
        assert np.isclose(gl, z @ a, rtol=2e-5, atol=1e-7)
        # lr = 0: S returns to its start up to fp32 rounding of the three passes
        assert np.max(np.abs(S1.astype(np.float64) - w[idx])) <= 4 * np.spacing(np.float32(0.2))


def test_zo_sgd_update_and_replay_identity():
    A, w, idx = _quad_problem(d=48, k=48)                     # full mask: k = d (plain MeZO)
    gidx = idx
    eps, lr = np.float32(1e-3), np.float32(1e-3)
    S = w.copy()
    S0 = S.astype(np.float64)
    acc = np.zeros(48)
    for step in range(20):
        z = so.gaussian(5, step, gidx).astype(np.float64)
        S_new, fp, fm, g = so.zo_sgd_step(lambda S_: 0.5 * S_.astype(np.float64) @ A @ S_.astype(np.float64),
                                          S, gidx, 5, step, eps, lr)
        # Definition 2 on all d coordinates: w <- w - lr g z
        assert np.allclose(S_new, S.astype(np.float64) - float(lr) * g * z, rtol=0, atol=1e-7)
        acc += float(lr) * g * z
        S = S_new
    assert np.allclose(S, S0 - acc, rtol=0, atol=1e-6)        # S_T = S_0 - sum_t lr g_t z_t


def test_n_sample_spsa_reduces_to_one_sample_and_averages():
    """zo_sgd_step_n: n = 1 is zo_sgd_step bit for bit; for a linear loss a.w the update is exactly
    -(lr/n) sum_i (zbar_i . a) zbar_i with the z of counters step*n + i; and the estimate's spread around
    the true masked gradient shrinks like 1/sqrt(n)."""
    A, w, idx = _quad_problem(d=64, k=10)
    state = w.copy()

    def quad(S):
        v = state.astype(np.float64).copy()
        v[idx] = S
        return 0.5 * v @ A @ v

    one = so.zo_sgd_step(quad, state[idx], idx, 3, 11, 1e-3, 1e-2)
    n1 = so.zo_sgd_step_n(quad, state[idx], idx, 3, 11, 1, 1e-3, 1e-2)
    assert np.array_equal(one[0].view(np.uint32), n1[0].view(np.uint32)) and one[3] == n1[3][0]
    g = np.random.default_rng(4)
    a = g.standard_normal(64)

    def lin(S):
        v = state.astype(np.float64).copy()
        v[idx] = S
        return float(a @ v)

    eps, lr, n = np.float32(1e-3), np.float32(1e-3), 4
    S_new, fps, fms, gs = so.zo_sgd_step_n(lin, state[idx], idx, 9, 5, n, eps, lr)
    exp = state[idx].astype(np.float64)
    for i in range(n):
        z = so.gaussian(9, 5 * n + i, idx).astype(np.float64)
        assert abs(gs[i] - z @ a[idx]) < 1e-3 * abs(z @ a[idx]) + 1e-4          # fp32 S limits the difference quotient
        exp = exp - float(lr) / n * gs[i] * z
    assert np.allclose(S_new, exp, rtol=0, atol=1e-6)
    # spread of the estimate (sum_i g_i z_i / n) around a[idx]: n = 16 against n = 1 over 400 draws each
    def spread(n):
        err = []
        for t in range(400):
            est = np.zeros(10)
            for i in range(n):
                z = so.gaussian(21, t * n + i, idx).astype(np.float64)
                est += (z @ a[idx]) * z / n
            err.append(np.sum((est - a[idx]) ** 2))
        return np.mean(err)
    assert 10.0 < spread(1) / spread(16) < 24.0


def test_replay_from_the_log_reproduces_the_run():
    """so.replay against the run it replays (itself pinned above): the same bits when the +-eps passes
    are replayed too, and S_0 - sum_t lr g_t z_t up to their drift when they are skipped."""
    A, w, idx = _quad_problem(d=64, k=10)
    state = w.copy()

    def loss(S):
        v = state.astype(np.float64).copy()
        v[idx] = S
        return 0.5 * v @ A @ v

    eps, lr = np.float32(1e-3), np.float32(1e-2)
    S, log, acc = state[idx].copy(), [], np.zeros(10)
    for step in (3, 4, 9, 10, 11, 40):                       # the log need not be contiguous
        S, fp, fm, g = so.zo_sgd_step(loss, S, idx, 77, step, eps, lr)
        log.append((step, g))
        acc += float(lr) * g * so.gaussian(77, step, idx).astype(np.float64)
    again = so.replay(state[idx], idx, 77, log, eps, lr)
    assert np.array_equal(again.view(np.uint32), S.view(np.uint32))
    plain = so.replay(state[idx], idx, 77, log, 0.0, lr)
    assert np.allclose(plain, state[idx].astype(np.float64) - acc, rtol=0, atol=1e-6)
    assert np.allclose(plain, S, rtol=0, atol=1e-6) and so.replay(state[idx], idx, 77, [], eps, lr).tolist() == state[idx].tolist()


def test_sparse_step_touches_only_masked_coordinates():
    A, w, idx = _quad_problem(d=64, k=8)
    state = w.copy()

    def loss(S):
        v = state.astype(np.float64).copy()
        v[idx] = S
        return 0.5 * v @ A @ v

    S_new, *_ = so.zo_sgd_step(loss, state[idx], idx, 1, 0, 1e-3, 1e-2)
    after = state.copy()
    after[idx] = S_new
    off = np.setdiff1d(np.arange(64), idx)
    assert np.array_equal(after[off].view(np.uint32), w[off].view(np.uint32))
    assert (after[idx] != w[idx]).any()


def test_sparse_zo_gradient_second_moments():
    # f = a^T w: ghat = (zbar^T a) zbar.  E||ghat||^2 = (k + 2) ||m.a||^2 (Lemma, sparse ZO
    # surrogate gradient norm) and E (f+ - f-)^2 = 4 eps^2 ||m.a||^2 (Section 3.1).
    g = np.random.default_rng(8)
    d, k, T = 200, 12, 40000
    a = g.standard_normal(d)
    idx = np.sort(g.choice(d, k, replace=False)).astype(np.int64)
    ma2 = float(np.sum(a[idx] ** 2))
    Z = np.stack([so.gaussian(99, t, idx).astype(np.float64) for t in range(T)])      # [T, k]
    proj = Z @ a[idx]
    gn2 = proj ** 2 * np.sum(Z * Z, axis=1)
    se = gn2.std() / np.sqrt(T)
    assert abs(gn2.mean() - (k + 2) * ma2) < 4 * se
    eps = 1e-3
    diff2 = (2 * eps * proj) ** 2
    assert abs(diff2.mean() - 4 * eps ** 2 * ma2) < 4 * diff2.std() / np.sqrt(T)
    # covariance of zbar is the masked identity
    C = Z.T @ Z / T
    assert np.max(np.abs(C - np.eye(k))) < 5 / np.sqrt(T)


def test_update_scale_and_projected_gradient():
    eps = np.float32(1e-3)
    g = so.projected_gradient(2.5, 2.25, eps)
    assert np.isclose(g, 0.25 / (2 * float(eps)), rtol=1e-15)
    sc = so.zo_update_scale(2.5, 2.25, eps, 1e-5)
    assert sc == np.float32(-(float(np.float32(1e-5)) * g)) and sc < 0


@pytest.mark.parametrize("fmt", ["f16", "bf16"])
def test_step_with_16_bit_sparse_storage(fmt):
    """Section 3.5 (w_sparse kept in 16 bits), reading: fp32 step on the widened values, one rounding to
    the storage format.  Pinned by what does not involve the oracle's own rounding code: the result
    of the fp32 step cast by a library (numpy's float16, torch's bfloat16), representability, the
    half-ulp bound, and the two regimes an update can fall in (lost below half an ulp, visible above)."""
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(5)
    k = 4096
    gidx = np.sort(rng.choice(10 ** 6, k, replace=False)).astype(np.int64)
    a = rng.normal(0, 1, k)
    loss = lambda S: float(np.dot(a, S.astype(np.float64)))          # linear: g = z.a up to rounding
    S0 = rng.normal(0, 0.02, k).astype(np.float32)
    bits0, S0r = so.round_to_16(S0, fmt)
    for lr in (1e-9, 1e-3):
        bits1, fp, fm, g = so.zo_sgd_step_16(loss, bits0, fmt, gidx, 77, 3, 1e-3, lr)
        S32, fp2, fm2, g2 = so.zo_sgd_step(loss, S0r, gidx, 77, 3, 1e-3, lr)
        assert (fp, fm, g) == (fp2, fm2, g2)                         # the losses see fp32 perturbations of the widened values
        # a library's cast of the fp32 result
        if fmt == "f16":
            lib_bits = S32.astype(np.float16).view(np.uint16)
        else:
            lib_bits = torch.from_numpy(S32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(bits1, lib_bits)
        S1 = so.bits16_to_f32(bits1, fmt)
        assert np.array_equal(so.round_to_16(S1, fmt)[0], bits1)     # representable
        ulp = np.abs(so.bits16_to_f32(bits1 + np.uint16(1), fmt) - S1)
        assert np.all(np.abs(S1.astype(np.float64) - S32.astype(np.float64)) <= 0.5 * ulp.astype(np.float64) * (1 + 1e-12))
        z = so.gaussian(77, 3, gidx)
        upd = np.abs(np.float64(lr) * g * z)
        if lr == 1e-9:
            small = upd < 0.25 * ulp                                  # (all but stored values next to zero)
            assert small.mean() > 0.99 and np.array_equal(bits1[small], bits0[small])   # such an update is lost
        else:
            moved = bits1 != bits0
            assert moved.mean() > 0.9 and np.all(moved[upd > ulp])                # an update above one ulp always shows
