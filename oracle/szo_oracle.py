"""CPU oracle: the element-level operations of the sensitive-sparse ZO step.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  numpy, single-threaded, written for
legibility; shares no code with the CUDA library.

What each function restates
---------------------------
philox4x32_10     Philox4x32-10 counter-based generator of Salmon, Moraes, Dror & Shaw
                  (SC'11), the published definition.  The paper only asks that z be
                  reproducible from a seed (Section 2.1, the "random seed trick"; Section 3.5,
                  "Gradients"); keying it by (seed, step, parameter index) is the reading taken here.
gaussian          z ~ N(0,1) per parameter (Definition 1, SPSA): Box-Muller in fp64.
select_mask       Definition 3 (sensitive parameter mask): the k coordinates with the largest
                  squared gradient, ties broken by lowest index.
decompose         Section 3.4, the sparse/dense decomposition w = w_sparse + w_dense.
quantize_int4     Section 3.5 "Integration with quantization": a 4-bit quantizer Q for w_dense.
                  The paper allows any post-training quantizer; the convention here (uniform,
                  asymmetric, group-wise, round-half-even) is parity unpinned by the paper.
dequantize        the inverse map, exact in fp64.
dequantize_lut    Section 4 / appendix on hyperparameters: the experiments quantize with a non-uniform
                  4-bit format (SqueezeLLM), i.e. a code selects one of 16 per-output-channel
                  values.  The inverse map is that table look-up, exact in fp64.  The paper does
                  not spell the format out: the convention here (per-row table of 16 values in a
                  16-bit float format, codes packed like the uniform format) is parity unpinned by
                  the paper.
effective_weight  Appendix "Implementation of Sparse Operations in Linear Layers":
                  Dequantize(Q(w_dense)) + w_sparse.
linear_fwd        the same appendix: y = x (Dequantize(Q(w_dense)) + w_sparse)^T.
perturb           Definition 4 / Section 3.4 update rule: w_sparse <- w_sparse + scale * z_k.
zo_update_scale   Definition 1 + Definition 2: the scalar -(lr * (f+ - f-) / (2 eps)).
zo_sgd_step       one whole step for any loss callable (Definitions 1, 2 and 4).
"""
from __future__ import annotations

import numpy as np

_M0 = np.uint64(0xD2511F53)
_M1 = np.uint64(0xCD9E8D57)
_W0 = np.uint64(0x9E3779B9)
_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)


# --------------------------------------------------------------------------- Philox
def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32-10.  All arguments are arrays (or scalars) of 32-bit words; returns the
    four output words as uint32 arrays.

    One round maps (c0,c1,c2,c3) -> (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0));
    the key is advanced by the Weyl constants (W0, W1) between rounds; ten rounds.
    """
    c0, c1, c2, c3, k0, k1 = (np.asarray(v).astype(np.uint64) & _MASK32
                              for v in np.broadcast_arrays(c0, c1, c2, c3, k0, k1))
    for _ in range(10):
        p0 = _M0 * c0            # 32x32 -> 64 bit product, exact in uint64
        p1 = _M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _W0) & _MASK32
        k1 = (k1 + _W1) & _MASK32
    return tuple(v.astype(np.uint32) for v in (c0, c1, c2, c3))


def philox_words(seed: int, step: int, gidx):
    """The four Philox words of parameter `gidx` (flat index over all linear parameters)
    at optimisation step `step`: key = (seed_lo, seed_hi), counter = (gidx_lo, gidx_hi,
    step_lo, step_hi)."""
    gidx = np.asarray(gidx, dtype=np.uint64)
    seed = int(seed) & 0xFFFFFFFFFFFFFFFF
    step = int(step) & 0xFFFFFFFFFFFFFFFF
    return philox4x32_10(gidx & _MASK32, gidx >> _SH32,
                         np.uint64(step & 0xFFFFFFFF), np.uint64(step >> 32),
                         np.uint64(seed & 0xFFFFFFFF), np.uint64(seed >> 32))


# --------------------------------------------------------------------------- Gaussian
def uniforms_from_words(r0, r1):
    """u1 in (0,1], u2 in [0,1): the top 24 bits of the first two words, as fp64 (both are
    exactly representable in fp32 as well)."""
    u1 = ((r0.astype(np.uint64) >> np.uint64(8)) + np.uint64(1)).astype(np.float64) * 2.0 ** -24
    u2 = (r1.astype(np.uint64) >> np.uint64(8)).astype(np.float64) * 2.0 ** -24
    return u1, u2


def gaussian(seed: int, step: int, gidx) -> np.ndarray:
    """z_i ~ N(0,1) for parameter index i (Definition 1: z ~ N(0, I_d)), regenerated from
    (seed, step, i) so that it is never stored.  Box-Muller cosine branch in fp64, rounded
    once to fp32.  Words r2, r3 are not used."""
    r0, r1, _, _ = philox_words(seed, step, gidx)
    u1, u2 = uniforms_from_words(r0, r1)
    z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return z.astype(np.float32)


# --------------------------------------------------------------------------- fp32 fma
def fmaf32(a, b, c) -> np.ndarray:
    """Correctly rounded fp32 fused multiply-add a*b+c for fp32 inputs.

    The product of two fp32 numbers is exact in fp64.  The fp64 sum is then formed with its
    rounding error (TwoSum) and, where inexact, forced to an odd last bit (round-to-odd); a
    final rounding fp64 -> fp32 of a round-to-odd value equals the single rounding of the
    exact result because fp64 carries more than 2*24+2 significand bits.
    """
    a = np.asarray(a, dtype=np.float32).astype(np.float64)
    b = np.asarray(b, dtype=np.float32).astype(np.float64)
    c = np.asarray(c, dtype=np.float32).astype(np.float64)
    a, b, c = np.broadcast_arrays(a, b, c)
    p = a * b
    s = p + c
    bb = s - p
    err = (p - (s - bb)) + (c - bb)
    s = np.ascontiguousarray(s)
    bits = s.view(np.int64)
    inexact_even = (err != 0.0) & ((bits & 1) == 0) & np.isfinite(s)
    toward = np.where(err > 0.0, np.inf, -np.inf)
    s_odd = np.where(inexact_even, np.nextafter(s, toward), s)
    return s_odd.astype(np.float32)


# --------------------------------------------------------------------------- mask
def select_mask(scores, k: int) -> np.ndarray:
    """Definition 3: indices of the k largest scores (score_i = squared gradient of
    coordinate i).  Total order (score descending, index ascending) so that ties go to the
    lowest index; result sorted ascending, int64.  NaN scores are an error."""
    scores = np.asarray(scores, dtype=np.float32).ravel()
    n = scores.size
    if not 0 <= k <= n:
        raise ValueError("k out of range")
    if np.isnan(scores).any():
        raise ValueError("NaN score")
    order = np.argsort(-(scores + np.float32(0.0)), kind="stable")  # stable: lower index first
    return np.sort(order[:k]).astype(np.int64)


def decompose(W, idx):
    """Section 3.4: w_sparse = w (.) m_k (returned as the k values S), w_dense = w (.) (1-m_k)
    (returned full-size with the masked entries set to zero)."""
    W = np.asarray(W, dtype=np.float32)
    W_dense = W.copy()
    S = W.ravel()[idx].copy()
    W_dense.ravel()[idx] = 0.0
    return S, W_dense


# --------------------------------------------------------------------------- 16-bit formats
def _round_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    b = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return r.astype(np.uint16)


def _bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_16(x32, fmt: str):
    """Round fp32 to a 16-bit float format ('bf16' or 'f16'); returns (bit patterns uint16,
    values as fp32)."""
    x32 = np.ascontiguousarray(x32, dtype=np.float32)
    if fmt == "bf16":
        bits = _round_bf16_bits(x32)
        return bits, _bf16_bits_to_f32(bits)
    if fmt == "f16":
        h = x32.astype(np.float16)
        return h.view(np.uint16), h.astype(np.float32)
    raise ValueError(fmt)


def bits16_to_f32(bits, fmt: str) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if fmt == "bf16":
        return _bf16_bits_to_f32(bits)
    if fmt == "f16":
        return bits.view(np.float16).astype(np.float32)
    raise ValueError(fmt)


# --------------------------------------------------------------------------- quantizer
def quantize_int4(W, G: int, fmt: str):
    """Group-wise asymmetric 4-bit quantizer for w_dense (Section 3.5).

    For every row n and every group of G consecutive columns:
        mn, mx        = min, max of the group                                  (fp32)
        scale         = round16((mx - mn) / 15)       zero = round16(mn)       (fmt)
        q             = clamp(rint((w - zero) / scale), 0, 15); q = 0 if scale == 0
    all in IEEE fp32 with true division and round-half-even.  Two codes per byte, the even
    column in the low nibble.  Returns (codes uint8 [N,K/2], scale bits uint16 [N,K/G],
    zero bits uint16 [N,K/G])."""
    W = np.asarray(W, dtype=np.float32)
    N, K = W.shape
    if K % G or G % 2:
        raise ValueError("K must be a multiple of G and G even")
    if not np.isfinite(W).all():
        raise ValueError("non-finite weight")
    Wg = W.reshape(N, K // G, G)
    mn = Wg.min(axis=2)
    mx = Wg.max(axis=2)
    scale32 = (mx - mn) / np.float32(15.0)
    s_bits, s = round_to_16(scale32, fmt)
    z_bits, z0 = round_to_16(mn, fmt)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (Wg - z0[:, :, None]) / s[:, :, None]
    q = np.where(s[:, :, None] == 0, np.float32(0), np.rint(t))
    q = np.clip(q, 0, 15).astype(np.uint8).reshape(N, K)
    codes = (q[:, 0::2] | (q[:, 1::2] << 4)).astype(np.uint8)
    return codes, s_bits, z_bits


def unpack_codes(codes) -> np.ndarray:
    codes = np.asarray(codes, dtype=np.uint8)
    N, Kh = codes.shape
    q = np.empty((N, Kh * 2), dtype=np.uint8)
    q[:, 0::2] = codes & 0xF
    q[:, 1::2] = codes >> 4
    return q


def dequantize(codes, s_bits, z_bits, G: int, fmt: str) -> np.ndarray:
    """Dequantize(Q(w_dense))[n,c] = q[n,c] * scale[n,c/G] + zero[n,c/G], exact in fp64."""
    q = unpack_codes(codes).astype(np.float64)
    s = bits16_to_f32(s_bits, fmt).astype(np.float64)
    z = bits16_to_f32(z_bits, fmt).astype(np.float64)
    return q * np.repeat(s, G, axis=1) + np.repeat(z, G, axis=1)


def dequantize_lut(codes, lut_bits, fmt: str) -> np.ndarray:
    """Non-uniform 4-bit format: Dequantize(Q(w_dense))[n,c] = lut[n][q[n,c]], where row n of the
    weight (one output channel) has its own table of 16 values stored in a 16-bit float format
    (lut_bits: uint16 [N,16]).  Exact in fp64."""
    q = unpack_codes(codes)
    lut = bits16_to_f32(lut_bits, fmt).astype(np.float64)
    N, K = q.shape
    W = np.empty((N, K), dtype=np.float64)
    for n in range(N):
        for c in range(K):
            W[n, c] = lut[n, q[n, c]]
    return W


# --------------------------------------------------------------------------- linear layer
def effective_weight(W_deq, idx, S) -> np.ndarray:
    """Dequantize(Q(w_dense)) + w_sparse as one dense fp64 matrix (the "SparseAdd" form of the
    appendix on sparse operations): the k values S are added at flat positions idx."""
    W_eff = np.array(W_deq, dtype=np.float64, copy=True)
    if len(idx):
        np.add.at(W_eff.reshape(-1), np.asarray(idx, dtype=np.int64), np.asarray(S, dtype=np.float64))
    return W_eff


def linear_fwd(x, W_deq, idx, S, bias=None) -> np.ndarray:
    """y = x W_eff^T (+ bias) in fp64; x is [M,K], W_eff [N,K]."""
    y = np.asarray(x, dtype=np.float64) @ effective_weight(W_deq, idx, S).T
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


def linear_fwd_sparse_addmm(x, W_deq, idx, S, bias=None) -> np.ndarray:
    """The appendix's other evaluation order ("SparseAddMM"): the dense product first, then
    y[:, r] += S_e * x[:, c] for each sparse entry e = (r, c).  Same result up to rounding."""
    x = np.asarray(x, dtype=np.float64)
    W_deq = np.asarray(W_deq, dtype=np.float64)
    K = W_deq.shape[1]
    y = x @ W_deq.T
    for e, v in zip(np.asarray(idx, dtype=np.int64), np.asarray(S, dtype=np.float64)):
        y[:, e // K] += v * x[:, e % K]
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64)[None, :]
    return y


# --------------------------------------------------------------------------- sparse ZO passes
def perturb(S, gidx, seed: int, step: int, scale) -> np.ndarray:
    """S_j <- fma(scale, z_j, S_j) in fp32, z_j = gaussian(seed, step, gidx_j)  (Definition 4
    with the Section 3.4 decomposition: only the k sensitive values are touched).  `scale` is
    +eps, -2 eps, +eps in the in-place order of the seed trick, or the update scale."""
    z = gaussian(seed, step, gidx)
    return fmaf32(np.float32(scale), z, np.asarray(S, dtype=np.float32))


def projected_gradient(f_plus: float, f_minus: float, eps) -> float:
    """Definition 1: g = (f(w + eps z) - f(w - eps z)) / (2 eps), in fp64; eps is an fp32 value."""
    return (float(f_plus) - float(f_minus)) / (2.0 * float(np.float32(eps)))


def zo_update_scale(f_plus: float, f_minus: float, eps, lr) -> np.float32:
    """Definition 2 with Definition 1: the update is S <- S + scale * z with
    scale = -(lr * g), formed in fp64 from the fp32 values lr and eps and rounded once to fp32."""
    g = projected_gradient(f_plus, f_minus, eps)
    return np.float32(-(float(np.float32(lr)) * g))


def zo_sgd_step_n(loss, S, gidx, seed: int, step: int, n: int, eps, lr):
    """n-sample SPSA (Definition 1 averaged over n independent perturbations, the usual variance
    reduction of a ZO estimate; the paper's runs use n = 1): for i = 0 .. n-1, z_i is drawn for the
    counter step * n + i, both losses are evaluated around the SAME S (in the in-place order
    +eps, -2 eps, +eps, which returns S to within an ulp or two), g_i = (f+_i - f-_i) / (2 eps); then
    S <- S - (lr / n) g_i z_i for i = 0 .. n-1 in turn.  Returns (S_new, [f+_i], [f-_i], [g_i]).
    n = 1 is zo_sgd_step."""
    e = np.float32(eps)
    S = np.asarray(S, dtype=np.float32)
    fps, fms, gs = [], [], []
    for i in range(n):
        c = step * n + i
        S = perturb(S, gidx, seed, c, e)
        fps.append(float(loss(S)))
        S = perturb(S, gidx, seed, c, np.float32(-2.0) * e)
        fms.append(float(loss(S)))
        S = perturb(S, gidx, seed, c, e)
        gs.append(projected_gradient(fps[-1], fms[-1], e))
    lr_n = float(np.float32(lr)) / n
    for i in range(n):
        S = perturb(S, gidx, seed, step * n + i, np.float32(-(lr_n * gs[i])))
    return S, fps, fms, gs


def replay(S0, gidx, seed: int, log, eps, lr) -> np.ndarray:
    """Section 2.1: the run's effect on the sparse values from its log [(step_t, g_t), ...] alone.  For
    every logged step, in order: the +eps, -2 eps, +eps passes (when eps != 0: they leave S within an
    ulp or two of where it was, and a replay that wants the same bits takes the same roundings), then
    the update S <- S - lr g_t z_t of Definitions 2 and 4, z_t regenerated from (seed, step_t)."""
    S = np.asarray(S0, dtype=np.float32).copy()
    e = np.float32(eps)
    for step, g in log:
        if e != 0:
            S = perturb(S, gidx, seed, step, e)
            S = perturb(S, gidx, seed, step, np.float32(-2.0) * e)
            S = perturb(S, gidx, seed, step, e)
        S = perturb(S, gidx, seed, step, np.float32(-(float(np.float32(lr)) * float(g))))
    return S


def zo_sgd_step_16(loss, S_bits, fmt: str, gidx, seed: int, step: int, eps, lr):
    """The same step with the sparse values STORED as 16-bit floats (Section 3.5 keeps w_sparse in 16
    bits; fmt 'bf16' or 'f16').  The paper does not say where the arithmetic of a step happens for
    such storage; the reading taken: the stored values are widened to fp32 (exact), the step runs in
    fp32 as zo_sgd_step (perturbations never rounded to 16 bits), and the updated values are rounded
    to the storage format once, to nearest even.  An update smaller than half a unit in the last
    place of a stored value therefore leaves it unchanged.  Returns (bits_new, f+, f-, g)."""
    S = bits16_to_f32(S_bits, fmt)
    S, f_plus, f_minus, g = zo_sgd_step(loss, S, gidx, seed, step, eps, lr)
    bits, _ = round_to_16(S, fmt)
    return bits, f_plus, f_minus, g


def zo_sgd_step(loss, S, gidx, seed: int, step: int, eps, lr):
    """One sensitive-sparse ZO-SGD step on the k trainable values S for a loss callable
    loss(S) -> float, in the in-place order of the seed trick (Section 2.1):
        S += eps z ; f+ = loss ; S -= 2 eps z ; f- = loss ; S += eps z ;
        g = (f+ - f-) / (2 eps)                                   (Definition 1)
        S -= lr g z                                               (Definitions 2 and 4)
    z is regenerated from (seed, step, gidx) in each of the four passes.  Returns
    (S_new, f+, f-, g)."""
    e = np.float32(eps)
    S = perturb(S, gidx, seed, step, e)
    f_plus = float(loss(S))
    S = perturb(S, gidx, seed, step, np.float32(-2.0) * e)
    f_minus = float(loss(S))
    S = perturb(S, gidx, seed, step, e)
    g = projected_gradient(f_plus, f_minus, e)
    S = perturb(S, gidx, seed, step, zo_update_scale(f_plus, f_minus, e, lr))
    return S, f_plus, f_minus, g
