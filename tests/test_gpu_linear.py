"""GPU parity of szo_linear_fwd (every mode) against the fp64 oracle on seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl

pytestmark = pytest.mark.gpu

LINEAR_TOL = 2e-2      # max |y - y_ref| / max |y_ref|, bf16 inputs with fp32 accumulation


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


def make_case(N, K, G, fmt, M, rho, seed, bias=False):
    W = wl.gaussian_matrix(N, K, 0.02, seed=seed, i=1)
    nnz = int(rho * N * K)
    g = wl.student_t_gradient(N * K, 3.0, seed=seed, i=2)
    idx = so.select_mask(g * g, nnz)
    S, Wd = so.decompose(W, idx)
    if G > 0:
        codes, sb, zb = so.quantize_int4(Wd, G, fmt)
        deq = so.dequantize(codes, sb, zb, G, fmt)
    else:
        Wd = wl.bf16_round(Wd)
        codes, sb, zb, deq = Wd, None, None, Wd.astype(np.float64)
    x = wl.activation(M, K, seed=seed, i=3)
    b = wl.rng(seed, wl.PURPOSE_WEIGHTS, 77).normal(0, 0.02, N).astype(np.float32) if bias else None
    # a perturbed S, as the forward sees it inside a ZO step
    S_pert = so.perturb(S, idx, 1234, 0, np.float32(1e-3))
    return dict(N=N, K=K, G=G, fmt=fmt, M=M, idx=idx, S=S_pert, codes=codes, sb=sb, zb=zb, deq=deq, x=x, bias=b)


def upload(B, c):
    dt = torch.bfloat16 if c["fmt"] == "bf16" else torch.float16
    if c["G"] > 0:
        codes = torch.from_numpy(c["codes"]).cuda()
        sc = torch.from_numpy(c["sb"].view(np.int16)).cuda().view(dt)
        ze = torch.from_numpy(c["zb"].view(np.int16)).cuda().view(dt)
    else:
        codes, sc, ze = torch.from_numpy(c["codes"]).cuda().to(torch.bfloat16), None, None
    idx = torch.from_numpy(c["idx"]).cuda()
    bias = None if c["bias"] is None else torch.from_numpy(c["bias"]).cuda()
    plan = B.Linear(c["N"], c["K"], c["G"], codes, sc, ze, c["fmt"], idx, bias)
    return plan, torch.from_numpy(c["x"]).cuda(), torch.from_numpy(c["S"]).cuda()


def max_rel(y, ref):
    return float(np.max(np.abs(y.astype(np.float64) - ref)) / np.max(np.abs(ref)))


CASES = [
    # N, K, G, fmt, M, rho, bias
    (256, 256, 64, "f16", 256, 1e-3, False),        # tiny-config q/k/v/o
    (1024, 256, 64, "f16", 100, 1e-3, False),       # ragged M
    (256, 1024, 64, "f16", 37, 1e-3, True),
    (384, 512, 128, "bf16", 300, 1e-2, True),       # several tiles and a ragged tail in M and N
    (200, 320, 32, "bf16", 65, 5e-3, False),        # N not a multiple of the tile
    (256, 512, 0, "bf16", 130, 1e-2, False),        # dense bf16 weight (no quantization)
    (128, 64, 64, "bf16", 1, 1e-2, True),           # one token, one k-block
    (512, 4096, 128, "bf16", 16, 1e-3, False),      # few tiles, long K: every tile split along K in four parts
    (300, 4160, 64, "f16", 257, 2e-3, True),        # K-split parts of unequal length, ragged N and M
    (256, 256, 64, "bf16", 200, 5e-2, False),       # dense mask: buckets larger than the record ring
]


@pytest.mark.parametrize("N,K,G,fmt,M,rho,bias", CASES)
def test_fp32_validation_mode(B, N, K, G, fmt, M, rho, bias):
    c = make_case(N, K, G, fmt, M, rho, seed=N + K + M, bias=bias)
    plan, x, S = upload(B, c)
    ref = so.linear_fwd(c["x"], c["deq"], c["idx"], c["S"], c["bias"])
    y = plan.fwd(x, S, B.MODE_FP32_VALIDATE, torch.float32).cpu().numpy()
    # fp32 accumulation of K products: a random walk of roundings, 4 * 2^-24 * sqrt(K) bounds it with margin
    assert max_rel(y, ref) < 4 * 2.0 ** -24 * np.sqrt(K)
    y16 = plan.fwd(x.to(torch.bfloat16), S, B.MODE_FP32_VALIDATE, torch.bfloat16).float().cpu().numpy()
    assert max_rel(y16, ref) < 4e-3                                    # only the output rounding
    plan.close()


@pytest.mark.parametrize("N,K,G,fmt,M,rho,bias", CASES)
@pytest.mark.parametrize("mode", ["sparse_add", "spmm"])
def test_tensor_core_modes(B, N, K, G, fmt, M, rho, bias, mode):
    c = make_case(N, K, G, fmt, M, rho, seed=N + K + M, bias=bias)
    plan, x, S = upload(B, c)
    ref = so.linear_fwd(c["x"], c["deq"], c["idx"], c["S"], c["bias"])
    md = B.MODE_SPARSE_ADD if mode == "sparse_add" else B.MODE_SPMM
    xb = x.to(torch.bfloat16)
    y = plan.fwd(xb, S, md, torch.float32).cpu().numpy()
    assert max_rel(y, ref) < LINEAR_TOL
    assert max_rel(y, ref) < 5e-3          # in practice: bf16 weight rounding only
    yb = plan.fwd(xb, S, md, torch.bfloat16).float().cpu().numpy()
    assert max_rel(yb, ref) < LINEAR_TOL
    # determinism: bitwise-same output on a second launch
    y2 = plan.fwd(xb, S, md, torch.float32).cpu().numpy()
    assert np.array_equal(y, y2)
    assert B.device_status() == 0
    plan.close()


SKINNY_CASES = [
    # N, K, G, fmt, M, rho, bias: at most 16 tokens, K a multiple of 128 -> the weight-streaming kernel
    (256, 256, 64, "f16", 1, 1e-3, False),
    (200, 640, 32, "bf16", 5, 5e-3, True),          # N not a multiple of the 128-row tile; 5 K steps for 8 CTAs
    (512, 4096, 128, "bf16", 8, 1e-3, False),       # every CTA takes four steps
    (300, 4224, 64, "f16", 13, 2e-3, True),         # two token tiles, the second ragged; 33 K steps
    (1024, 11008, 128, "bf16", 16, 1e-3, False),    # the longest K of the 7B shapes
    (128, 128, 128, "bf16", 3, 5e-2, True),         # one K step: seven CTAs of the cluster idle; dense mask
    (512, 1024, 256, "f16", 7, 1e-3, False),        # a quantization group spans two steps
    (640, 2048, 64, "bf16", 16, 3e-2, True),        # small groups; more sparse entries per 16 rows than one chunk
    # at most four tokens, groups of a multiple of 128, at least eight K steps: the kernel with one CTA per 16 rows
    (200, 1024, 128, "bf16", 1, 5e-3, True),        # N not a multiple of 16; one step per warp
    (512, 4096, 128, "bf16", 1, 1e-3, False),       # four steps per warp: the ring exactly full
    (304, 11008, 128, "f16", 4, 2e-3, True),        # 86 steps: 10 or 11 per warp, slots refilled; four tokens
    (256, 2048, 256, "f16", 3, 3e-2, False),        # a group spans two steps; 61 entries per row: several rounds of the sparse warp
    (1024, 4096, 128, "bf16", 2, 1e-3, True),
]


@pytest.mark.parametrize("N,K,G,fmt,M,rho,bias", SKINNY_CASES)
def test_auto_mode_few_tokens(B, N, K, G, fmt, M, rho, bias):
    """SZO_MODE_AUTO with M <= 16: weight-streaming kernel, sparse term in fp32 (SparseAddMM)."""
    c = make_case(N, K, G, fmt, M, rho, seed=N + K + M, bias=bias)
    plan, x, S = upload(B, c)
    xb = x.to(torch.bfloat16)
    ref = so.linear_fwd(xb.float().cpu().numpy(), c["deq"], c["idx"], c["S"], c["bias"])
    assert plan.workspace_bytes(M, B.MODE_AUTO) == 0                   # the streaming kernel needs none
    assert plan.workspace_bytes(M, B.MODE_SPARSE_ADD) > 0
    y = plan.fwd(xb, S, B.MODE_AUTO, torch.float32).cpu().numpy()
    assert max_rel(y, ref) < LINEAR_TOL
    assert max_rel(y, ref) < 5e-3          # at most the bf16 rounding of the dequantised weight
    if G % 128 == 0:
        # scale and zero are applied to the fp32 sums of a group, the weight is never rounded to bf16:
        # what is left is fp32 accumulation
        assert max_rel(y, ref) < 1e-4
    else:
        # same bf16 weights as the pair-tile kernel: the two differ by accumulation order and by the
        # sparse term (fp32 here and in SZO_MODE_SPMM)
        y_pair = plan.fwd(xb, S, B.MODE_SPMM, torch.float32).cpu().numpy()
        assert max_rel(y, y_pair) < 1e-4
    yb = plan.fwd(xb, S, B.MODE_AUTO, torch.bfloat16).float().cpu().numpy()
    assert max_rel(yb, ref) < LINEAR_TOL
    y2 = plan.fwd(xb, S, B.MODE_AUTO, torch.float32).cpu().numpy()
    assert np.array_equal(y, y2)
    assert B.device_status() == 0
    plan.close()


def test_k_split_does_not_depend_on_the_scratch_contents(B):
    """Tiles split along K meet in the caller's workspace; whatever it held before must not matter,
    and two launches give the same bits."""
    c = make_case(512, 4096, 128, "bf16", 48, 1e-3, seed=11)
    plan, x, S = upload(B, c)
    xb = x.to(torch.bfloat16)
    y1 = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32).clone()
    assert plan._ws is not None and plan._ws.numel() > c["idx"].size * 8 + 4096      # records + split scratch
    plan._ws.fill_(0x7F)
    y2 = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32).clone()
    plan._ws.zero_()
    y3 = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32)
    assert torch.equal(y1, y2) and torch.equal(y1, y3)
    ref = so.linear_fwd(xb.float().cpu().numpy(), c["deq"], c["idx"], c["S"], c["bias"])
    assert max_rel(y1.cpu().numpy(), ref) <= LINEAR_TOL
    assert B.device_status() == 0
    plan.close()


def test_materialised_and_fused_forms_give_the_same_bits(B):
    """M >= 4096 tokens take the materialised form (effective bf16 weight written to scratch, dense
    kernel), fewer tokens the fused form; both build the same bf16 weights and accumulate in the
    same order (K = 512: no tile is split along K), so the rows they share are bit-identical."""
    c = make_case(1024, 512, 64, "bf16", 4096, 2e-3, seed=13, bias=True)
    plan, x, S = upload(B, c)
    xb = x.to(torch.bfloat16)
    y_mat = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32).clone()
    y_fused = plan.fwd(xb[:2000], S, B.MODE_SPARSE_ADD, torch.float32)
    assert torch.equal(y_mat[:2000], y_fused)
    ref = so.linear_fwd(xb.float().cpu().numpy(), c["deq"], c["idx"], c["S"], c["bias"])
    assert max_rel(y_mat.cpu().numpy(), ref) <= LINEAR_TOL
    assert B.device_status() == 0
    plan.close()


def test_special_cases_identity_input_and_sparse_only(B):
    # x = I returns W_eff^T tile by tile (exposes layout mistakes); zero codes leave the sparse term
    N, K, G = 256, 256, 64
    c = make_case(N, K, G, "bf16", K, 2e-3, seed=5)
    c["x"] = np.eye(K, dtype=np.float32)
    plan, x, S = upload(B, c)
    Weff = so.effective_weight(c["deq"], c["idx"], c["S"])
    for md in (B.MODE_FP32_VALIDATE, B.MODE_SPARSE_ADD, B.MODE_SPMM):
        y = plan.fwd(x.to(torch.bfloat16), S, md, torch.float32).cpu().numpy()
        tol = 1e-6 if md == B.MODE_FP32_VALIDATE else 2.0 ** -8
        assert np.max(np.abs(y - Weff.T)) <= tol * np.max(np.abs(Weff))
    plan.close()
    zc = dict(c)
    zc["codes"] = np.zeros_like(c["codes"])
    zc["sb"] = np.zeros_like(c["sb"])
    zc["zb"] = np.zeros_like(c["zb"])
    zc["x"] = wl.activation(64, K, seed=6)
    plan, x, S = upload(B, zc)
    ref = so.linear_fwd(zc["x"], np.zeros((N, K)), c["idx"], c["S"])
    for md in (B.MODE_FP32_VALIDATE, B.MODE_SPARSE_ADD, B.MODE_SPMM):
        y = plan.fwd(x.to(torch.bfloat16), S, md, torch.float32).cpu().numpy()
        assert max_rel(y, ref) < (1e-5 if md != B.MODE_SPARSE_ADD else 5e-3)
    plan.close()


def test_linear_argument_errors(B):
    c = make_case(64, 128, 64, "bf16", 8, 1e-2, seed=9)
    plan, x, S = upload(B, c)
    with pytest.raises(B.SzoError) as ei:
        plan.fwd(x, S, B.MODE_SPARSE_ADD, torch.float32)               # fp32 x outside validation
    assert ei.value.name == "SZO_ERR_UNSUPPORTED"
    bad = torch.from_numpy(c["idx"][::-1].copy()).cuda()
    with pytest.raises(B.SzoError) as ei:
        B.Linear(64, 128, 64, plan._keep[0], plan._keep[1], plan._keep[2], "bf16", bad)
    assert ei.value.name == "SZO_ERR_INVALID_ARG"
    with pytest.raises(B.SzoError) as ei:
        B.Linear(64, 100, 0, plan._keep[0], None, None, "bf16", None)
    assert ei.value.name == "SZO_ERR_SHAPE"
    y = plan.fwd(x[:0].to(torch.bfloat16), S, B.MODE_SPARSE_ADD, torch.float32)     # M = 0
    assert y.shape == (0, 64)
    plan.close()


LUT_CASES = [
    # N, K, fmt, M, rho, bias: non-uniform 4-bit format (codes into a per-row table of 16 values)
    (256, 256, "f16", 256, 1e-3, False),
    (384, 512, "bf16", 300, 1e-2, True),            # several tiles and a ragged tail in M and N
    (200, 320, "f16", 65, 5e-3, False),             # N not a multiple of the tile: padded table rows
    (512, 4096, "f16", 16, 1e-3, True),             # long K, few tokens: K-split tiles
    (128, 64, "bf16", 1, 0.0, False),               # one token, one k-block, no sparse entries
    # one or two tokens, at least eight 128-column steps: SZO_MODE_AUTO looks the codes up inside the few-token kernel
    (200, 1024, "f16", 1, 5e-3, True),              # N not a multiple of 16; one step per warp
    (512, 4096, "bf16", 2, 1e-3, False),
    (304, 11008, "f16", 1, 2e-3, True),             # 86 steps: several row groups per CTA, tables change with them
    # 3 to 16 tokens, K a multiple of 128: looked up inside the cluster kernel
    (200, 640, "bf16", 5, 5e-3, True),              # 5 K steps for 8 CTAs, N not a multiple of 128
    (300, 4224, "f16", 13, 2e-3, True),             # two token tiles, the second ragged
    (1024, 11008, "f16", 8, 1e-3, False),
]


def make_lut_case(N, K, fmt, M, rho, seed, bias):
    codes = wl.random_codes(N, K, seed=seed, i=4)
    lut_bits, _ = so.round_to_16(wl.random_lut(N, seed=seed, i=5), fmt)
    deq = so.dequantize_lut(codes, lut_bits, fmt)
    nnz = int(rho * N * K)
    idx = wl.sorted_random_indices(N * K, nnz, seed=seed, i=6)
    S0 = wl.rng(seed, wl.PURPOSE_WEIGHTS, 7).normal(0, 0.02, nnz).astype(np.float32)
    S = so.perturb(S0, idx, 1234, 0, np.float32(1e-3)) if nnz else S0
    x = wl.activation(M, K, seed=seed, i=3)
    b = wl.rng(seed, wl.PURPOSE_WEIGHTS, 77).normal(0, 0.02, N).astype(np.float32) if bias else None
    return dict(codes=codes, lut_bits=lut_bits, deq=deq, idx=idx, S=S, x=x, bias=b)


@pytest.mark.parametrize("N,K,fmt,M,rho,bias", LUT_CASES)
def test_lut_format_validation_and_tensor_core_modes(B, N, K, fmt, M, rho, bias):
    c = make_lut_case(N, K, fmt, M, rho, seed=N + K + M + 1, bias=bias)
    dt = torch.bfloat16 if fmt == "bf16" else torch.float16
    lut = torch.from_numpy(c["lut_bits"].view(np.int16)).cuda().view(dt)
    idx = torch.from_numpy(c["idx"]).cuda() if len(c["idx"]) else None
    b = None if c["bias"] is None else torch.from_numpy(c["bias"]).cuda()
    plan = B.Linear(N, K, 0, torch.from_numpy(c["codes"]).cuda(), None, None, fmt, idx, b, lut=lut)
    x, S = torch.from_numpy(c["x"]).cuda(), torch.from_numpy(c["S"]).cuda()
    ref = so.linear_fwd(c["x"], c["deq"], c["idx"], c["S"], c["bias"])
    y = plan.fwd(x, S, B.MODE_FP32_VALIDATE, torch.float32).cpu().numpy()
    assert max_rel(y, ref) < 4 * 2.0 ** -24 * np.sqrt(K)               # exact table values, fp32 accumulation
    xb = x.to(torch.bfloat16)
    for md in (B.MODE_SPARSE_ADD, B.MODE_AUTO):
        yt = plan.fwd(xb, S, md, torch.float32).cpu().numpy()
        assert max_rel(yt, ref) < LINEAR_TOL
        assert max_rel(yt, ref) < 5e-3                                 # bf16 rounding of the table values only
        assert np.array_equal(yt, plan.fwd(xb, S, md, torch.float32).cpu().numpy())
    yb = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.bfloat16).float().cpu().numpy()
    assert max_rel(yb, ref) < LINEAR_TOL
    with pytest.raises(B.SzoError):
        plan.fwd(xb, S, B.MODE_SPMM, torch.float32)
    assert B.device_status() == 0
    plan.close()
