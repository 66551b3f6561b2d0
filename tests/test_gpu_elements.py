"""GPU parity: szo_perturb / szo_update / szo_projected_gradient / szo_quantize / szo_select_mask
through the C ABI against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


def _z_tol(z_ref):
    return 1e-6 * np.maximum(1.0, np.abs(z_ref.astype(np.float64)))


@pytest.mark.parametrize("k", [1, 2, 7, 4096, 100_003])
def test_perturb_matches_oracle(B, k):
    n = 12_582_912_000                                      # OPT-13B linear parameter count (> 2^32)
    idx = wl.sorted_random_indices(n, k, seed=1, i=k)
    S = wl.rng(2, wl.PURPOSE_WEIGHTS, k).normal(0, 0.02, k).astype(np.float32)
    seed, step, base = 0x1234_5678_9ABC_DEF0, 3 + (1 << 33), 17
    d_idx = torch.from_numpy(idx).cuda()
    d_S = torch.from_numpy(S).cuda()
    # z itself: S_in = 0, scale = 1  ->  S_out = z exactly
    zero = torch.zeros_like(d_S)
    out = torch.empty_like(d_S)
    B.szo_perturb(zero, out, d_idx, base, seed, step, 1.0)
    z = out.cpu().numpy()
    z_ref = so.gaussian(seed, step, idx + base)
    assert np.all(np.abs(z.astype(np.float64) - z_ref) <= _z_tol(z_ref))
    # the axpy with the GPU's own z is a single fp32 fma (bit-exact), out of place
    eps = np.float32(1e-3)
    B.szo_perturb(d_S, out, d_idx, base, seed, step, float(eps))
    assert np.array_equal(out.cpu().numpy().view(np.uint32), so.fmaf32(eps, z, S).view(np.uint32))
    assert np.array_equal(d_S.cpu().numpy(), S)                          # input untouched
    ref = so.perturb(S, idx + base, seed, step, eps)
    assert np.all(np.abs(out.cpu().numpy().astype(np.float64) - ref) <= 3e-8)


def test_perturb_in_place_sequence_and_canaries(B):
    k = 33_333
    idx = wl.sorted_random_indices(16_777_216, k, seed=3)
    S = wl.rng(4, wl.PURPOSE_WEIGHTS).normal(0, 0.02, k).astype(np.float32)
    buf = torch.full((k + 64,), 7.25, dtype=torch.float32, device="cuda")    # canaries on both sides
    view = buf[32:32 + k]
    view.copy_(torch.from_numpy(S))
    d_idx = torch.from_numpy(idx).cuda()
    eps = np.float32(1e-3)
    ref = S.copy()
    z0 = torch.zeros(k, device="cuda")
    zbuf = torch.empty(k, device="cuda")
    B.szo_perturb(z0, zbuf, d_idx, 0, 1234, 5, 1.0)
    z = zbuf.cpu().numpy()
    for sc in (eps, np.float32(-2.0) * eps, eps):                 # +eps, -2eps, +eps (seed trick order)
        B.szo_perturb(view, view, d_idx, 0, 1234, 5, float(sc))
        ref = so.fmaf32(sc, z, ref)
        assert np.array_equal(view.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    full = buf.cpu().numpy()
    assert (full[:32] == 7.25).all() and (full[32 + k:] == 7.25).all()
    assert np.max(np.abs(ref - S)) <= 2 * np.spacing(np.float32(0.25))


def test_update_and_projected_gradient(B):
    k = 5001
    idx = wl.sorted_random_indices(1 << 24, k, seed=5)
    S = wl.rng(6, wl.PURPOSE_WEIGHTS).normal(0, 0.02, k).astype(np.float32)
    f = torch.tensor([6.931471805599453, 6.931099123], dtype=torch.float64, device="cuda")
    g = torch.zeros(1, dtype=torch.float64, device="cuda")
    eps, lr = np.float32(1e-3), np.float32(1e-5)
    B.szo_projected_gradient(f[0:1], f[1:2], float(eps), g)
    g_ref = so.projected_gradient(6.931471805599453, 6.931099123, eps)
    assert g.item() == g_ref
    d_S = torch.from_numpy(S).cuda()
    d_idx = torch.from_numpy(idx).cuda()
    zbuf = torch.empty(k, device="cuda")
    B.szo_perturb(torch.zeros(k, device="cuda"), zbuf, d_idx, 99, 42, 7, 1.0)
    B.szo_update(d_S, d_idx, 99, 42, 7, float(lr), f[0:1], f[1:2], float(eps))
    sc = so.zo_update_scale(6.931471805599453, 6.931099123, eps, lr)
    ref = so.fmaf32(sc, zbuf.cpu().numpy(), S)
    assert np.array_equal(d_S.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    full = so.perturb(S, idx + 99, 42, 7, sc)
    assert np.allclose(d_S.cpu().numpy(), full, rtol=0, atol=1e-12 + abs(float(sc)) * 1e-5)


@pytest.mark.parametrize("k", [1, 3, 8, 4099, 250_001])
def test_kept_z_passes_equal_the_regenerating_ones(B, k):
    """First pass keeps z; the -2 eps pass, the restore and the update then read it.  Every result
    must be bit-identical to the regenerating entry points (same z, same single fma)."""
    n = 6_476_005_376
    idx = torch.from_numpy(wl.sorted_random_indices(n, k, seed=21, i=k)).cuda()
    S0 = torch.from_numpy(wl.rng(22, wl.PURPOSE_WEIGHTS, k).normal(0, 0.02, k).astype(np.float32)).cuda()
    seed, step, eps, lr = 99, 7, 1e-3, 1e-4
    f = torch.tensor([0.70, 0.69], dtype=torch.float64, device="cuda")
    a, b = S0.clone(), S0.clone()
    z = torch.full((k,), 123.0, device="cuda")
    zref = torch.empty(k, device="cuda")
    B.szo_perturb(torch.zeros(k, device="cuda"), zref, idx, 5, seed, step, 1.0)        # z itself
    B.szo_perturb(a, a, idx, 5, seed, step, eps)
    B.szo_perturb_keep_z(b, b, idx, 5, seed, step, eps, z)
    assert torch.equal(a, b) and torch.equal(z, zref)
    z_ref = so.gaussian(seed, step, idx.cpu().numpy() + 5)
    assert np.all(np.abs(z.cpu().numpy().astype(np.float64) - z_ref) <= _z_tol(z_ref))
    for sc in (-2e-3, 1e-3):
        B.szo_perturb(a, a, idx, 5, seed, step, sc)
        B.szo_perturb_kept_z(b, b, z, sc)
        assert torch.equal(a, b)
    B.szo_update(a, idx, 5, seed, step, lr, f[0:1], f[1:2], eps)
    B.szo_update_kept_z(b, z, lr, f[0:1], f[1:2], eps)
    assert torch.equal(a, b)
    out = torch.empty_like(b)                                                          # out of place
    B.szo_perturb_kept_z(b, out, z, 0.5)
    assert np.array_equal(out.cpu().numpy().view(np.uint32),
                          so.fmaf32(np.float32(0.5), z.cpu().numpy(), b.cpu().numpy()).view(np.uint32))


@pytest.mark.parametrize("k", [1, 7, 8, 4099, 250_001])
def test_three_passes_in_one_launch_equal_the_three_launches(B, k):
    """szo_perturb3_keep_z: the +eps, -2 eps, +eps passes of one (seed, step) in one launch leave the bits of
    the three separate launches in S, in S_plus / S_minus (where asked for) and in z; in place and out of place."""
    n = 6_476_005_376
    idx = torch.from_numpy(wl.sorted_random_indices(n, k, seed=31, i=k)).cuda()
    S0 = torch.from_numpy(wl.rng(32, wl.PURPOSE_WEIGHTS, k).normal(0, 0.02, k).astype(np.float32)).cuda()
    seed, step, eps = 99, 11, 1e-3
    a = S0.clone()
    z = torch.empty(k, device="cuda")
    B.szo_perturb_keep_z(a, a, idx, 5, seed, step, eps, z)
    plus = a.clone()
    B.szo_perturb_kept_z(a, a, z, -2.0 * eps)
    minus = a.clone()
    B.szo_perturb_kept_z(a, a, z, eps)
    b, z3 = S0.clone(), torch.full((k,), 7.0, device="cuda")
    B.szo_perturb3_keep_z(b, b, idx, 5, seed, step, eps, z3)                    # in place, no copies asked for
    assert torch.equal(a, b) and torch.equal(z, z3)
    out, p3, m3 = torch.empty_like(S0), torch.empty_like(S0), torch.empty_like(S0)
    B.szo_perturb3_keep_z(S0, out, idx, 5, seed, step, eps, z3, p3, m3)           # out of place, both copies
    assert torch.equal(out, a) and torch.equal(p3, plus) and torch.equal(m3, minus)
    ref = so.perturb(so.perturb(so.perturb(S0.cpu().numpy(), idx.cpu().numpy() + 5, seed, step, np.float32(eps)),
                                idx.cpu().numpy() + 5, seed, step, np.float32(-2.0) * np.float32(eps)),
                     idx.cpu().numpy() + 5, seed, step, np.float32(eps))
    assert np.allclose(out.cpu().numpy(), ref, rtol=0, atol=1e-8)               # (z agrees to 5e-7, eps = 1e-3: an ulp of S or two)
    assert B.device_status() == 0


def test_perturb_empty_and_bad_arguments(B):
    e = torch.empty(0, device="cuda")
    B.szo_perturb(e, e, torch.empty(0, dtype=torch.int64, device="cuda"), 0, 1, 1, 1.0)
    S = torch.zeros(16, device="cuda")
    idx = torch.arange(16, dtype=torch.int64, device="cuda")
    with pytest.raises(B.SzoError) as ei:
        B.szo_perturb(S[1:], S[1:], idx[:15], 0, 1, 1, 1.0)            # misaligned
    assert ei.value.name == "SZO_ERR_ALIGNMENT"
    with pytest.raises(B.SzoError):
        B.szo_perturb(S, S, idx, -5, 1, 1, 1.0)


@pytest.mark.parametrize("N,K,G,fmt,wdt", [(64, 256, 64, "f16", torch.float32), (96, 4096, 128, "bf16", torch.float32),
                                           (33, 320, 32, "bf16", torch.float32), (16, 512, 128, "bf16", torch.bfloat16),
                                           (40, 384, 32, "f16", torch.float32), (8, 512, 256, "bf16", torch.float32)])
def test_quantize_bit_exact(B, N, K, G, fmt, wdt):
    W = wl.gaussian_matrix(N, K, 0.02, seed=7, i=N)
    if wdt == torch.bfloat16:
        W = wl.bf16_round(W)
    idx = wl.sorted_random_indices(N * K, max(1, N * K // 1000), seed=8)
    _, Wd = so.decompose(W, idx)
    Wd[1, :G] = 0.03125                                       # constant group -> scale 0
    codes, sb, zb = so.quantize_int4(Wd, G, fmt)
    dW = torch.from_numpy(Wd).cuda().to(wdt)
    g_codes, g_s, g_z = B.szo_quantize(dW, G, fmt)
    assert np.array_equal(g_codes.cpu().numpy(), codes)
    assert np.array_equal(g_s.cpu().view(torch.int16).numpy().view(np.uint16), sb)
    assert np.array_equal(g_z.cpu().view(torch.int16).numpy().view(np.uint16), zb)


def test_quantize_rejects_bad_shapes(B):
    W = torch.zeros((4, 100), device="cuda")
    with pytest.raises(B.SzoError) as ei:
        B.szo_quantize(W, 64, "bf16")
    assert ei.value.name == "SZO_ERR_SHAPE"


@pytest.mark.parametrize("n,k", [(1, 1), (37, 5), (8192, 8), (8193, 8193), (1_000_003, 1000), (16_777_216, 16_777)])
def test_select_mask_matches_oracle(B, n, k):
    g = wl.student_t_gradient(n, 3.0, seed=9, i=n % 1000)
    scores = (g * g).astype(np.float32)
    got = B.szo_select_mask(torch.from_numpy(scores).cuda(), k).cpu().numpy()
    assert np.array_equal(got, so.select_mask(scores, k))


def test_select_mask_ties_zero_k_and_nan(B):
    n = 50_000
    scores = wl.rng(10, wl.PURPOSE_SCORES).integers(0, 6, n).astype(np.float32)      # heavy ties
    for k in (0, 1, 777, 25_000, n):
        got = B.szo_select_mask(torch.from_numpy(scores).cuda(), k).cpu().numpy()
        assert np.array_equal(got, so.select_mask(scores, k))
    same = np.ones(10_000, np.float32)
    assert np.array_equal(B.szo_select_mask(torch.from_numpy(same).cuda(), 100).cpu().numpy(), np.arange(100))
    z = np.array([0.0, -0.0, 0.0, 1.0] * 4, np.float32)
    assert np.array_equal(B.szo_select_mask(torch.from_numpy(z).cuda(), 6).cpu().numpy(), so.select_mask(z, 6))
    bad = scores.copy()
    bad[123] = np.nan
    with pytest.raises(B.SzoError) as ei:
        B.szo_select_mask(torch.from_numpy(bad).cuda(), 5)
    assert ei.value.name == "SZO_ERR_NONFINITE"
    with pytest.raises(B.SzoError):
        B.szo_select_mask(torch.from_numpy(same).cuda(), same.size + 1)


def test_bounded_wait_gives_up_and_reports_a_timeout(B):
    """A wait inside a kernel that nothing will ever satisfy (a barrier without an arrival, limit 2 ms):
    the kernel returns, the device status word holds SZO_ERR_TIMEOUT once, and the library keeps
    working afterwards (the K-split tickets of every plan are cleared before its next launch)."""
    import numpy as np
    from oracle import szo_oracle as so
    from tests.test_gpu_linear import make_case, max_rel, upload
    assert B.device_status() == 0
    c = make_case(512, 4096, 128, "bf16", 16, 1e-3, seed=5)           # every tile split along K: uses tickets
    plan, x, S = upload(B, c)
    ref = so.linear_fwd(c["x"], c["deq"], c["idx"], c["S"], c["bias"])
    xb = x.to(torch.bfloat16)
    y0 = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32).cpu().numpy()
    assert B.selftest_wait_timeout(2.0) == 1
    assert B.device_status() == -8
    assert B.device_status() == 0
    y1 = plan.fwd(xb, S, B.MODE_SPARSE_ADD, torch.float32).cpu().numpy()
    assert np.array_equal(y0, y1) and max_rel(y1, ref) < 5e-3
    assert B.device_status() == 0
    plan.close()
