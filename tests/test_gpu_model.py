"""GPU parity of the whole loss path and ZO step (szo_model_*) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import model_oracle as mo
from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl
from tests.fixtures import DecoderFixture

pytestmark = pytest.mark.gpu

LOSS_TOL = 1e-3        # relative, bf16 tensor-core path
G_TOL = 1e-3           # relative, projected gradient in the fp32 validation mode


def g_tol(g, f, eps):
    """|g_gpu - g_ref| bound: 1e-3 relative plus the resolution of the loss difference.  The
    validation path accumulates in fp32, so each loss carries an error of a fraction of
    ulp32(f); g divides the difference of two losses by 2 eps."""
    return G_TOL * abs(g) + 0.25 * float(np.spacing(np.float32(f))) / (2 * eps)


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


@pytest.fixture(scope="module")
def tiny():
    return DecoderFixture("tiny", seed=0, mask="gradient", B=4, S=64)


def build_gpu(B, fx, act, mode, loss_kind=0, quantize_on_gpu=True):
    qfun = (lambda W, G, fmt: B.szo_quantize(W, G, fmt)) if quantize_on_gpu else None
    t = fx.gpu_tensors(torch, qfun)
    S = torch.from_numpy(fx.S_init.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=act, linear_mode=mode, loss_kind=loss_kind,
                max_batch=fx.B, max_seq=fx.S)
    return m, S, t


def test_fixture_mask_and_codes_reproduced_by_the_library(B, tiny):
    """The library's own select_mask and quantize give the oracle's mask and codes bit for bit
    on the tiny decoder (k = floor(1e-3 n) per tensor from 4 accumulated squared gradients)."""
    fx = tiny
    assert len(fx.S_init) == 2092
    for l in range(fx.shape["n_layers"]):
        for nm in fx.names:
            sc = torch.from_numpy(fx.scores[l][nm].ravel()).cuda()
            k = len(fx.idx[l][nm])
            assert np.array_equal(B.szo_select_mask(sc, k).cpu().numpy(), fx.idx[l][nm])
            codes, sb, zb = fx.q[l][nm]
            gc, gs, gz = B.szo_quantize(torch.from_numpy(fx.W_dense[l][nm]).cuda(), fx.shape["group"], fx.shape["sz_fmt"])
            assert np.array_equal(gc.cpu().numpy(), codes)
            assert np.array_equal(gs.cpu().view(torch.int16).numpy().view(np.uint16), sb)
            assert np.array_equal(gz.cpu().view(torch.int16).numpy().view(np.uint16), zb)


def test_model_gidx_matches_model_order(B, tiny):
    m, S, _ = build_gpu(B, tiny, B.SZO_F32, B.MODE_FP32_VALIDATE)
    assert m.k_total == len(tiny.gidx)
    assert np.array_equal(m.gidx().cpu().numpy(), tiny.gidx)
    m.close()


def test_loss_fp32_validation_matches_oracle(B, tiny):
    fx = tiny
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    om = fx.oracle_model()
    for i in range(2):
        toks = fx.batch(i)
        ref = om.loss(om.S, toks)
        got = m.loss(torch.from_numpy(toks).cuda()).item()
        assert abs(got - ref) <= 2e-6 * abs(ref)
    m.close()


def test_ten_zo_steps_fp32_validation(B, tiny):
    """Config 1: 10 ZO-SGD steps, eps 1e-3, lr 1e-5, Philox seed 1234; per-step f+, f-, g and the
    final S against the oracle."""
    fx = tiny
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    om = fx.oracle_model()
    frozen = {k: v.clone() for k, v in m.tensors.items()}
    eps, lr = 1e-3, 1e-5
    for step in range(10):
        toks = fx.batch(step)
        fp, fm, g = mo.zo_step(om, toks, 1234, step, eps, lr)
        out = m.zo_step(torch.from_numpy(toks).cuda(), 1234, step, eps, lr).cpu().numpy()
        assert abs(out[0] - fp) <= 2e-6 * abs(fp) and abs(out[1] - fm) <= 2e-6 * abs(fm)
        # g amplifies the loss error by f / (f+ - f-); the bound is relative to the gradient scale
        assert abs(out[2] - g) <= g_tol(g, fp, eps), (step, out[2], g)
    assert np.allclose(S.cpu().numpy(), om.S, rtol=0, atol=2e-7)
    assert m.last_launches() > 0
    for k, v in frozen.items():                      # frozen parts are bit-identical after the steps
        assert torch.equal(v, m.tensors[k]), k
    assert B.device_status() == 0
    m.close()


@pytest.mark.parametrize("name,loss_kind", [("tiny_opt", 0), ("tiny_gqa", 1), ("tiny_lut", 0)])
def test_other_architectures_fp32_validation(B, name, loss_kind):
    fx = DecoderFixture(name, seed=1, mask="random", B=3, S=32)
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE, loss_kind, quantize_on_gpu=fx.shape["group"] > 0)
    om = fx.oracle_model()
    toks = fx.batch(0)
    kind = "lm" if loss_kind == 0 else "cls2"
    labels = wl.binary_labels(fx.B, 1, 0)
    cand = np.array([11, 301], np.int32)
    ref = om.loss(om.S, toks, kind, labels, cand)
    d = lambda a: torch.from_numpy(a).cuda()
    got = m.loss(d(toks), d(labels), d(cand)).item()
    assert abs(got - ref) <= 3e-6 * abs(ref)
    fp, fm, g = mo.zo_step(om, toks, 7, 3, 1e-3, 1e-4, kind, labels, cand)
    out = m.zo_step(d(toks), 7, 3, 1e-3, 1e-4, d(labels), d(cand)).cpu().numpy()
    assert abs(out[0] - fp) <= 3e-6 * abs(fp) and abs(out[1] - fm) <= 3e-6 * abs(fm)
    assert abs(out[2] - g) <= g_tol(g, fp, 1e-3)
    assert np.allclose(S.cpu().numpy(), om.S, rtol=0, atol=2e-7)
    m.close()


@pytest.mark.parametrize("mode", ["sparse_add", "spmm"])
def test_bf16_tensor_core_path_losses(B, tiny, mode):
    fx = tiny
    md = B.MODE_SPARSE_ADD if mode == "sparse_add" else B.MODE_SPMM
    m, S, _ = build_gpu(B, fx, B.SZO_BF16, md)
    om = fx.oracle_model()
    for step in range(3):
        toks = fx.batch(step)
        fp, fm, g = mo.zo_step(om, toks, 1234, step, 1e-3, 1e-5)
        out = m.zo_step(torch.from_numpy(toks).cuda(), 1234, step, 1e-3, 1e-5).cpu().numpy()
        assert abs(out[0] - fp) <= LOSS_TOL * abs(fp) and abs(out[1] - fm) <= LOSS_TOL * abs(fm)
        assert np.isfinite(out[2])
        om.S = S.cpu().numpy().copy()      # follow the GPU's own trajectory (g differs at bf16)
    assert B.device_status() == 0
    m.close()


def test_host_buffer_step_equals_device_step(B, tiny):
    fx = tiny
    m1, S1, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    m2, S2, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    toks = fx.batch(0)
    a = m1.zo_step(torch.from_numpy(toks).cuda(), 1, 0, 1e-3, 1e-5).cpu().numpy()
    b = m2.zo_step_host(torch.from_numpy(toks).pin_memory(), 1, 0, 1e-3, 1e-5)
    assert tuple(a) == tuple(b) and torch.equal(S1, S2)
    m1.close()
    m2.close()


def test_model_argument_errors(B, tiny):
    m, S, _ = build_gpu(B, tiny, B.SZO_F32, B.MODE_FP32_VALIDATE)
    toks = torch.zeros((tiny.B + 1, tiny.S), dtype=torch.int32, device="cuda")
    with pytest.raises(B.SzoError) as ei:
        m.loss(toks)
    assert ei.value.name == "SZO_ERR_SHAPE"
    m.close()


@pytest.mark.parametrize("B_,S,H,Hkv,hd", [(2, 64, 4, 4, 64), (1, 256, 4, 2, 128), (3, 100, 2, 1, 128), (2, 37, 4, 2, 64),
                                           (1, 200, 8, 8, 64)])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_attention_matches_oracle(B, B_, S, H, Hkv, hd, dtype):
    g = wl.rng(3, wl.PURPOSE_ACTIVATION, S + hd)
    mk = lambda heads: wl.bf16_round(g.standard_normal((B_ * S, heads * hd)).astype(np.float32))
    q, k, v = mk(H), mk(Hkv), mk(Hkv)
    t64 = lambda a, heads: torch.from_numpy(a.astype(np.float64)).view(B_, S, heads, hd)
    ref = mo.causal_attention(t64(q, H), t64(k, Hkv), t64(v, Hkv)).reshape(B_ * S, H * hd).numpy()
    dt = torch.bfloat16 if dtype == "bf16" else torch.float32
    d = lambda a: torch.from_numpy(a).cuda().to(dt)
    got = B.szo_attention(d(q), d(k), d(v), B_, S, H, Hkv, hd).float().cpu().numpy()
    tol = 1.5e-2 if dtype == "bf16" else 2e-6          # bf16: probabilities and outputs are rounded to bf16
    assert np.max(np.abs(got - ref)) <= tol * np.max(np.abs(ref))


@pytest.mark.parametrize("name,loss_kind,mode", [("tiny_opt", 0, "sparse_add"), ("tiny_gqa", 1, "sparse_add"),
                                                 ("tiny_gqa", 0, "spmm"), ("tiny_lut", 0, "sparse_add")])
def test_other_architectures_bf16_tensor_core_path(B, name, loss_kind, mode):
    """OPT-shaped (LayerNorm, biases, ReLU, learned positions, int4) and Mistral-shaped (GQA, dense bf16
    weights, 1 % mask) decoders, and the tiny decoder in the non-uniform 4-bit format, on the
    tensor-core path: losses within 1e-3 of the oracle."""
    fx = DecoderFixture(name, seed=2, mask="random", B=3, S=48)
    md = B.MODE_SPARSE_ADD if mode == "sparse_add" else B.MODE_SPMM
    m, S, _ = build_gpu(B, fx, B.SZO_BF16, md, loss_kind, quantize_on_gpu=fx.shape["group"] > 0)
    om = fx.oracle_model()
    toks = fx.batch(0)
    kind = "lm" if loss_kind == 0 else "cls2"
    labels = wl.binary_labels(fx.B, 2, 0)
    cand = np.array([5, 77], np.int32)
    d = lambda a: torch.from_numpy(a).cuda()
    fp, fm, g = mo.zo_step(om, toks, 9, 1, 1e-3, 1e-4, kind, labels, cand)
    out = m.zo_step(d(toks), 9, 1, 1e-3, 1e-4, d(labels), d(cand)).cpu().numpy()
    # The LM loss averages B*(S-1) positions.  The 2-candidate loss of three sequences does not: it is
    # softplus(+-(l1 - l0)) of two logits of size ~0.3 whose bf16-path error is ~1.5e-3 absolute
    # (activations carry 2^-9 relative rounding), and |d loss / d (l1 - l0)| <= 1/2, i.e. about
    # 1.2e-3 of a loss near ln 2: the bound for that case is 3e-3.
    tol = LOSS_TOL if loss_kind == 0 else 3e-3
    assert abs(out[0] - fp) <= tol * abs(fp) and abs(out[1] - fm) <= tol * abs(fm)
    assert np.isfinite(out[2]) and B.device_status() == 0
    m.close()


def test_resident_and_materialised_forms_at_test_size():
    """The forms that large token counts select (int4: effective weight materialised per launch group;
    dense bf16: effective weight resident per launch group, masked entries rewritten per forward) are
    forced at test size, where the oracle can check them: SZO_LINEAR_MATERIALISE=1 is read once per
    process, so the oracle-parity tests of the three architectures run again in a child process."""
    import os
    import subprocess
    import sys
    env = dict(os.environ, SZO_LINEAR_MATERIALISE="1")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-m", "pytest", "-x", "-q", "-m", "gpu", "-p", "no:cacheprovider",
                          os.path.join(root, "tests", "test_gpu_model.py"), "-k",
                          "test_other_architectures_bf16_tensor_core_path or test_bf16_tensor_core_path_losses "
                          "or test_host_buffer_step_equals_device_step"],
                         cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-2000:]
    assert " passed" in res.stdout


@pytest.mark.parametrize("name,rho", [("tiny_gqa", 1.6e-5), ("tiny", 1.6e-5), ("tiny", 0.0), ("tiny_gqa", 0.0)])
def test_degenerate_masks(B, name, rho):
    """Linears without a single sensitive entry next to linears with one or two (rho * n < 1 for the
    narrow k/v projections), and a model with no sensitive entry at all (k = 0: both perturbed losses
    equal the unperturbed one, g = 0, nothing to update), on the fp32 validation path against the
    oracle and on the tensor-core path."""
    fx = DecoderFixture(name, seed=1, mask="random", B=2, S=32, rho=rho)
    om = fx.oracle_model()
    toks = fx.batch(0)
    fp, fm, g = mo.zo_step(om, toks, 7, 3, 1e-3, 1e-4, "lm", None, None)
    d = lambda a: torch.from_numpy(a).cuda()
    for act, mode, tol in ((B.SZO_F32, B.MODE_FP32_VALIDATE, 3e-6), (B.SZO_BF16, B.MODE_SPARSE_ADD, LOSS_TOL)):
        t = fx.gpu_tensors(torch, None)
        for key in [k for k, v in t.items() if k.endswith(".idx") and v.numel() == 0]:
            del t[key]                                  # a linear without entries passes no index list
        S = torch.from_numpy(fx.S_init.copy()).cuda() if len(fx.S_init) else torch.zeros(0, device="cuda")
        m = B.Model(fx.shape, fx.names, t, S, act_dtype=act, linear_mode=mode, loss_kind=0, max_batch=fx.B, max_seq=fx.S)
        assert m.k_total == len(fx.S_init)
        out = m.zo_step(d(toks), 7, 3, 1e-3, 1e-4).cpu().numpy()
        assert abs(out[0] - fp) <= tol * abs(fp) and abs(out[1] - fm) <= tol * abs(fm)
        if rho == 0.0:
            assert out[0] == out[1] and out[2] == 0.0
        elif mode == B.MODE_FP32_VALIDATE:
            assert abs(out[2] - g) <= g_tol(g, fp, 1e-3)
            assert np.allclose(S.cpu().numpy(), om.S, rtol=0, atol=2e-7)
        assert B.device_status() == 0
        m.close()


@pytest.mark.parametrize("act,mode", [("f32", "fp32"), ("bf16", "paired")])
def test_two_half_batches_through_losses_and_apply_equal_the_full_batch_step(B, tiny, act, mode):
    """Data-parallel replicas emulated in one process: szo_model_zo_losses on each half of the batch
    (both from the same S, as two replicas would), the two (sum f+, sum f-, count) added, then
    szo_model_zo_apply, against szo_model_zo_step on the whole batch.  fp32 validation path: the same
    per-position losses in another summation order.  Paired bf16 path: the same kernels on other tile
    shapes, compared at the loss tolerance."""
    fx = tiny
    a, md = (B.SZO_F32, B.MODE_FP32_VALIDATE) if mode == "fp32" else (B.SZO_BF16, B.MODE_PAIRED)
    toks = torch.from_numpy(fx.batch(0)).cuda()
    eps, lr = 1e-3, 1e-3
    m_full, S_full, _ = build_gpu(B, fx, a, md)
    out_full = m_full.zo_step(toks, 1234, 3, eps, lr).cpu().numpy().copy()
    m_dp, S_dp, _ = build_gpu(B, fx, a, md)
    S0 = S_dp.clone()
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")
    for half in (toks[:2].contiguous(), toks[2:].contiguous()):
        S_dp.copy_(S0)                                   # every replica starts the step from the same S
        sums += m_dp.zo_losses(half, 1234, 3, eps)
    assert float(sums[2]) == fx.B * (fx.S - 1)
    out_dp = m_dp.zo_apply(eps, lr, sums).cpu().numpy().copy()
    tol = 1e-12 if mode == "fp32" else 2e-5
    assert abs(out_dp[0] - out_full[0]) <= tol * abs(out_full[0]) and abs(out_dp[1] - out_full[1]) <= tol * abs(out_full[1])
    gtol = 1e-8 if mode == "fp32" else 2e-2
    assert abs(out_dp[2] - out_full[2]) <= gtol * abs(out_full[2]), (out_dp, out_full)
    assert torch.allclose(S_dp, S_full, rtol=0, atol=1e-9 if mode == "fp32" else abs(lr * out_full[2]) * 0.1)
    with pytest.raises(B.SzoError):                      # apply without a preceding losses call
        m_dp.zo_apply(eps, lr, sums)
    assert B.device_status() == 0
    m_full.close()
    m_dp.close()


def test_replay_from_the_g_log_reproduces_the_sparse_values(B, tiny):
    """Five steps on the fp32 validation path, their (step, g) pairs logged; szo_replay from S_0 gives the
    run's final S bit for bit (with the +-eps passes replayed), and the oracle's replay of the same log
    agrees to the accuracy of z."""
    fx = tiny
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    S0 = S.clone()
    eps, lr = 1e-3, 1e-3
    log = []
    for step in (0, 1, 2, 7, 8):
        out = m.zo_step(torch.from_numpy(fx.batch(step)).cuda(), 1234, step, eps, lr).cpu().numpy()
        log.append((step, float(out[2])))
    S_rep = S0.clone()
    B.szo_replay(S_rep, m.gidx(), 0, 1234, log, eps, lr)
    assert torch.equal(S_rep, S)
    ref = so.replay(S0.cpu().numpy(), fx.gidx, 1234, log, eps, lr)
    assert np.allclose(S_rep.cpu().numpy(), ref, rtol=0, atol=5e-7)
    S_plain = S0.clone()
    B.szo_replay(S_plain, m.gidx(), 0, 1234, log, 0.0, lr)
    assert torch.allclose(S_plain, S, rtol=0, atol=1e-6) and not torch.equal(S_plain, S0)
    m.close()


def test_n_sample_spsa_step_matches_the_oracle(B, tiny):
    """szo_model_zo_step_n with n = 3 on the fp32 validation path against the oracle's n-sample step
    (losses, the three projected gradients, the updated S); n = 1 equals szo_model_zo_step."""
    fx = tiny
    toks = fx.batch(0)
    eps, lr = 1e-3, 1e-3
    om = fx.oracle_model()
    S_ref, fps, fms, gs = so.zo_sgd_step_n(lambda S_: om.loss(S_, toks), om.S, om.gidx, 1234, 2, 3, eps, lr)
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    out = m.zo_step_n(torch.from_numpy(toks).cuda(), 1234, 2, 3, eps, lr).cpu().numpy()
    for i in range(3):
        assert abs(out[0, i] - fps[i]) <= 2e-6 * abs(fps[i]) and abs(out[1, i] - fms[i]) <= 2e-6 * abs(fms[i])
        assert abs(out[2, i] - gs[i]) <= g_tol(gs[i], fps[i], eps)
    assert np.allclose(S.cpu().numpy(), S_ref, rtol=0, atol=3e-7)
    m1, S1, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    m2, S2, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    a = m1.zo_step_n(torch.from_numpy(toks).cuda(), 1234, 5, 1, eps, lr).cpu().numpy()[:, 0]
    b = m2.zo_step(torch.from_numpy(toks).cuda(), 1234, 5, eps, lr).cpu().numpy()
    assert tuple(a) == tuple(b) and torch.equal(S1, S2)
    for mm in (m, m1, m2):
        mm.close()


@pytest.mark.parametrize("fmt", ["f16", "bf16"])
def test_sparse_values_stored_in_16_bits(B, tiny, fmt):
    """Section 3.5 (w_sparse in 16 bits): szo_round_sparse16 against the oracle's rounding bit for bit, and three
    steps of a model whose sparse values are stored in the format: after every step S holds representable values,
    the mirror holds their bits, and S agrees with the oracle's zo_sgd_step_16 to the difference of the two fp32
    updates (lr |z| times the tolerance on g) plus the one unit in the last place by which values on different
    sides of a rounding boundary part."""
    fx = tiny
    x = torch.from_numpy(wl.rng(3, wl.PURPOSE_WEIGHTS, 1).normal(0, 0.05, 100003).astype(np.float32)).cuda()
    x[:4] = torch.tensor([0.0, -0.0, 65519.9, 1e-9], device="cuda")
    ref_bits, ref_vals = so.round_to_16(x.cpu().numpy(), fmt)
    dt16 = torch.float16 if fmt == "f16" else torch.bfloat16
    mirror = torch.zeros(x.numel(), dtype=dt16, device="cuda")
    B.szo_round_sparse16(x, fmt, mirror)
    assert np.array_equal(x.cpu().numpy().view(np.uint32), ref_vals.view(np.uint32))
    assert np.array_equal(mirror.cpu().view(torch.int16).numpy().view(np.uint16), ref_bits)

    toks = fx.batch(0)
    eps, lr = 1e-3, 3e-3
    om = fx.oracle_model()
    m, S, _ = build_gpu(B, fx, B.SZO_F32, B.MODE_FP32_VALIDATE)
    S16 = torch.zeros(S.numel(), dtype=dt16, device="cuda")
    m.set_sparse_storage(fmt, S16)
    bits = so.round_to_16(om.S, fmt)[0]
    assert np.array_equal(S16.cpu().view(torch.int16).numpy().view(np.uint16), bits)       # the call rounds the current S
    bits0 = bits.copy()
    for step in range(3):
        bits, fp, fm, g = so.zo_sgd_step_16(lambda S_: om.loss(S_, toks), bits, fmt, om.gidx, 1234, step, eps, lr)
        out = m.zo_step(torch.from_numpy(toks).cuda(), 1234, step, eps, lr).cpu().numpy()
        assert abs(out[0] - fp) <= 2e-6 * abs(fp) and abs(out[2] - g) <= g_tol(g, fp, eps)
        got = S.cpu().numpy()
        got_bits = S16.cpu().view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(so.round_to_16(got, fmt)[1].view(np.uint32), got.view(np.uint32))     # representable
        assert np.array_equal(so.round_to_16(got, fmt)[0], got_bits)                                 # the mirror
        ref = so.bits16_to_f32(bits, fmt)
        ulp = np.abs(so.bits16_to_f32(bits + np.uint16(1), fmt) - ref)
        slack = lr * 6.0 * g_tol(g, fp, eps) + 2e-7              # |z| < 6; the in-place order's own ulps of fp32
        excess = np.abs(got.astype(np.float64) - ref) - ulp - slack
        assert excess.max() <= 0, (step, excess.max(), int(np.argmax(excess)))
        assert np.mean(got_bits == bits) > 0.9, (step, np.mean(got_bits == bits))
        bits = got_bits.copy()                                   # the next step starts from the library's values
    assert np.mean(bits != bits0) > 0.3                          # the updates are large enough to show in 16 bits
    m.set_sparse_storage(None)
    m.close()
