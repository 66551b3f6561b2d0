"""GPU parity of the paired form (centre / half-difference of a ZO step's two forwards) against the
fp64 oracle: the linear layer, the attention, and whole steps, where the quantity under test is the
projected gradient g of Definition 1 on the bf16 tensor-core path."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import model_oracle as mo
from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl
from tests.fixtures import DecoderFixture
from tests.test_gpu_linear import make_case, max_rel, upload

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


def paired_rows(B, c_rows, d_rows):
    """[centre rows | gap | half-difference rows] as one bf16 CUDA tensor."""
    M = c_rows.shape[0]
    row0 = B.paired_row0(M)
    buf = np.zeros((row0 + M, c_rows.shape[1]), np.float32)
    buf[:M] = c_rows
    buf[row0:] = d_rows
    return torch.from_numpy(buf).cuda().to(torch.bfloat16), row0


PAIRED_LINEAR_CASES = [
    # N, K, G, fmt, M, rho, bias
    (256, 256, 64, "f16", 256, 1e-3, False),
    (1024, 256, 64, "f16", 100, 1e-3, True),        # ragged M, bias (centre rows only)
    (384, 512, 128, "bf16", 300, 1e-2, True),       # two token tiles per part, ragged N
    (200, 320, 32, "bf16", 65, 5e-3, False),
    (256, 512, 0, "bf16", 130, 1e-2, True),         # dense bf16 weight
    (512, 4096, 128, "bf16", 16, 1e-3, False),      # every tile split along K
    (300, 4160, 64, "f16", 257, 2e-3, True),
    (256, 256, 64, "bf16", 200, 5e-2, False),       # 13 entries per weight row
    (1280, 1024, 128, "bf16", 2600, 2e-3, False),   # more tiles than clusters: full rounds and a tail
    (2080, 512, 128, "bf16", 2100, 1e-3, False),    # sparse product: slabs of 16 tokens, the last one ragged
    (72, 16384, 128, "bf16", 24, 1e-3, False),      # ... of four tokens: K too wide for eight
    (251, 512, 128, "bf16", 50, 1e-3, False),       # odd N: one weight row per thread in that product
    (256, 256, 64, "bf16", 70, 0.0, True),          # no sensitive entries at all: no sparse product
]


@pytest.mark.parametrize("N,K,G,fmt,M,rho,bias", PAIRED_LINEAR_CASES)
def test_linear_paired_matches_oracle(B, N, K, G, fmt, M, rho, bias):
    """yc, yd against centre and half-difference of the oracle's two forwards x+-(Dequantize(Q) + S +- eps Z)^T."""
    c = make_case(N, K, G, fmt, M, rho, seed=N + K + M + 1, bias=bias)
    plan, _, _ = upload(B, c)
    eps = np.float32(1e-3)
    g = wl.rng(5, wl.PURPOSE_ACTIVATION, N + M)
    xc = c["x"]
    xd = wl.bf16_round((2e-3 * g.standard_normal(xc.shape)).astype(np.float32))
    S = c["S"]
    z = so.gaussian(77, 3, c["idx"])
    ez = (eps.astype(np.float64) * z.astype(np.float64))
    Wp = so.effective_weight(c["deq"], c["idx"], S.astype(np.float64) + ez)
    Wm = so.effective_weight(c["deq"], c["idx"], S.astype(np.float64) - ez)
    b = 0.0 if c["bias"] is None else c["bias"].astype(np.float64)
    yp = (xc.astype(np.float64) + xd) @ Wp.T + b
    ym = (xc.astype(np.float64) - xd) @ Wm.T + b
    ref_c, ref_d = 0.5 * (yp + ym), 0.5 * (yp - ym)
    x, row0 = paired_rows(B, xc, xd)
    d = lambda a: torch.from_numpy(a).cuda()
    y = plan.fwd_paired(x, M, d(S), d(z), float(eps), torch.float32).cpu().numpy()
    assert max_rel(y[:M], ref_c) < 5e-3            # bf16 rounding of the effective weight
    assert max_rel(y[row0:], ref_d) < 5e-3
    yb = plan.fwd_paired(x, M, d(S), d(z), float(eps), torch.bfloat16).float().cpu().numpy()
    assert max_rel(yb[:M], ref_c) < 2e-2 and max_rel(yb[row0:], ref_d) < 2e-2
    # with xd = 0 the half-difference rows are eps * xc Zbar^T alone.  Sparse masks (below 0.2 %): an fp32 sum
    # of a few products, of eps * z kept with 23 - ceil(log2 K) mantissa bits (one word holds the column and
    # eps * z).  Denser masks: the product runs on the tensor cores with eps * z rounded to bf16.
    x0, _ = paired_rows(B, xc, np.zeros_like(xd))
    y0 = plan.fwd_paired(x0, M, d(S), d(z), float(eps), torch.float32).cpu().numpy()
    Zs = so.effective_weight(np.zeros_like(c["deq"]), c["idx"], ez)
    ref0 = xc.astype(np.float64) @ Zs.T
    dense_cross = len(c["idx"]) >= 0.002 * N * K
    if len(c["idx"]) == 0:
        assert not y0[row0:].any()                 # no entries: the half-difference rows of x W^T with xd = 0
    else:
        assert max_rel(y0[row0:], ref0) < (2.0 ** -8 if dense_cross else 2e-6 + 2.0 ** -(24 - int(np.ceil(np.log2(K)))))
    y1 = plan.fwd_paired(x0, M, d(S), d(z), float(eps), torch.float32).cpu().numpy()
    assert np.array_equal(y0[:M], y1[:M]) and np.array_equal(y0[row0:], y1[row0:])     # bit-repeatable
    assert B.device_status() == 0
    plan.close()


@pytest.mark.parametrize("B_,S,H,Hkv,hd", [(2, 64, 4, 4, 64), (1, 256, 4, 2, 128), (3, 100, 2, 1, 128), (2, 37, 4, 2, 64)])
@pytest.mark.parametrize("rel", [1e-2, 1e-5])
def test_attention_paired_matches_oracle(B, B_, S, H, Hkv, hd, rel):
    """Centre and half-difference of attention(q+, k+, v+) and attention(q-, k-, v-); the half-difference
    is checked relative to its own size, for a perturbation of 1e-2 and of 1e-5 of the activations."""
    g = wl.rng(4, wl.PURPOSE_ACTIVATION, S + hd)
    M = B_ * S
    mk = lambda heads, s: wl.bf16_round((s * g.standard_normal((M, heads * hd))).astype(np.float32))
    parts = {n: (mk(h, 1.0), mk(h, rel)) for n, h in (("q", H), ("k", Hkv), ("v", Hkv))}
    t64 = lambda a, heads: torch.from_numpy(a.astype(np.float64)).view(B_, S, heads, hd)
    outs = []
    for sgn in (1.0, -1.0):
        q, k, v = (t64(parts[n][0].astype(np.float64) + sgn * parts[n][1], h) for n, h in (("q", H), ("k", Hkv), ("v", Hkv)))
        outs.append(mo.causal_attention(q, k, v).reshape(M, H * hd).numpy())
    ref_c, ref_d = 0.5 * (outs[0] + outs[1]), 0.5 * (outs[0] - outs[1])
    bufs = {n: paired_rows(B, *parts[n]) for n in parts}
    row0 = bufs["q"][1]
    o = B.szo_attention_paired(bufs["q"][0], bufs["k"][0], bufs["v"][0], row0, B_, S, H, Hkv, hd).float().cpu().numpy()
    assert max_rel(o[:M], ref_c) <= 1.5e-2          # probabilities and outputs are rounded to bf16
    assert max_rel(o[row0:], ref_d) <= 1.5e-2


# ------------------------------------------------------------------------------------ whole steps
# The bound on the projected gradient of the bf16 tensor-core path, over 16 steps from the oracle's
# own trajectory: rms(g_gpu - g_oracle) <= G_RMS_TOL * rms(g_oracle), every sign equal where
# |g_oracle| > 5 % of its rms, correlation >= 0.999 (0.995 for the OPT-shaped decoder).  Observed: 0.3-0.8 % for the SiLU decoders
# (2 % for the 2-candidate loss of 64 short sequences), 3-6 % for the
# OPT-shaped one (a ReLU unit whose input sits near zero switches under the bf16 rounding of the centre,
# which moves the derivative itself; the two-forward modes show 15 % to 950 % on the same steps).
G_RMS_TOL = {"llama": 0.05, "opt": 0.10}
STEPS = 16


def run_steps(B, fx, mode, eps, loss_kind, steps=STEPS, lr=1e-4):
    t = fx.gpu_tensors(torch, None)
    S = torch.from_numpy(fx.S_init.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=B.SZO_BF16, linear_mode=mode, loss_kind=loss_kind,
                max_batch=fx.B, max_seq=fx.S)
    om = fx.oracle_model()
    kind = "lm" if loss_kind == 0 else "cls2"
    cand = np.array([5, 77], np.int32)
    d = lambda a: torch.from_numpy(a).cuda()
    rows = []
    for step in range(steps):
        toks = fx.batch(step)
        labels = wl.binary_labels(fx.B, 2, step)
        S.copy_(d(om.S))                               # every step starts from the oracle's S
        fp, fm, g = mo.zo_step(om, toks, 1234, step, eps, lr, kind, labels, cand)
        out = m.zo_step(d(toks), 1234, step, eps, lr, d(labels), d(cand)).cpu().numpy()
        rows.append((fp, fm, g, out[0], out[1], out[2]))
    assert B.device_status() == 0
    m.close()
    return np.array(rows)


def g_stats(r):
    g, gg = r[:, 2], r[:, 5]
    rms = np.sqrt(np.mean(g * g))
    big = np.abs(g) > 0.05 * rms
    return dict(rms_g=float(rms), rms_err=float(np.sqrt(np.mean((gg - g) ** 2)) / rms),
                median_rel=float(np.median(np.abs(gg - g) / np.abs(g))), max_rel=float(np.max(np.abs(gg - g) / np.abs(g))),
                sign=float(np.mean(np.sign(gg[big]) == np.sign(g[big]))), corr=float(np.corrcoef(g, gg)[0, 1]),
                loss_rel=float(max(np.max(np.abs(r[:, 3] - r[:, 0]) / r[:, 0]), np.max(np.abs(r[:, 4] - r[:, 1]) / r[:, 1]))))


@pytest.mark.parametrize("name,loss_kind", [("tiny", 0), ("tiny_gqa", 0), ("tiny_gqa", 1), ("tiny_opt", 0), ("tiny_lut", 0)])
@pytest.mark.parametrize("eps", [1e-3, 1e-4])
def test_paired_step_projected_gradient(B, name, loss_kind, eps):
    """16 ZO steps on the bf16 tensor-core path in the paired form: losses within 1e-3 of the oracle
    (2-candidate loss included) and the projected gradient within the bound above.  The same steps in
    the two-forward modes are run for the record (their error is printed, not bounded: it is the
    reason the paired form exists)."""
    fx = DecoderFixture(name, seed=3, mask="random", B=4, S=64)
    st = g_stats(run_steps(B, fx, B.MODE_PAIRED, eps, loss_kind))
    record = {"model": name, "loss": loss_kind, "eps": eps, "paired": st}
    for mode_name, mode in (("sparse_add", B.MODE_SPARSE_ADD), ("spmm", B.MODE_SPMM)):
        if mode == B.MODE_SPMM and fx.shape["group"] < 0:
            continue
        record[mode_name] = g_stats(run_steps(B, fx, mode, eps, loss_kind))
    print("G_ERROR " + json.dumps(record))
    out_dir = os.environ.get("SZO_G_ERROR_DIR")
    if out_dir:
        with open(os.path.join(out_dir, "g_error.jsonl"), "a") as f:
            f.write(json.dumps(record) + "\n")
    # the 2-candidate loss of four sequences does not average the bf16 rounding of the activations
    # (3e-3 there; test_two_candidate_loss_of_many_sequences holds 1e-3 at 64 sequences)
    assert st["loss_rel"] <= (1e-3 if loss_kind == 0 else 3e-3)
    arch = fx.shape["arch"]
    assert st["rms_err"] <= G_RMS_TOL[arch] and st["sign"] == 1.0 and st["corr"] >= (0.999 if arch == "llama" else 0.995), st


@pytest.mark.parametrize("mode", ["paired", "sparse_add"])
def test_two_candidate_loss_of_many_sequences(B, mode):
    """The loss kind of the 7B-shape workload (2-way cross-entropy at the last position) over 64
    sequences, bf16 tensor-core path: within 1e-3 of the oracle."""
    fx = DecoderFixture("tiny_gqa", seed=5, mask="random", B=64, S=32)
    r = run_steps(B, fx, B.MODE_PAIRED if mode == "paired" else B.MODE_SPARSE_ADD, 1e-3, 1, steps=3)
    assert np.max(np.abs(r[:, 3] - r[:, 0]) / r[:, 0]) <= 1e-3 and np.max(np.abs(r[:, 4] - r[:, 1]) / r[:, 1]) <= 1e-3
    if mode == "paired":
        assert np.max(np.abs(r[:, 5] - r[:, 2])) <= G_RMS_TOL["llama"] * np.sqrt(np.mean(r[:, 2] ** 2))


def test_paired_step_moves_S_like_the_oracle(B):
    """Ten steps of the tiny decoder on the paired path, each on the trajectory the GPU itself produced:
    S after the steps stays within the accumulated effect of the g error on the update."""
    fx = DecoderFixture("tiny", seed=0, mask="gradient", B=4, S=64)
    t = fx.gpu_tensors(torch, lambda W, G, fmt: B.szo_quantize(W, G, fmt))
    S = torch.from_numpy(fx.S_init.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=B.SZO_BF16, linear_mode=B.MODE_PAIRED, max_batch=fx.B, max_seq=fx.S)
    om = fx.oracle_model()
    eps, lr = 1e-3, 1e-3
    gs = []
    for step in range(10):
        toks = fx.batch(step)
        fp, fm, g = mo.zo_step(om, toks, 1234, step, eps, lr)
        out = m.zo_step(torch.from_numpy(toks).cuda(), 1234, step, eps, lr).cpu().numpy()
        assert abs(out[0] - fp) <= 1e-3 * abs(fp) and abs(out[1] - fm) <= 1e-3 * abs(fm)
        gs.append((g, out[2]))
    gs = np.array(gs)
    rms = np.sqrt(np.mean(gs[:, 0] ** 2))
    assert np.sqrt(np.mean((gs[:, 1] - gs[:, 0]) ** 2)) <= G_RMS_TOL["llama"] * rms
    moved = om.S - fx.S_init
    err = S.cpu().numpy() - om.S
    assert np.linalg.norm(err) <= 2 * G_RMS_TOL["llama"] * np.linalg.norm(moved)
    assert B.device_status() == 0
    m.close()


_STEP_SWITCH_SCRIPT = r"""
import sys, numpy as np, torch
from paper_2406_02913_b200 import binding as B, workloads as wl
shape = dict(wl.MODEL_SHAPES["llama2_7b"], n_layers=2)
tensors, S_all = wl.device_decoder_tensors(shape, seed=4)
Bn, S = 5, 256                                   # 1280 tokens: slabs of 16 tokens in the sparse product
m = B.Model(shape, wl.linear_names(shape), tensors, S_all, act_dtype=B.SZO_BF16, linear_mode=B.MODE_PAIRED,
            loss_kind=B.LOSS_CLS2, max_batch=Bn, max_seq=S)
toks = torch.from_numpy(wl.token_batch(shape["vocab"], Bn, S, 4, wl.PURPOSE_TRAIN_BATCH, 0)).cuda()
labs = torch.from_numpy(wl.binary_labels(Bn, 4, 0)).cuda()
cand = torch.tensor([9906, 13], dtype=torch.int32, device="cuda")
rows = [m.zo_step(toks, 77, step, 1e-3, 1e-4, labs, cand).double().cpu().numpy().copy() for step in range(3)]
assert B.device_status() == 0
np.savez(sys.argv[1], out=np.array(rows), S=S_all.cpu().numpy())
"""


def test_switches_of_the_training_step_leave_the_bits_alone(tmp_path):
    """Three paired steps at the Llama-2-7B width (two layers) with the step's kernels launched as a chain
    (the default), with ordinary launches, and with the other slab height of the sparse product: a chained
    launch changes when a kernel starts, not what it computes, and a thread of the sparse product walks the same
    entries in the same order whatever the number of tokens per slab, so losses, g and the updated sparse
    values must be the same bits.  The switches are read once per process: one child process per setting."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = {}
    for name, extra in (("default", {}), ("no_chain", {"SZO_STEP_CHAIN": "0"}), ("slab8", {"SZO_CROSS_TM": "8"})):
        out = str(tmp_path / (name + ".npz"))
        r = subprocess.run([sys.executable, "-c", _STEP_SWITCH_SCRIPT, out], cwd=root, env=dict(os.environ, **extra),
                           capture_output=True, text=True, timeout=900)
        assert r.returncode == 0, name + ": " + r.stdout[-2000:] + r.stderr[-2000:]
        res[name] = np.load(out)
    assert np.isfinite(res["default"]["out"]).all()
    for other in ("no_chain", "slab8"):
        assert np.array_equal(res["default"]["out"], res[other]["out"]), other
        assert np.array_equal(res["default"]["S"], res[other]["S"]), other
