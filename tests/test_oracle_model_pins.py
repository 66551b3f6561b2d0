"""Pins for oracle/model_oracle.py: each block against a PyTorch library routine or an
invariant, the gradients against central differences, the whole step against identities."""
import math

import numpy as np
import torch
import torch.nn.functional as F

from oracle import model_oracle as mo
from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl

torch.manual_seed(0)


def _cfg(name):
    s = wl.MODEL_SHAPES[name]
    return mo.DecoderConfig(arch=s["arch"], n_layers=s["n_layers"], d_model=s["d_model"],
                            n_heads=s["n_heads"], n_kv_heads=s["n_kv_heads"], d_ff=s["d_ff"],
                            vocab=s["vocab"], max_pos=s["max_pos"])


def _small(arch="llama", kv=2):
    cfg = mo.DecoderConfig(arch=arch, n_layers=2, d_model=32, n_heads=4, n_kv_heads=kv if arch == "llama" else 4,
                           d_ff=64, vocab=50, max_pos=16)
    shape = dict(arch=arch, n_layers=2, d_model=32, n_heads=4, n_kv_heads=cfg.n_kv_heads, d_ff=64,
                 vocab=50, max_pos=16)
    params, lin_W = wl.init_params(shape, seed=3, std=0.2)
    for k in list(params):                       # non-trivial gains and shifts
        if k.endswith("norm"):
            params[k] = (1 + 0.1 * np.random.default_rng(1).standard_normal(32)).astype(np.float32)
        if k.endswith("norm_b"):
            params[k] = (0.1 * np.random.default_rng(2).standard_normal(32)).astype(np.float32)
    tokens = wl.token_batch(50, 3, 8, 0, wl.PURPOSE_TRAIN_BATCH, 0)
    return cfg, params, lin_W, tokens


def test_norms_match_library():
    x = torch.randn(5, 7, 32, dtype=torch.float64)
    g = torch.randn(32, dtype=torch.float64)
    b = torch.randn(32, dtype=torch.float64)
    assert torch.allclose(mo.rms_norm(x, g, 1e-5), F.rms_norm(x, (32,), g, 1e-5), atol=1e-13)
    assert torch.allclose(mo.layer_norm(x, g, b, 1e-5), F.layer_norm(x, (32,), g, b, 1e-5), atol=1e-13)


def test_attention_matches_library_and_is_causal():
    B, S, H, Hkv, hd = 2, 9, 4, 2, 8
    q = torch.randn(B, S, H, hd, dtype=torch.float64)
    k = torch.randn(B, S, Hkv, hd, dtype=torch.float64)
    v = torch.randn(B, S, Hkv, hd, dtype=torch.float64)
    out = mo.causal_attention(q, k, v)
    kr = k.repeat_interleave(H // Hkv, dim=2)
    vr = v.repeat_interleave(H // Hkv, dim=2)
    ref = F.scaled_dot_product_attention(q.transpose(1, 2), kr.transpose(1, 2), vr.transpose(1, 2),
                                         is_causal=True).transpose(1, 2)
    assert torch.allclose(out, ref, atol=1e-13)
    # changing a later token leaves earlier outputs alone
    k2, v2 = k.clone(), v.clone()
    k2[:, 6] += 1.0
    v2[:, 6] -= 1.0
    out2 = mo.causal_attention(q, k2, v2)
    assert torch.equal(out[:, :6], out2[:, :6]) and not torch.allclose(out[:, 6:], out2[:, 6:])
    # first position attends to itself only
    assert torch.allclose(out[:, 0], vr[:, 0], atol=1e-14)


def test_rope_properties():
    B, S, H, hd = 1, 12, 2, 16
    x = torch.randn(B, S, H, hd, dtype=torch.float64)
    y = mo.rope(x, 10000.0)
    assert torch.equal(y[:, 0], x[:, 0])                                   # position 0: identity
    assert torch.allclose(y.norm(dim=-1), x.norm(dim=-1), atol=1e-13)       # a rotation
    # pair (i, i+hd/2) at position p is rotated by p * base^(-2i/hd)
    p, i = 5, 3
    th = p * 10000.0 ** (-2 * i / hd)
    a, b = x[0, p, 1, i], x[0, p, 1, i + hd // 2]
    assert math.isclose(y[0, p, 1, i], a * math.cos(th) - b * math.sin(th), abs_tol=1e-13)
    assert math.isclose(y[0, p, 1, i + hd // 2], b * math.cos(th) + a * math.sin(th), abs_tol=1e-13)
    # inner products depend on the relative position only
    qv = torch.randn(hd, dtype=torch.float64)
    kv = torch.randn(hd, dtype=torch.float64)
    qs = mo.rope(qv.expand(1, S, 1, hd).clone(), 10000.0)
    ks = mo.rope(kv.expand(1, S, 1, hd).clone(), 10000.0)
    d1 = (qs[0, 7, 0] * ks[0, 4, 0]).sum()
    d2 = (qs[0, 10, 0] * ks[0, 7, 0]).sum()
    assert math.isclose(d1, d2, abs_tol=1e-12)


def test_losses_match_library():
    for arch in ("llama", "opt"):
        cfg, params, lin_W, tokens = _small(arch)
        hs = mo.hidden_states(cfg, params, lin_W, tokens)
        E = torch.as_tensor(params["lm_head"], dtype=torch.float64)
        tok = torch.as_tensor(tokens, dtype=torch.long)
        logits = hs @ E.T
        ref = F.cross_entropy(logits[:, :-1].reshape(-1, cfg.vocab), tok[:, 1:].reshape(-1))
        got = mo.loss_fn(cfg, params, lin_W, tokens, "lm")
        assert math.isclose(float(got), float(ref), rel_tol=1e-13)
        cand = np.array([7, 31])
        labels = np.array([0, 1, 1])
        ref2 = F.cross_entropy(logits[:, -1][:, cand], torch.as_tensor(labels))
        got2 = mo.loss_fn(cfg, params, lin_W, tokens, "cls2", labels=labels, cand=cand)
        assert math.isclose(float(got2), float(ref2), rel_tol=1e-13)


def test_zero_lm_head_gives_log_vocab():
    cfg, params, lin_W, tokens = _small("llama")
    params = dict(params)
    params["lm_head"] = np.zeros_like(params["lm_head"])
    assert math.isclose(float(mo.loss_fn(cfg, params, lin_W, tokens, "lm")), math.log(cfg.vocab), rel_tol=1e-14)
    assert math.isclose(float(mo.loss_fn(cfg, params, lin_W, tokens, "cls2", labels=[0, 1, 0], cand=[1, 2])),
                        math.log(2), rel_tol=1e-14)


def test_decoder_blocks_against_an_independent_einsum_statement():
    """One llama layer restated with numpy einsum (no torch) and compared on the hidden state."""
    cfg, params, lin_W, tokens = _small("llama", kv=2)
    cfg1 = mo.DecoderConfig(**{**cfg.__dict__, "n_layers": 1})
    got = mo.hidden_states(cfg1, params, lin_W[:1], tokens).numpy()
    W = {k: v.astype(np.float64) for k, v in lin_W[0].items()}
    B, S = tokens.shape
    H, Hkv, hd, d = 4, 2, 8, 32
    h = params["embed"].astype(np.float64)[tokens]

    def rms(x, gname):
        return x / np.sqrt(np.mean(x * x, -1, keepdims=True) + 1e-5) * params[gname].astype(np.float64)

    a = rms(h, "l0.attn_norm")
    q = np.einsum("bsk,nk->bsn", a, W["wq"]).reshape(B, S, H, hd)
    k = np.einsum("bsk,nk->bsn", a, W["wk"]).reshape(B, S, Hkv, hd)
    v = np.einsum("bsk,nk->bsn", a, W["wv"]).reshape(B, S, Hkv, hd)

    def rot(x):
        out = np.empty_like(x)
        for p in range(S):
            for i in range(hd // 2):
                th = p * 10000.0 ** (-2.0 * i / hd)
                out[:, p, :, i] = x[:, p, :, i] * np.cos(th) - x[:, p, :, i + hd // 2] * np.sin(th)
                out[:, p, :, i + hd // 2] = x[:, p, :, i + hd // 2] * np.cos(th) + x[:, p, :, i] * np.sin(th)
        return out

    q, k = rot(q), rot(k)
    o = np.zeros((B, S, H, hd))
    for b in range(B):
        for hh in range(H):
            for s in range(S):
                sc = np.array([q[b, s, hh] @ k[b, t, hh // 2] / np.sqrt(hd) for t in range(s + 1)])
                p = np.exp(sc - sc.max())
                p /= p.sum()
                o[b, s, hh] = sum(p[t] * v[b, t, hh // 2] for t in range(s + 1))
    h = h + np.einsum("bsk,nk->bsn", o.reshape(B, S, d), W["wo"])
    m = rms(h, "l0.mlp_norm")
    gate = np.einsum("bsk,nk->bsn", m, W["w_gate"])
    up = np.einsum("bsk,nk->bsn", m, W["w_up"])
    h = h + np.einsum("bsk,nk->bsn", gate / (1 + np.exp(-gate)) * up, W["w_down"])
    ref = rms(h, "final_norm")
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


def _opt_layer_numpy(params, W, tokens, H, eps=1e-5, act=lambda t: np.maximum(t, 0.0)):
    """One OPT decoder layer + final LayerNorm written with numpy loops and einsum (no torch, nothing
    from the oracle): token + learned-position embedding from position 0, pre-LayerNorm with gain and
    shift, a bias on each of q/k/v/o/fc1/fc2, causal softmax attention without rotary positions,
    fc2(relu(fc1 x + b1)) + b2, residuals around both blocks."""
    f64 = lambda a: np.asarray(a, dtype=np.float64)
    B, S = tokens.shape
    d = params["embed"].shape[1]
    hd = d // H
    h = np.empty((B, S, d))
    for b in range(B):
        for s in range(S):
            h[b, s] = f64(params["embed"])[tokens[b, s]] + f64(params["pos"])[s]

    def ln(x, name):
        mu = x.sum(-1, keepdims=True) / d
        var = ((x - mu) ** 2).sum(-1, keepdims=True) / d
        return (x - mu) / np.sqrt(var + eps) * f64(params[name]) + f64(params[name + "_b"])

    def lin(x, nm):
        return np.einsum("bsk,nk->bsn", x, f64(W[nm])) + f64(params[f"l0.{nm}_b"])

    a = ln(h, "l0.attn_norm")
    q, k, v = (lin(a, nm).reshape(B, S, H, hd) for nm in ("wq", "wk", "wv"))
    o = np.zeros((B, S, H, hd))
    for b in range(B):
        for hh in range(H):
            for s in range(S):
                sc = np.array([q[b, s, hh] @ k[b, t, hh] / np.sqrt(hd) for t in range(s + 1)])
                p = np.exp(sc - sc.max())
                p /= p.sum()
                o[b, s, hh] = sum(p[t] * v[b, t, hh] for t in range(s + 1))
    h = h + lin(o.reshape(B, S, d), "wo")
    m = ln(h, "l0.mlp_norm")
    h = h + lin(act(lin(m, "fc1")), "fc2")
    return ln(h, "final_norm")


def _opt_case():
    cfg, params, lin_W, tokens = _small("opt")
    params = dict(params)
    g = np.random.default_rng(5)
    for k in list(params):                        # a different gain and shift for every norm
        if k.endswith("norm"):
            params[k] = (1 + 0.2 * g.standard_normal(32)).astype(np.float32)
        if k.endswith("norm_b"):
            params[k] = (0.3 * g.standard_normal(32)).astype(np.float32)
    cfg1 = mo.DecoderConfig(**{**cfg.__dict__, "n_layers": 1})
    return cfg1, params, lin_W[:1], tokens


def test_opt_blocks_against_an_independent_numpy_statement():
    """The OPT branch of hidden_states (learned positions, LayerNorm with shift, biases, ReLU MLP)
    against a restatement that shares nothing with it."""
    cfg1, params, lin_W, tokens = _opt_case()
    got = mo.hidden_states(cfg1, params, lin_W, tokens).numpy()
    ref = _opt_layer_numpy(params, lin_W[0], tokens, H=4)
    assert np.allclose(got, ref, rtol=0, atol=1e-12)


def test_opt_statement_notices_a_dropped_bias_a_position_shift_and_post_norm():
    """The pin above has teeth: handing the oracle inputs that stand for a plausible mistake (fc2's
    bias missing, positions starting at 1, a zeroed norm shift, no ReLU effect) moves its output far
    beyond the comparison's tolerance, so such a mistake inside the oracle would be seen."""
    cfg1, params, lin_W, tokens = _opt_case()
    ref = _opt_layer_numpy(params, lin_W[0], tokens, H=4)

    def oracle_with(**changes):
        p = dict(params)
        p.update(changes)
        return mo.hidden_states(cfg1, p, lin_W, tokens).numpy()

    for nm in ("wq", "wk", "wv", "wo", "fc1", "fc2"):
        key = f"l0.{nm}_b"
        if nm == "wk":
            continue           # a bias on k shifts every score of a row equally: softmax removes it
        assert np.abs(oracle_with(**{key: np.zeros_like(params[key])}) - ref).max() > 1e-6, nm
    assert np.abs(oracle_with(pos=np.roll(params["pos"], -1, axis=0)) - ref).max() > 1e-6
    for key in ("l0.attn_norm_b", "l0.mlp_norm_b", "final_norm_b"):
        assert np.abs(oracle_with(**{key: np.zeros_like(params[key])}) - ref).max() > 1e-6, key
    # the ReLU matters on these inputs: a statement without the clamp is far from the oracle
    got = mo.hidden_states(cfg1, params, lin_W, tokens).numpy()
    assert np.abs(_opt_layer_numpy(params, lin_W[0], tokens, H=4, act=lambda t: t) - got).max() > 1e-6


def test_incremental_decode_equals_the_full_forward():
    """decode_step with a KV cache (prefill of 3 tokens, then a chunk of 2, then one token at a time)
    gives, at every stop, the logits that the full forward gives at that position: both architectures,
    grouped-query attention included."""
    for arch in ("llama", "opt"):
        cfg, params, lin_W, tokens = _small(arch)
        hs = mo.hidden_states(cfg, params, lin_W, tokens)
        full = (hs @ torch.as_tensor(params["lm_head"], dtype=torch.float64).T).numpy()      # [B, S, V]
        cache = mo.KVCache(cfg.n_layers)
        at = 0
        for T in (3, 2, 1, 1, 1):
            logits = mo.decode_step(cfg, params, lin_W, tokens[:, at:at + T], cache).numpy()
            at += T
            assert cache.n == at
            assert np.allclose(logits, full[:, at - 1, :], rtol=0, atol=1e-11), (arch, at)


def test_gqa_reduces_to_mha_when_kv_heads_are_duplicated():
    cfg, params, lin_W, tokens = _small("llama", kv=2)
    full = mo.DecoderConfig(**{**cfg.__dict__, "n_kv_heads": 4})
    hd = 8
    lin_full = []
    for W in lin_W:
        Wf = dict(W)
        for nm in ("wk", "wv"):
            blocks = W[nm].reshape(2, hd, -1)
            Wf[nm] = np.repeat(blocks, 2, axis=0).reshape(4 * hd, -1)
        lin_full.append(Wf)
    a = mo.loss_fn(cfg, params, lin_W, tokens)
    b = mo.loss_fn(full, params, lin_full, tokens)
    assert math.isclose(float(a), float(b), rel_tol=1e-13)


def test_gradients_match_central_differences():
    for arch in ("llama", "opt"):
        cfg, params, lin_W, tokens = _small(arch)
        grads, loss = mo.linear_gradients(cfg, params, lin_W, tokens)
        g = np.random.default_rng(0)
        names = cfg.linear_names()
        for _ in range(40):
            l = int(g.integers(cfg.n_layers))
            nm = names[int(g.integers(len(names)))]
            N, K = lin_W[l][nm].shape
            i, j = int(g.integers(N)), int(g.integers(K))
            h = 1e-5
            Wp = [{k: v.astype(np.float64).copy() for k, v in L.items()} for L in lin_W]
            Wm = [{k: v.astype(np.float64).copy() for k, v in L.items()} for L in lin_W]
            Wp[l][nm][i, j] += h
            Wm[l][nm][i, j] -= h
            fd = (float(mo.loss_fn(cfg, params, Wp, tokens)) - float(mo.loss_fn(cfg, params, Wm, tokens))) / (2 * h)
            assert math.isclose(grads[l][nm][i, j], fd, rel_tol=1e-5, abs_tol=1e-9)


def test_score_accumulation_is_sum_of_squares_in_fp32():
    g1 = [{"a": np.array([1.5, -2.0])}]
    g2 = [{"a": np.array([0.5, 1.0])}]
    sc = mo.accumulate_scores([g1, g2])
    assert sc[0]["a"].dtype == np.float32 and list(sc[0]["a"]) == [2.5, 5.0]


def _build_sparse_model(name="tiny", seed=0, n_layers=None):
    shape = dict(wl.MODEL_SHAPES[name])
    if n_layers:
        shape["n_layers"] = n_layers
    cfg = mo.DecoderConfig(arch=shape["arch"], n_layers=shape["n_layers"], d_model=shape["d_model"],
                           n_heads=shape["n_heads"], n_kv_heads=shape["n_kv_heads"], d_ff=shape["d_ff"],
                           vocab=shape["vocab"], max_pos=shape["max_pos"])
    params, lin_W = wl.init_params(shape, seed)
    W_deq, idx_local, offsets, gidx, S = [], [], [0], [], []
    base = 0
    for l in range(cfg.n_layers):
        dq, il = {}, {}
        for nm in cfg.linear_names():
            W = lin_W[l][nm]
            k = int(shape["rho"] * W.size)
            idx = wl.sorted_random_indices(W.size, k, seed, 100 * l + len(dq))
            s, Wd = so.decompose(W, idx)
            codes, sb, zb = so.quantize_int4(Wd, shape["group"], shape["sz_fmt"])
            dq[nm] = so.dequantize(codes, sb, zb, shape["group"], shape["sz_fmt"])
            il[nm] = idx
            gidx.append(idx + base)
            S.append(s)
            offsets.append(offsets[-1] + k)
            base += W.size
        W_deq.append(dq)
        idx_local.append(il)
    return mo.SparseQuantModel(cfg, params, W_deq, idx_local, offsets,
                               np.concatenate(gidx), np.concatenate(S)), shape


def test_zo_step_on_the_decoder_keeps_frozen_parts_and_follows_the_update_rule():
    model, shape = _build_sparse_model("tiny", n_layers=1)
    frozen = [{k: v.copy() for k, v in L.items()} for L in model.W_deq]
    tokens = wl.token_batch(shape["vocab"], 2, 16, 0, wl.PURPOSE_TRAIN_BATCH, 0)
    S0 = model.S.copy()
    fp, fm, g = mo.zo_step(model, tokens, seed=1234, step=0, eps=1e-3, lr=1e-2)
    assert all(np.array_equal(a[k], b[k]) for a, b in zip(frozen, model.W_deq) for k in a)
    z = so.gaussian(1234, 0, model.gidx).astype(np.float64)
    assert np.isclose(g, (fp - fm) / (2 * float(np.float32(1e-3))), rtol=1e-15)
    assert np.allclose(model.S, S0 - float(np.float32(1e-2)) * g * z, rtol=0, atol=2e-8)
    # the projected gradient approximates zbar . grad f (first-order Taylor, Section 3.1)
    lin_eff = model.lin_W(S0)
    grads, _ = mo.linear_gradients(model.cfg, model.params, lin_eff, tokens)
    gs = np.concatenate([grads[0][nm].ravel()[model.idx_local[0][nm]] for nm in model.cfg.linear_names()])
    assert np.isclose(g, z @ gs, rtol=1e-3, atol=1e-7)


def test_llama2_7b_linear_parameter_count_and_4bit_footprint():
    shape = wl.MODEL_SHAPES["llama2_7b"]
    d_lin = sum(np.prod(wl.linear_shape(shape, nm)) for nm in wl.linear_names(shape)) * shape["n_layers"]
    assert d_lin == 6_476_005_376
    total = d_lin + 2 * shape["vocab"] * shape["d_model"] + (2 * shape["n_layers"] + 1) * shape["d_model"]
    # Section 3.5: a Llama2-7B model shrinks from 13.5 to 3.4 (GB) when the weights go to 4 bits
    assert abs(total * 2 / 1e9 - 13.5) < 0.05
    assert abs(total * 0.5 / 1e9 - 3.4) < 0.05
