"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input generators only: random weights, token ids, heavy-tailed gradient
scores, index samples and activations.  It contains none of the method's arithmetic (no
quantizer, no mask selection, no Philox/Gaussian perturbation, no forward pass), so the same
arrays can be handed to the CUDA library and to an independent checker.

Every generator draws from numpy.random.default_rng([seed, purpose, i]) so that streams with
different purposes never overlap.
"""
from __future__ import annotations

import numpy as np

PURPOSE_WEIGHTS = 0
PURPOSE_MASK_BATCH = 1
PURPOSE_TRAIN_BATCH = 2
PURPOSE_SCORES = 3
PURPOSE_INDICES = 4
PURPOSE_ACTIVATION = 5
PURPOSE_LABELS = 6
PURPOSE_CODES = 7


def rng(seed: int, purpose: int, i: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(purpose), int(i)])


def bf16_round(a) -> np.ndarray:
    """fp32 array rounded to the nearest bf16-representable value (ties to even), still fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    b = a.view(np.uint32).astype(np.uint64)
    b = ((b + 0x7FFF + ((b >> 16) & 1)) >> 16) << 16
    return b.astype(np.uint32).view(np.float32).reshape(a.shape)


# name -> architecture dictionary (the decoder shapes of the paper's Section 4 models)
MODEL_SHAPES = {
    "tiny": dict(arch="llama", n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, d_ff=1024,
                 vocab=1024, max_pos=0, group=64, sz_fmt="f16", rho=1e-3),
    "tiny_gqa": dict(arch="llama", n_layers=2, d_model=256, n_heads=4, n_kv_heads=2, d_ff=512,
                     vocab=512, max_pos=0, group=0, sz_fmt="bf16", rho=1e-2),
    "tiny_opt": dict(arch="opt", n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, d_ff=1024,
                     vocab=1024, max_pos=128, group=128, sz_fmt="bf16", rho=1e-3),
    "tiny_lut": dict(arch="llama", n_layers=2, d_model=256, n_heads=4, n_kv_heads=4, d_ff=1024,
                     vocab=1024, max_pos=0, group=-1, sz_fmt="f16", rho=1e-3),
    # test shapes wide enough for the kernels of one or two tokens (K >= 896), with grouped-query attention, so
    # that the q/k/v launch holds matrices of different heights
    "small_gqa": dict(arch="llama", n_layers=2, d_model=1024, n_heads=16, n_kv_heads=4, d_ff=2816,
                      vocab=1024, max_pos=0, group=128, sz_fmt="bf16", rho=2e-3),
    "small_gqa_lut": dict(arch="llama", n_layers=2, d_model=1024, n_heads=16, n_kv_heads=4, d_ff=2816,
                          vocab=1024, max_pos=0, group=-1, sz_fmt="f16", rho=2e-3),
    "llama2_7b_lut": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32,
                          d_ff=11008, vocab=32000, max_pos=0, group=-1, sz_fmt="f16", rho=1e-3),
    "llama2_7b": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=32,
                      d_ff=11008, vocab=32000, max_pos=0, group=128, sz_fmt="bf16", rho=1e-3),
    "mistral_7b": dict(arch="llama", n_layers=32, d_model=4096, n_heads=32, n_kv_heads=8,
                       d_ff=14336, vocab=32000, max_pos=0, group=0, sz_fmt="bf16", rho=1e-2),
    "opt_13b": dict(arch="opt", n_layers=40, d_model=5120, n_heads=40, n_kv_heads=40,
                    d_ff=20480, vocab=50272, max_pos=2048, group=128, sz_fmt="bf16", rho=1e-3),
}

LLAMA_LINEARS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
OPT_LINEARS = ("wq", "wk", "wv", "wo", "fc1", "fc2")


def linear_names(shape: dict):
    return LLAMA_LINEARS if shape["arch"] == "llama" else OPT_LINEARS


def linear_shape(shape: dict, name: str):
    d = shape["d_model"]
    kv = shape["n_kv_heads"] * (d // shape["n_heads"])
    ff = shape["d_ff"]
    return {"wq": (d, d), "wk": (kv, d), "wv": (kv, d), "wo": (d, d), "w_gate": (ff, d),
            "w_up": (ff, d), "w_down": (d, ff), "fc1": (ff, d), "fc2": (d, ff)}[name]


def init_params(shape: dict, seed: int = 0, std: float = 0.02):
    """Random-init weights N(0, std).  Returns (params, lin_W): params holds embeddings, LM
    head, position table (bf16-representable fp32), norm gains (1) and biases; lin_W is
    [layer][name] -> fp32 [N, K]."""
    g = rng(seed, PURPOSE_WEIGHTS)
    d, V = shape["d_model"], shape["vocab"]
    opt = shape["arch"] == "opt"
    params = {"embed": bf16_round(g.normal(0, std, (V, d))),
              "lm_head": bf16_round(g.normal(0, std, (V, d))),
              "final_norm": np.ones(d, np.float32)}
    if opt:
        params["pos"] = bf16_round(g.normal(0, std, (shape["max_pos"], d)))
        params["final_norm_b"] = np.zeros(d, np.float32)
    lin_W = []
    for l in range(shape["n_layers"]):
        params[f"l{l}.attn_norm"] = np.ones(d, np.float32)
        params[f"l{l}.mlp_norm"] = np.ones(d, np.float32)
        if opt:
            params[f"l{l}.attn_norm_b"] = np.zeros(d, np.float32)
            params[f"l{l}.mlp_norm_b"] = np.zeros(d, np.float32)
        layer = {}
        for nm in linear_names(shape):
            N, K = linear_shape(shape, nm)
            layer[nm] = g.normal(0, std, (N, K)).astype(np.float32)
            if opt:
                params[f"l{l}.{nm}_b"] = g.normal(0, std, N).astype(np.float32)
        lin_W.append(layer)
    return params, lin_W


def token_batch(vocab: int, B: int, S: int, seed: int, purpose: int, i: int) -> np.ndarray:
    """Uniform token ids, int32 [B, S]."""
    return rng(seed, purpose, i).integers(0, vocab, (B, S), dtype=np.int32)


def binary_labels(B: int, seed: int, i: int) -> np.ndarray:
    return rng(seed, PURPOSE_LABELS, i).integers(0, 2, (B,), dtype=np.int32)


def student_t_gradient(n: int, nu: float = 3.0, seed: int = 0, i: int = 0) -> np.ndarray:
    """Heavy-tailed stand-in for a first-order gradient: g = N(0,1) / sqrt(chi2_nu / nu), fp32.
    (A few coordinates carry most of the squared norm, as the paper observes for LLM linears.)"""
    g = rng(seed, PURPOSE_SCORES, i)
    t = g.standard_normal(n) / np.sqrt(g.chisquare(nu, n) / nu)
    return t.astype(np.float32)


def sorted_random_indices(n: int, k: int, seed: int = 0, i: int = 0) -> np.ndarray:
    """k distinct indices in [0, n), ascending, int64 (without materialising a permutation)."""
    g = rng(seed, PURPOSE_INDICES, i)
    if k > n:
        raise ValueError("k > n")
    if k * 4 > n:
        return np.sort(g.choice(n, size=k, replace=False)).astype(np.int64)
    got = np.unique(g.integers(0, n, int(k * 1.1) + 16, dtype=np.int64))
    while got.size < k:
        got = np.unique(np.concatenate([got, g.integers(0, n, k, dtype=np.int64)]))
    if got.size > k:
        got = np.sort(g.choice(got, size=k, replace=False))
    return got.astype(np.int64)


def activation(M: int, K: int, seed: int = 0, i: int = 0) -> np.ndarray:
    """x ~ N(0,1), bf16-representable fp32 [M, K]."""
    return bf16_round(rng(seed, PURPOSE_ACTIVATION, i).standard_normal((M, K)).astype(np.float32))


def gaussian_matrix(N: int, K: int, std: float, seed: int = 0, i: int = 0) -> np.ndarray:
    return rng(seed, PURPOSE_WEIGHTS, 1000 + i).normal(0, std, (N, K)).astype(np.float32)


def random_codes(N: int, K: int, seed: int = 0, i: int = 0) -> np.ndarray:
    """Uniform random packed nibbles uint8 [N, K/2] (timing stand-in for a quantized tensor)."""
    return rng(seed, PURPOSE_CODES, i).integers(0, 256, (N, K // 2), dtype=np.uint8)


def random_lut(N: int, seed: int = 0, i: int = 0, std: float = 0.02) -> np.ndarray:
    """Per-row tables of the non-uniform 4-bit format, fp32 [N,16]: 16 ascending draws from
    N(0, std) per row (the shape a sensitivity-weighted k-means over a Gaussian row produces:
    dense near zero, sparse in the tails).  Input generator only; the caller rounds to fp16/bf16."""
    return np.sort(rng(seed, PURPOSE_WEIGHTS, 900 + i).normal(0.0, std, (N, 16)), axis=1).astype(np.float32)


# ------------------------------------------------------------------------------ large workloads
# Full-size decoders (billions of parameters) are generated directly in device memory with a seeded
# torch generator: quantizing 6.5 G fp32 weights on the host only to time a step would take
# minutes.  These are input generators too: random codes, scales, zeros, indices and values.
def device_decoder_tensors(shape: dict, seed: int = 0, device: str = "cuda"):
    """Random-init quantized decoder in device memory, named as binding.Model expects.
    Codes are uniform nibbles; scale ~ U(0.004, 0.006) and zero = -7.5 scale so that the
    dequantised weights are centred with a spread close to N(0, 0.02); the sensitive set of each
    tensor is a sorted random sample of floor(rho n) indices with values N(0, 0.02).
    Returns (tensors, S_all)."""
    import torch

    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    d, V, G = shape["d_model"], shape["vocab"], shape["group"]
    sz_dt = torch.bfloat16 if shape["sz_fmt"] == "bf16" else torch.float16
    opt = shape["arch"] == "opt"
    randn = lambda *s: torch.randn(*s, generator=g, device=device, dtype=torch.float32)
    t = {"embed": (randn(V, d) * 0.02).to(torch.bfloat16), "lm_head": (randn(V, d) * 0.02).to(torch.bfloat16),
         "final_norm": torch.ones(d, device=device)}
    if opt:
        t["pos"] = (randn(shape["max_pos"], d) * 0.02).to(torch.bfloat16)
        t["final_norm_b"] = torch.zeros(d, device=device)
    S_parts = []
    for l in range(shape["n_layers"]):
        for nm in ("attn_norm", "mlp_norm"):
            t[f"l{l}.{nm}"] = torch.ones(d, device=device)
            if opt:
                t[f"l{l}.{nm}_b"] = torch.zeros(d, device=device)
        for nm in linear_names(shape):
            N, K = linear_shape(shape, nm)
            p = f"l{l}.{nm}."
            if G > 0:
                t[p + "codes"] = torch.randint(0, 256, (N, K // 2), generator=g, device=device, dtype=torch.uint8)
                sc = (0.004 + 0.002 * torch.rand(N, K // G, generator=g, device=device)).to(sz_dt)
                t[p + "scales"] = sc
                t[p + "zeros"] = (-7.5 * sc.float()).to(sz_dt)
            elif G < 0:     # non-uniform 4-bit format: uniform codes into 16 ascending N(0, 0.02) draws per row
                t[p + "codes"] = torch.randint(0, 256, (N, K // 2), generator=g, device=device, dtype=torch.uint8)
                t[p + "lut"] = torch.sort(randn(N, 16) * 0.02, dim=1).values.to(sz_dt).contiguous()
            else:
                t[p + "codes"] = (randn(N, K) * 0.02).to(torch.bfloat16)
            k = int(shape["rho"] * N * K)
            draw = torch.randint(0, N * K, (int(k * 1.05) + 64,), generator=g, device=device, dtype=torch.int64)
            u = torch.unique(draw)
            while u.numel() < k:
                more = torch.randint(0, N * K, (k,), generator=g, device=device, dtype=torch.int64)
                u = torch.unique(torch.cat([u, more]))
            keep = torch.randperm(u.numel(), generator=g, device=device)[:k]
            t[p + "idx"] = torch.sort(u[keep]).values.contiguous()
            S_parts.append(randn(k) * 0.02)
            if opt:
                t[p + "bias"] = randn(N) * 0.02
    S_all = torch.cat(S_parts).contiguous() if S_parts else torch.zeros(0, device=device)
    return t, S_all
