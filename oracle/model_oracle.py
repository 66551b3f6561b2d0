"""CPU oracle: the loss f(w; (x, y)) of a decoder-only language model and the ZO-SGD step.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  Plain PyTorch CPU ops in fp64; shares no
code with the CUDA library.

The paper treats the loss as a black box evaluated twice per step (Definition 1, SPSA) on
decoder-only transformers (Section 4: Llama2-7B, Mistral-7B, OPT-6.7B).  The architecture
details below are the standard ones of those model families:

  llama / mistral   pre-norm; RMSNorm x / sqrt(mean x^2 + eps) * gamma; rotary position
                    embedding (base 10000, pairs (i, i + hd/2)); causal softmax attention with
                    scale 1/sqrt(hd), grouped-query attention by sharing each KV head among
                    H / H_kv query heads; MLP down(silu(gate x) * up x); untied LM head.
  opt               pre-LayerNorm with bias; learned positions added to the token embedding;
                    biases on every linear; MLP fc2(relu(fc1 x + b1)) + b2.

Losses: "lm"   mean next-token cross-entropy over the B*(S-1) predicted positions;
        "cls2" per sequence, cross-entropy of the 2-way softmax over the logits of two
               candidate label ids at the last position, mean over B.

zo_step follows Definition 1 (SPSA), Definition 2 (ZO-SGD), Definition 4 (sensitive sparse
ZO-SGD) and the Section 3.4 update rule on w_sparse, with z regenerated from the seed for each
of the four passes (Section 2.1, the seed trick).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch

from . import szo_oracle as so

LLAMA_LINEARS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")
OPT_LINEARS = ("wq", "wk", "wv", "wo", "fc1", "fc2")


@dataclass
class DecoderConfig:
    arch: str            # "llama" (also Mistral: n_kv_heads < n_heads) or "opt"
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    d_ff: int
    vocab: int
    max_pos: int = 0     # opt only
    norm_eps: float = 1e-5
    rope_base: float = 10000.0

    @property
    def head_dim(self) -> int:
        return self.d_model // self.n_heads

    def linear_names(self):
        return LLAMA_LINEARS if self.arch == "llama" else OPT_LINEARS

    def linear_shape(self, name: str):
        d, kv, ff = self.d_model, self.n_kv_heads * self.head_dim, self.d_ff
        return {"wq": (d, d), "wk": (kv, d), "wv": (kv, d), "wo": (d, d),
                "w_gate": (ff, d), "w_up": (ff, d), "w_down": (d, ff),
                "fc1": (ff, d), "fc2": (d, ff)}[name]

    def linear_list(self):
        """(layer, name, N, K) of every linear in model order; the flat parameter index used
        to key z runs over these tensors in this order, row-major within each."""
        out = []
        for l in range(self.n_layers):
            for nm in self.linear_names():
                N, K = self.linear_shape(nm)
                out.append((l, nm, N, K))
        return out


def _t(a):
    return a if isinstance(a, torch.Tensor) else torch.as_tensor(np.asarray(a), dtype=torch.float64)


def rms_norm(x, gamma, eps):
    return x / torch.sqrt((x * x).mean(dim=-1, keepdim=True) + eps) * gamma


def layer_norm(x, gamma, beta, eps):
    mu = x.mean(dim=-1, keepdim=True)
    var = ((x - mu) ** 2).mean(dim=-1, keepdim=True)
    return (x - mu) / torch.sqrt(var + eps) * gamma + beta


def rope(x, base):
    """x: [B, S, H, hd].  Position p = sequence index; angle theta_i = p * base^(-2i/hd) for the
    pair (i, i + hd/2)."""
    B, S, H, hd = x.shape
    half = hd // 2
    inv = base ** (-(torch.arange(half, dtype=torch.float64) * 2.0) / hd)
    ang = torch.arange(S, dtype=torch.float64)[:, None] * inv[None, :]       # [S, half]
    cos, sin = torch.cos(ang)[None, :, None, :], torch.sin(ang)[None, :, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


def causal_attention(q, k, v):
    """q: [B,S,H,hd]; k, v: [B,S,Hkv,hd].  Returns [B,S,H,hd]."""
    B, S, H, hd = q.shape
    rep = H // k.shape[2]
    out = torch.empty_like(q)
    neg = torch.full((S, S), float("-inf"), dtype=torch.float64).triu(1)
    for h in range(H):
        kh, vh = k[:, :, h // rep, :], v[:, :, h // rep, :]
        s = torch.einsum("bsd,btd->bst", q[:, :, h, :], kh) / math.sqrt(hd) + neg
        p = torch.softmax(s, dim=-1)
        out[:, :, h, :] = torch.einsum("bst,btd->bsd", p, vh)
    return out


def hidden_states(cfg: DecoderConfig, params: dict, lin_W: list, tokens):
    """Final-norm output [B, S, d].  params: 'embed' [V,d], 'final_norm' (+ '_b' for opt),
    'pos' [max_pos,d] (opt), per layer l: f'l{l}.attn_norm', f'l{l}.mlp_norm' (+ '_b'), and
    for opt f'l{l}.{name}_b' biases.  lin_W[l][name] is the effective weight [N,K]."""
    tokens = torch.as_tensor(np.asarray(tokens), dtype=torch.long)
    B, S = tokens.shape
    H, Hkv, hd = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    opt = cfg.arch == "opt"
    h = _t(params["embed"])[tokens]
    if opt:
        h = h + _t(params["pos"])[:S][None, :, :]
    for l in range(cfg.n_layers):
        W = lin_W[l]
        P = lambda nm: _t(params[f"l{l}.{nm}"])

        def lin(x, nm):
            y = x @ _t(W[nm]).T
            return y + P(nm + "_b") if opt else y

        if opt:
            a = layer_norm(h, P("attn_norm"), P("attn_norm_b"), cfg.norm_eps)
        else:
            a = rms_norm(h, P("attn_norm"), cfg.norm_eps)
        q = lin(a, "wq").view(B, S, H, hd)
        k = lin(a, "wk").view(B, S, Hkv, hd)
        v = lin(a, "wv").view(B, S, Hkv, hd)
        if not opt:
            q, k = rope(q, cfg.rope_base), rope(k, cfg.rope_base)
        o = causal_attention(q, k, v).reshape(B, S, H * hd)
        h = h + lin(o, "wo")
        if opt:
            m = layer_norm(h, P("mlp_norm"), P("mlp_norm_b"), cfg.norm_eps)
            h = h + lin(torch.relu(lin(m, "fc1")), "fc2")
        else:
            m = rms_norm(h, P("mlp_norm"), cfg.norm_eps)
            h = h + lin(torch.nn.functional.silu(lin(m, "w_gate")) * lin(m, "w_up"), "w_down")
    if opt:
        return layer_norm(h, _t(params["final_norm"]), _t(params["final_norm_b"]), cfg.norm_eps)
    return rms_norm(h, _t(params["final_norm"]), cfg.norm_eps)


def rope_at(x, base, positions):
    """rope for rows at the given positions: x [B, T, H, hd], positions [T]."""
    B, T, H, hd = x.shape
    half = hd // 2
    inv = base ** (-(torch.arange(half, dtype=torch.float64) * 2.0) / hd)
    ang = torch.as_tensor(positions, dtype=torch.float64)[:, None] * inv[None, :]
    cos, sin = torch.cos(ang)[None, :, None, :], torch.sin(ang)[None, :, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1)


class KVCache:
    """Keys and values of the positions decoded so far, per layer: lists of [B, n, Hkv, hd] tensors."""

    def __init__(self, n_layers):
        self.k = [None] * n_layers
        self.v = [None] * n_layers
        self.n = 0


def decode_step(cfg: DecoderConfig, params: dict, lin_W: list, new_tokens, cache: KVCache):
    """Token generation with a KV cache (the regime of the paper's inference measurements: Section 1's
    speed figure and the appendix on sparse operations): processes T new tokens per sequence
    (new_tokens [B, T]) that follow the cache.n positions already in the cache, appends their keys and
    values, and returns the logits of the LAST new token, [B, V].  Each new position attends to every
    cached position and to the new positions up to itself.  Same blocks as hidden_states."""
    tok = torch.as_tensor(np.asarray(new_tokens), dtype=torch.long)
    B, T = tok.shape
    H, Hkv, hd = cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    opt = cfg.arch == "opt"
    pos = list(range(cache.n, cache.n + T))
    h = _t(params["embed"])[tok]
    if opt:
        h = h + _t(params["pos"])[pos][None, :, :]
    rep = H // Hkv
    for l in range(cfg.n_layers):
        W = lin_W[l]
        P = lambda nm: _t(params[f"l{l}.{nm}"])

        def lin(x, nm):
            y = x @ _t(W[nm]).T
            return y + P(nm + "_b") if opt else y

        a = layer_norm(h, P("attn_norm"), P("attn_norm_b"), cfg.norm_eps) if opt else rms_norm(h, P("attn_norm"), cfg.norm_eps)
        q = lin(a, "wq").view(B, T, H, hd)
        k = lin(a, "wk").view(B, T, Hkv, hd)
        v = lin(a, "wv").view(B, T, Hkv, hd)
        if not opt:
            q, k = rope_at(q, cfg.rope_base, pos), rope_at(k, cfg.rope_base, pos)
        cache.k[l] = k if cache.k[l] is None else torch.cat([cache.k[l], k], dim=1)
        cache.v[l] = v if cache.v[l] is None else torch.cat([cache.v[l], v], dim=1)
        o = torch.empty(B, T, H, hd, dtype=torch.float64)
        for t in range(T):
            n_keys = cache.n + t + 1
            for hh in range(H):
                kh, vh = cache.k[l][:, :n_keys, hh // rep, :], cache.v[l][:, :n_keys, hh // rep, :]
                sc = torch.einsum("bd,bnd->bn", q[:, t, hh, :], kh) / math.sqrt(hd)
                o[:, t, hh, :] = torch.einsum("bn,bnd->bd", torch.softmax(sc, dim=-1), vh)
        h = h + lin(o.reshape(B, T, H * hd), "wo")
        if opt:
            m = layer_norm(h, P("mlp_norm"), P("mlp_norm_b"), cfg.norm_eps)
            h = h + lin(torch.relu(lin(m, "fc1")), "fc2")
        else:
            m = rms_norm(h, P("mlp_norm"), cfg.norm_eps)
            h = h + lin(torch.nn.functional.silu(lin(m, "w_gate")) * lin(m, "w_up"), "w_down")
    cache.n += T
    last = h[:, -1, :]
    if opt:
        last = layer_norm(last, _t(params["final_norm"]), _t(params["final_norm_b"]), cfg.norm_eps)
    else:
        last = rms_norm(last, _t(params["final_norm"]), cfg.norm_eps)
    return last @ _t(params["lm_head"]).T


def _log_softmax(x):
    m = x.max(dim=-1, keepdim=True).values
    return x - m - torch.log(torch.exp(x - m).sum(dim=-1, keepdim=True))


def loss_fn(cfg, params, lin_W, tokens, loss_kind="lm", labels=None, cand=None):
    """Scalar loss f(w; (x, y)) as a 0-d fp64 tensor."""
    hs = hidden_states(cfg, params, lin_W, tokens)
    E = _t(params["lm_head"])
    tok = torch.as_tensor(np.asarray(tokens), dtype=torch.long)
    B, S = tok.shape
    if loss_kind == "lm":
        logits = hs[:, :-1, :] @ E.T                                       # [B, S-1, V]
        lp = _log_softmax(logits)
        tgt = tok[:, 1:]
        return -lp.gather(-1, tgt[..., None]).squeeze(-1).mean()
    if loss_kind == "cls2":
        cand = torch.as_tensor(np.asarray(cand), dtype=torch.long)          # [2]
        lab = torch.as_tensor(np.asarray(labels), dtype=torch.long)         # [B] in {0,1}
        logits = hs[:, -1, :] @ E[cand].T                                    # [B, 2]
        lp = _log_softmax(logits)
        return -lp.gather(-1, lab[:, None]).squeeze(-1).mean()
    raise ValueError(loss_kind)


def linear_gradients(cfg, params, lin_W32: list, tokens, loss_kind="lm", labels=None, cand=None):
    """First-order gradient of the batch-mean loss w.r.t. every linear weight (autograd, fp64),
    used only to choose the sensitive mask before fine-tuning (Definition 3; Section 3.3)."""
    leaves = [{nm: torch.tensor(np.asarray(W[nm], dtype=np.float64), requires_grad=True)
               for nm in cfg.linear_names()} for W in lin_W32]
    loss = loss_fn(cfg, params, leaves, tokens, loss_kind, labels, cand)
    flat = [lv[nm] for lv in leaves for nm in cfg.linear_names()]
    grads = torch.autograd.grad(loss, flat)
    it = iter(grads)
    return [{nm: next(it).numpy() for nm in cfg.linear_names()} for _ in leaves], float(loss.detach())


def accumulate_scores(grad_batches: list) -> list:
    """score = sum over batches of (gradient of the batch-mean loss)^2, formed and accumulated
    in fp32 in batch order: the diagonal of the empirical Fisher that Section 3.1 ties to
    Definition 3."""
    out = None
    for gb in grad_batches:
        sq = [{nm: np.square(g.astype(np.float32)) for nm, g in layer.items()} for layer in gb]
        if out is None:
            out = sq
        else:
            out = [{nm: (o[nm] + s[nm]).astype(np.float32) for nm in o} for o, s in zip(out, sq)]
    return out


# --------------------------------------------------------------------------- ZO-SGD
@dataclass
class SparseQuantModel:
    """The fine-tuning state of Section 3.4/3.5: frozen dequantised dense parts, the index
    list of the mask and the trainable sparse values S (fp32), concatenated over all linears
    in model order.  gidx = flat index over all linear parameters."""
    cfg: DecoderConfig
    params: dict
    W_deq: list                 # [layer][name] fp64 [N,K], Dequantize(Q(w_dense)) (or the dense weight)
    idx_local: list             # [layer][name] int64 indices local to the tensor
    offsets: list               # start of each tensor's entries in S, model order, + total
    gidx: np.ndarray            # int64 [k_total]
    S: np.ndarray               # fp32 [k_total]
    log: list = field(default_factory=list)

    def lin_W(self, S):
        out, t = [], 0
        for l in range(self.cfg.n_layers):
            d = {}
            for nm in self.cfg.linear_names():
                a, b = self.offsets[t], self.offsets[t + 1]
                d[nm] = so.effective_weight(self.W_deq[l][nm], self.idx_local[l][nm], S[a:b])
                t += 1
            out.append(d)
        return out

    def loss(self, S, tokens, loss_kind="lm", labels=None, cand=None) -> float:
        with torch.no_grad():
            return float(loss_fn(self.cfg, self.params, self.lin_W(S), tokens, loss_kind, labels, cand))


def zo_step(model: SparseQuantModel, tokens, seed: int, step: int, eps, lr,
            loss_kind="lm", labels=None, cand=None):
    """One sensitive-sparse ZO-SGD step, in place on model.S, in the seed trick's order:
    S += eps z; f+ ; S -= 2 eps z; f- ; S += eps z; g = (f+ - f-)/(2 eps); S -= lr g z."""
    S, f_plus, f_minus, g = so.zo_sgd_step(
        lambda S_: model.loss(S_, tokens, loss_kind, labels, cand),
        model.S, model.gidx, seed, step, eps, lr)
    model.S = S
    model.log.append((f_plus, f_minus, g))
    return f_plus, f_minus, g
