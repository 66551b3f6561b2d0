"""Test fixtures shared by the parity tests: one seeded decoder workload, prepared once on the CPU
(oracle side) and uploadable to the GPU library.  Nothing here computes on the GPU."""
from __future__ import annotations

import numpy as np

from oracle import model_oracle as mo
from oracle import szo_oracle as so
from paper_2406_02913_b200 import workloads as wl


def decoder_config(shape: dict) -> mo.DecoderConfig:
    return mo.DecoderConfig(arch=shape["arch"], n_layers=shape["n_layers"], d_model=shape["d_model"],
                            n_heads=shape["n_heads"], n_kv_heads=shape["n_kv_heads"], d_ff=shape["d_ff"],
                            vocab=shape["vocab"], max_pos=shape["max_pos"])


def table_coded(Wd: np.ndarray, fmt: str):
    """A stand-in for a non-uniform 4-bit quantizer (fitting the tables is outside the library): per
    row the 16 values are the (i + 1/2)/16 quantiles of the row, rounded to `fmt`; each weight takes
    the code of its nearest value.  Returns (packed codes uint8 [N,K/2], table bits uint16 [N,16])."""
    q = (np.arange(16) + 0.5) / 16.0
    lut = np.quantile(Wd.astype(np.float64), q, axis=1).T.astype(np.float32)           # [N,16], ascending
    lb, lv = so.round_to_16(lut, fmt)
    code = np.argmin(np.abs(Wd[:, :, None].astype(np.float64) - lv[:, None, :].astype(np.float64)), axis=2).astype(np.uint8)
    return (code[:, 0::2] | (code[:, 1::2] << 4)).astype(np.uint8), lb


class DecoderFixture:
    """Weights -> mask (top-k of accumulated squared gradients, or a random sample) -> decompose ->
    quantize, all with the oracle; keeps every intermediate for comparison."""

    def __init__(self, name: str, seed: int = 0, mask: str = "gradient", n_mask_batches: int = 4,
                 B: int = 4, S: int = 64, n_layers: int | None = None, rho: float | None = None):
        shape = dict(wl.MODEL_SHAPES[name])
        if n_layers:
            shape["n_layers"] = n_layers
        if rho is not None:
            shape["rho"] = rho
        self.shape, self.seed, self.B, self.S = shape, seed, B, S
        self.cfg = decoder_config(shape)
        self.names = wl.linear_names(shape)
        self.params, self.lin_W = wl.init_params(shape, seed)
        G, fmt = shape["group"], shape["sz_fmt"]
        if mask == "gradient":
            grads = []
            for b in range(n_mask_batches):
                toks = wl.token_batch(shape["vocab"], B, S, seed, wl.PURPOSE_MASK_BATCH, b)
                g, _ = mo.linear_gradients(self.cfg, self.params, self.lin_W, toks)
                grads.append(g)
            self.scores = mo.accumulate_scores(grads)
        else:
            self.scores = None
        self.idx, self.S0, self.W_dense, self.q = [], [], [], []
        W_deq, offsets, gidx = [], [0], []
        base = 0
        for l in range(shape["n_layers"]):
            il, dl, ql, wl_ = {}, {}, {}, {}
            for j, nm in enumerate(self.names):
                W = self.lin_W[l][nm]
                k = int(np.floor(shape["rho"] * W.size))
                if self.scores is not None:
                    idx = so.select_mask(self.scores[l][nm].ravel(), k)
                else:
                    idx = wl.sorted_random_indices(W.size, k, seed, 100 * l + j)
                s, Wd = so.decompose(W, idx)
                if G > 0:
                    codes, sb, zb = so.quantize_int4(Wd, G, fmt)
                    dq = so.dequantize(codes, sb, zb, G, fmt)
                    ql[nm] = (codes, sb, zb)
                elif G < 0:
                    codes, lb = table_coded(Wd, fmt)
                    dq = so.dequantize_lut(codes, lb, fmt)
                    ql[nm] = (codes, lb, None)
                else:
                    Wd = wl.bf16_round(Wd)
                    dq = Wd.astype(np.float64)
                    ql[nm] = None
                il[nm], dl[nm], wl_[nm] = idx, dq, Wd
                self.S0.append(s)
                gidx.append(idx + base)
                offsets.append(offsets[-1] + k)
                base += W.size
            self.idx.append(il)
            W_deq.append(dl)
            self.q.append(ql)
            self.W_dense.append(wl_)
        self.offsets = offsets
        self.gidx = np.concatenate(gidx)
        self.S_init = np.concatenate(self.S0).astype(np.float32)
        self.W_deq = W_deq

    def oracle_model(self) -> mo.SparseQuantModel:
        return mo.SparseQuantModel(self.cfg, self.params, self.W_deq, self.idx, self.offsets, self.gidx,
                                   self.S_init.copy())

    def batch(self, i: int):
        return wl.token_batch(self.shape["vocab"], self.B, self.S, self.seed, wl.PURPOSE_TRAIN_BATCH, i)

    def gpu_tensors(self, torch, quantize_on_gpu=None):
        """Upload to CUDA tensors named as binding.Model expects.  quantize_on_gpu(Wd_cuda, G, fmt)
        -> (codes, scales, zeros) lets the caller run the library's own quantizer instead of
        uploading the oracle's codes."""
        G, fmt = self.shape["group"], self.shape["sz_fmt"]
        t = {}
        up = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).cuda() if dt is None
                                 else torch.from_numpy(np.ascontiguousarray(a)).cuda().to(dt))
        t["embed"] = up(self.params["embed"], torch.bfloat16)
        t["lm_head"] = up(self.params["lm_head"], torch.bfloat16)
        t["final_norm"] = up(self.params["final_norm"])
        if self.shape["arch"] == "opt":
            t["pos"] = up(self.params["pos"], torch.bfloat16)
            t["final_norm_b"] = up(self.params["final_norm_b"])
        for l in range(self.shape["n_layers"]):
            for nm in ("attn_norm", "mlp_norm"):
                t[f"l{l}.{nm}"] = up(self.params[f"l{l}.{nm}"])
                if self.shape["arch"] == "opt":
                    t[f"l{l}.{nm}_b"] = up(self.params[f"l{l}.{nm}_b"])
            for nm in self.names:
                p = f"l{l}.{nm}."
                if G < 0:
                    codes, lb, _ = self.q[l][nm]
                    dt = torch.bfloat16 if fmt == "bf16" else torch.float16
                    t[p + "codes"], t[p + "lut"] = up(codes), up(lb.view(np.int16)).view(dt)
                elif G > 0:
                    if quantize_on_gpu is not None:
                        codes, sc, ze = quantize_on_gpu(up(self.W_dense[l][nm]), G, fmt)
                    else:
                        codes, sb, zb = self.q[l][nm]
                        dt = torch.bfloat16 if fmt == "bf16" else torch.float16
                        codes = up(codes)
                        sc = up(sb.view(np.int16)).view(dt)
                        ze = up(zb.view(np.int16)).view(dt)
                    t[p + "codes"], t[p + "scales"], t[p + "zeros"] = codes, sc, ze
                else:
                    t[p + "codes"] = up(self.W_dense[l][nm], torch.bfloat16)
                t[p + "idx"] = up(self.idx[l][nm])
                if self.shape["arch"] == "opt":
                    t[p + "bias"] = up(self.params[f"l{l}.{nm}_b"])
        return t
