"""Thin ctypes binding of libszo.so: argument marshalling only.

Function names mirror include/szo.h.  Tensors are torch CUDA tensors (torch is used for device
memory and streams only); every computation runs in the library's kernels.  Loading fails loudly
when the library has not been built: there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libszo.so")

SZO_F32, SZO_BF16, SZO_F16 = 0, 1, 2
MODE_AUTO, MODE_SPARSE_ADD, MODE_SPMM, MODE_FP32_VALIDATE, MODE_PAIRED = 0, 1, 2, 3, 4
LOSS_LM, LOSS_CLS2 = 0, 1
ARCH_LLAMA, ARCH_OPT = 0, 1

_DT = {torch.float32: SZO_F32, torch.bfloat16: SZO_BF16, torch.float16: SZO_F16}
SZ_FMT = {"bf16": (SZO_BF16, torch.bfloat16), "f16": (SZO_F16, torch.float16)}


class SzoError(RuntimeError):
    def __init__(self, code: int, name: str, detail: str):
        super().__init__(f"{name} ({code}): {detail}")
        self.code = code
        self.name = name


class ModelConfig(C.Structure):
    _fields_ = [("arch", C.c_int32), ("n_layers", C.c_int32), ("d_model", C.c_int32),
                ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("d_ff", C.c_int32),
                ("vocab", C.c_int32), ("max_pos", C.c_int32), ("norm_eps", C.c_float),
                ("rope_base", C.c_float), ("group", C.c_int32), ("sz_dtype", C.c_int32),
                ("act_dtype", C.c_int32), ("linear_mode", C.c_int32), ("loss_kind", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32)]


class LinearWeights(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scales", C.c_void_p), ("zeros", C.c_void_p),
                ("idx", C.c_void_p), ("nnz", C.c_int64), ("bias", C.c_void_p)]


class LayerWeights(C.Structure):
    _fields_ = [("attn_norm_g", C.c_void_p), ("attn_norm_b", C.c_void_p),
                ("mlp_norm_g", C.c_void_p), ("mlp_norm_b", C.c_void_p),
                ("lin", LinearWeights * 7)]


class ModelWeights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("pos", C.c_void_p), ("lm_head", C.c_void_p),
                ("final_norm_g", C.c_void_p), ("final_norm_b", C.c_void_p)]


_lib = None

_SIGS = {
    "szo_status_string": (C.c_char_p, [C.c_int32]),
    "szo_last_error": (C.c_char_p, []),
    "szo_version": (C.c_int, []),
    "szo_device_status": (C.c_int32, [C.POINTER(C.c_int32)]),
    "szo_selftest_wait_timeout": (C.c_int32, [C.c_double, C.POINTER(C.c_int32), C.c_void_p]),
    "szo_quantize": (C.c_int32, [C.c_void_p, C.c_int, C.c_int64, C.c_int64, C.c_int32, C.c_int,
                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "szo_select_mask": (C.c_int32, [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                    C.POINTER(C.c_size_t), C.c_void_p]),
    "szo_select_mask_static": (C.c_int32, [C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]),
    "szo_perturb": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                C.c_uint64, C.c_uint64, C.c_float, C.c_void_p]),
    "szo_perturb_keep_z": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64,
                                       C.c_uint64, C.c_uint64, C.c_float, C.c_void_p, C.c_void_p]),
    "szo_perturb3_keep_z": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_uint64, C.c_uint64,
                                        C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "szo_perturb_kept_z": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_float, C.c_void_p]),
    "szo_update_kept_z": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_float, C.c_void_p, C.c_void_p,
                                      C.c_float, C.c_void_p]),
    "szo_projected_gradient": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]),
    "szo_update": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_uint64, C.c_uint64,
                               C.c_float, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]),
    "szo_round_sparse16": (C.c_int32, [C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_void_p]),
    "szo_model_set_sparse_storage": (C.c_int32, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]),
    "szo_replay": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_uint64, C.POINTER(C.c_uint64),
                               C.POINTER(C.c_double), C.c_int64, C.c_float, C.c_float, C.c_void_p]),
    "szo_linear_create": (C.c_int32, [C.POINTER(C.c_void_p), C.c_int64, C.c_int64, C.c_int32,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                      C.c_int64, C.c_void_p, C.c_void_p]),
    "szo_linear_create_lut": (C.c_int32, [C.POINTER(C.c_void_p), C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                          C.c_int, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]),
    "szo_linear_fwd": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int, C.c_int64, C.c_void_p, C.c_void_p,
                                   C.c_int, C.c_int32, C.c_void_p, C.c_size_t, C.c_void_p]),
    "szo_linear_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int64, C.c_int32]),
    "szo_linear_paired_workspace_bytes": (C.c_size_t, [C.c_void_p, C.c_int64]),
    "szo_linear_fwd_paired": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_float,
                                          C.c_void_p, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]),
    "szo_linear_destroy": (None, [C.c_void_p]),
    "szo_attention_paired": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int64, C.c_int32,
                                         C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "szo_attention": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int32, C.c_int32,
                                  C.c_int32, C.c_int32, C.c_int32, C.c_void_p]),
    "szo_model_create": (C.c_int32, [C.POINTER(C.c_void_p), C.POINTER(ModelConfig),
                                     C.POINTER(ModelWeights), C.POINTER(LayerWeights), C.c_void_p,
                                     C.c_void_p]),
    "szo_model_k_total": (C.c_int64, [C.c_void_p]),
    "szo_model_gidx": (C.c_void_p, [C.c_void_p]),
    "szo_model_loss": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                   C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "szo_model_zo_step": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                      C.c_int32, C.c_uint64, C.c_uint64, C.c_float, C.c_float,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "szo_model_zo_step_n": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_uint64, C.c_uint64, C.c_int32, C.c_float, C.c_float, C.c_void_p,
                                        C.c_void_p, C.c_void_p, C.c_void_p]),
    "szo_model_zo_losses": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_uint64, C.c_uint64, C.c_float, C.c_void_p, C.c_void_p]),
    "szo_model_zo_apply": (C.c_int32, [C.c_void_p, C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p,
                                       C.c_void_p, C.c_void_p]),
    "szo_model_zo_step_host": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                           C.c_int32, C.c_uint64, C.c_uint64, C.c_float, C.c_float,
                                           C.c_void_p, C.c_void_p]),
    "szo_model_enable_decode": (C.c_int32, [C.c_void_p, C.c_void_p]),
    "szo_model_decode_step": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                          C.c_void_p, C.c_void_p]),
    "szo_model_last_launches": (C.c_int64, [C.c_void_p]),
    "szo_model_enable_timing": (C.c_int32, [C.c_void_p, C.c_int32]),
    "szo_model_linear_time": (C.c_int32, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "szo_model_destroy": (None, [C.c_void_p]),
}


def exported_symbols():
    """Names declared in include/szo.h."""
    return sorted(_SIGS)


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2406_02913_b200.build` (no fallback exists)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGS.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _check(code: int):
    if code != 0:
        L = lib()
        raise SzoError(code, L.szo_status_string(code).decode(), L.szo_last_error().decode())


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous(), "expected a contiguous CUDA tensor"
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def device_status() -> int:
    v = C.c_int32(0)
    _check(lib().szo_device_status(C.byref(v)))
    return v.value


def selftest_wait_timeout(limit_ms: float = 2.0) -> int:
    """1 when the kernel's bounded wait gave up (as it must); the status word then holds SZO_ERR_TIMEOUT."""
    v = C.c_int32(0)
    _check(lib().szo_selftest_wait_timeout(limit_ms, C.byref(v), _stream()))
    return v.value


# ------------------------------------------------------------------------------ element ops
def szo_quantize(W: torch.Tensor, G: int, sz_fmt: str = "bf16"):
    """Returns (codes uint8 [N,K/2], scales [N,K/G], zeros [N,K/G])."""
    N, K = W.shape
    sz_code, sz_torch = SZ_FMT[sz_fmt]
    codes = torch.empty((N, K // 2), dtype=torch.uint8, device=W.device)
    ng = K // G if G > 0 and K % G == 0 else 1
    scales = torch.empty((N, ng), dtype=sz_torch, device=W.device)
    zeros = torch.empty((N, ng), dtype=sz_torch, device=W.device)
    _check(lib().szo_quantize(_ptr(W), _DT[W.dtype], N, K, G, sz_code, _ptr(codes), _ptr(scales),
                              _ptr(zeros), _stream()))
    return codes, scales, zeros


def szo_select_mask(scores: torch.Tensor, k: int) -> torch.Tensor:
    n = scores.numel()
    idx = torch.empty((max(k, 1),), dtype=torch.int64, device=scores.device)
    nbytes = C.c_size_t(0)
    _check(lib().szo_select_mask(_ptr(scores), n, k, _ptr(idx), None, C.byref(nbytes), _stream()))
    ws = torch.empty((max(nbytes.value, 16),), dtype=torch.uint8, device=scores.device)
    _check(lib().szo_select_mask(_ptr(scores), n, k, _ptr(idx), _ptr(ws), C.byref(nbytes), _stream()))
    return idx[:k]


def szo_select_mask_static(scores: torch.Tensor, k: int, out: torch.Tensor) -> torch.Tensor:
    """Top-k mask into the caller's `out` (int64, at least k long) using the library's built-in
    scratch: for callers that must not allocate device memory.  At most 2**26 scores."""
    _check(lib().szo_select_mask_static(_ptr(scores), scores.numel(), k, _ptr(out), _stream()))
    return out[:k]


def szo_perturb(S_in, S_out, idx, idx_base: int, seed: int, step: int, scale: float):
    _check(lib().szo_perturb(_ptr(S_in), _ptr(S_out), _ptr(idx), idx.numel(), idx_base, seed, step,
                             scale, _stream()))


def szo_perturb_keep_z(S_in, S_out, idx, idx_base: int, seed: int, step: int, scale: float, z_out):
    _check(lib().szo_perturb_keep_z(_ptr(S_in), _ptr(S_out), _ptr(idx), idx.numel(), idx_base, seed, step,
                                    scale, _ptr(z_out), _stream()))


def szo_perturb3_keep_z(S_in, S_out, idx, idx_base: int, seed: int, step: int, eps: float, z_out, S_plus=None, S_minus=None):
    """The +eps, -2 eps, +eps passes in one launch (szo_perturb3_keep_z)."""
    _check(lib().szo_perturb3_keep_z(_ptr(S_in), _ptr(S_out), _ptr(idx), idx.numel(), idx_base, seed, step, eps,
                                     _ptr(z_out), _ptr(S_plus), _ptr(S_minus), _stream()))


def szo_perturb_kept_z(S_in, S_out, z, scale: float):
    _check(lib().szo_perturb_kept_z(_ptr(S_in), _ptr(S_out), _ptr(z), z.numel(), scale, _stream()))


def szo_update_kept_z(S, z, lr: float, f_plus, f_minus, eps: float):
    _check(lib().szo_update_kept_z(_ptr(S), _ptr(z), z.numel(), lr, _ptr(f_plus), _ptr(f_minus), eps, _stream()))


def szo_projected_gradient(f_plus, f_minus, eps: float, g_out):
    _check(lib().szo_projected_gradient(_ptr(f_plus), _ptr(f_minus), eps, _ptr(g_out), _stream()))


def szo_update(S, idx, idx_base: int, seed: int, step: int, lr: float, f_plus, f_minus, eps: float):
    _check(lib().szo_update(_ptr(S), _ptr(idx), idx.numel(), idx_base, seed, step, lr, _ptr(f_plus),
                            _ptr(f_minus), eps, _stream()))


def szo_replay(S, idx, idx_base: int, seed: int, log, eps: float, lr: float):
    """Applies the logged steps [(step, g), ...] to S in place (szo_replay)."""
    n = len(log)
    steps = (C.c_uint64 * max(n, 1))(*[int(s) for s, _ in log])
    gs = (C.c_double * max(n, 1))(*[float(g) for _, g in log])
    _check(lib().szo_replay(_ptr(S), _ptr(idx), idx.numel(), idx_base, seed, steps, gs, n, eps, lr, _stream()))


def szo_round_sparse16(S, fmt: str, out=None):
    """Rounds S (fp32 CUDA tensor) in place to values representable in 'bf16' or 'f16'; `out` (16-bit tensor of
    the same length) receives the stored form (szo_round_sparse16)."""
    _check(lib().szo_round_sparse16(_ptr(S), S.numel(), SZO_BF16 if fmt == "bf16" else SZO_F16, _ptr(out), _stream()))


# ------------------------------------------------------------------------------ linear layer
class Linear:
    """Plan for one decomposed linear (szo_linear_create / szo_linear_fwd)."""

    def __init__(self, N, K, G, codes_or_W, scales, zeros, sz_fmt, idx, bias=None, lut=None):
        """lut (16-bit float CUDA tensor [N,16]) selects the non-uniform 4-bit format
        (szo_linear_create_lut); G, scales and zeros are then ignored."""
        self.N, self.K, self.G = N, K, (-1 if lut is not None else G)
        self._keep = (codes_or_W, scales, zeros, idx, bias, lut)      # plan borrows these buffers
        self.nnz = 0 if idx is None else idx.numel()
        h = C.c_void_p()
        if lut is not None:
            _check(lib().szo_linear_create_lut(C.byref(h), N, K, _ptr(codes_or_W), _ptr(lut), _DT[lut.dtype],
                                               _ptr(idx) if self.nnz else None, self.nnz, _ptr(bias), _stream()))
        else:
            _check(lib().szo_linear_create(C.byref(h), N, K, G, _ptr(codes_or_W), _ptr(scales), _ptr(zeros),
                                           SZ_FMT[sz_fmt][0], _ptr(idx) if self.nnz else None, self.nnz,
                                           _ptr(bias), _stream()))
        self.h = h
        self._ws = None

    def workspace_bytes(self, M, mode):
        return lib().szo_linear_workspace_bytes(self.h, M, mode)

    def fwd(self, x, S_pert, mode=MODE_AUTO, out_dtype=torch.bfloat16, y=None):
        M = x.shape[0]
        if y is None:
            y = torch.empty((M, self.N), dtype=out_dtype, device=x.device)
        need = self.workspace_bytes(M, mode)
        if need and (self._ws is None or self._ws.numel() < need):
            self._ws = torch.empty((need,), dtype=torch.uint8, device=x.device)
        _check(lib().szo_linear_fwd(self.h, _ptr(x), _DT[x.dtype], M, _ptr(S_pert) if self.nnz else None,
                                    _ptr(y), _DT[y.dtype], mode, _ptr(self._ws) if need else None, need,
                                    _stream()))
        return y

    def fwd_paired(self, x, M, S, z, eps, out_dtype=torch.bfloat16):
        """x: bf16 [paired_row0(M) + M, K] (centre rows, then half-difference rows); returns y in the
        same row layout."""
        rows = paired_row0(M) + M
        assert x.shape[0] == rows
        y = torch.zeros((rows, self.N), dtype=out_dtype, device=x.device)
        need = lib().szo_linear_paired_workspace_bytes(self.h, M)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty((need,), dtype=torch.uint8, device=x.device)
        _check(lib().szo_linear_fwd_paired(self.h, _ptr(x), M, _ptr(S) if self.nnz else None,
                                           _ptr(z) if self.nnz else None, eps, _ptr(y), _DT[y.dtype], _ptr(self._ws),
                                           need, _stream()))
        return y

    def close(self):
        if getattr(self, "h", None):
            lib().szo_linear_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def paired_row0(M: int) -> int:
    """First half-difference row of a paired buffer with M centre rows."""
    return (M + 255) // 256 * 256


def szo_attention_paired(q, k, v, row0: int, B: int, S: int, n_heads: int, n_kv_heads: int, head_dim: int):
    """Paired causal attention; every tensor holds B*S centre rows and, from row row0 on, B*S
    half-difference rows (bf16).  Returns o like q."""
    o = torch.zeros_like(q)
    _check(lib().szo_attention_paired(_ptr(q), _ptr(k), _ptr(v), _ptr(o), row0, B, S, n_heads, n_kv_heads,
                                      head_dim, _stream()))
    return o


def szo_attention(q, k, v, B: int, S: int, n_heads: int, n_kv_heads: int, head_dim: int):
    """Causal attention; q [B*S, H*hd], k/v [B*S, Hkv*hd] (bf16 or fp32).  Returns o like q."""
    o = torch.empty_like(q)
    _check(lib().szo_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(o), _DT[q.dtype], B, S, n_heads, n_kv_heads,
                               head_dim, _stream()))
    return o


# ------------------------------------------------------------------------------ model
class Model:
    """Whole-decoder loss and ZO step (szo_model_*).  `tensors` maps names to CUDA tensors:
    'embed', 'lm_head', 'pos', 'final_norm', 'final_norm_b', per layer 'l{i}.attn_norm',
    'l{i}.mlp_norm' (+'_b'), and per linear 'l{i}.{name}.codes|scales|zeros|idx|bias'.
    S_all is the fp32 CUDA tensor of all sparse values in model order."""

    def __init__(self, shape: dict, linear_names, tensors: dict, S_all, *, act_dtype=SZO_BF16,
                 linear_mode=MODE_AUTO, loss_kind=LOSS_LM, max_batch=16, max_seq=512,
                 norm_eps=1e-5, rope_base=10000.0):
        self.tensors = tensors
        self.S_all = S_all
        cfg = ModelConfig(arch=ARCH_LLAMA if shape["arch"] == "llama" else ARCH_OPT,
                          n_layers=shape["n_layers"], d_model=shape["d_model"], n_heads=shape["n_heads"],
                          n_kv_heads=shape["n_kv_heads"], d_ff=shape["d_ff"], vocab=shape["vocab"],
                          max_pos=shape["max_pos"], norm_eps=norm_eps, rope_base=rope_base,
                          group=shape["group"], sz_dtype=SZ_FMT[shape["sz_fmt"]][0], act_dtype=act_dtype,
                          linear_mode=linear_mode, loss_kind=loss_kind, max_batch=max_batch,
                          max_seq=max_seq)
        top = ModelWeights(embed=_ptr(tensors["embed"]), pos=_ptr(tensors.get("pos")),
                           lm_head=_ptr(tensors["lm_head"]), final_norm_g=_ptr(tensors["final_norm"]),
                           final_norm_b=_ptr(tensors.get("final_norm_b")))
        layers = (LayerWeights * shape["n_layers"])()
        for l in range(shape["n_layers"]):
            lw = layers[l]
            lw.attn_norm_g = _ptr(tensors[f"l{l}.attn_norm"])
            lw.attn_norm_b = _ptr(tensors.get(f"l{l}.attn_norm_b"))
            lw.mlp_norm_g = _ptr(tensors[f"l{l}.mlp_norm"])
            lw.mlp_norm_b = _ptr(tensors.get(f"l{l}.mlp_norm_b"))
            for j, nm in enumerate(linear_names):
                p = f"l{l}.{nm}."
                idx = tensors.get(p + "idx")
                lw.lin[j].codes = _ptr(tensors[p + "codes"])
                lw.lin[j].scales = _ptr(tensors.get(p + ("lut" if shape["group"] == -1 else "scales")))
                lw.lin[j].zeros = _ptr(tensors.get(p + "zeros"))
                lw.lin[j].nnz = 0 if idx is None else idx.numel()
                lw.lin[j].idx = _ptr(idx) if lw.lin[j].nnz else None
                lw.lin[j].bias = _ptr(tensors.get(p + "bias"))
        h = C.c_void_p()
        _check(lib().szo_model_create(C.byref(h), C.byref(cfg), C.byref(top), layers, _ptr(S_all), _stream()))
        self.h = h
        self.cfg = cfg
        self.k_total = lib().szo_model_k_total(h)
        self._scalars = torch.zeros(4, dtype=torch.float64, device=S_all.device)

    def gidx(self) -> torch.Tensor:
        """Copy of the model's global index list (int64 [k_total])."""
        out = torch.empty((self.k_total,), dtype=torch.int64, device=self.S_all.device)
        src = lib().szo_model_gidx(self.h)
        if self.k_total:
            _memcpy_d2d(out.data_ptr(), src, self.k_total * 8)
        return out

    def loss(self, tokens, labels=None, cand=None, S_vals=None) -> torch.Tensor:
        B, S = tokens.shape
        out = self._scalars[3:4]
        _check(lib().szo_model_loss(self.h, _ptr(tokens), _ptr(labels), _ptr(cand), B, S, _ptr(S_vals),
                                    _ptr(out), _stream()))
        return out

    def zo_step(self, tokens, seed, step, eps, lr, labels=None, cand=None) -> torch.Tensor:
        """Enqueues one step; returns the device tensor (f+, f-, g) (fp64 [3])."""
        B, S = tokens.shape
        sc = self._scalars
        _check(lib().szo_model_zo_step(self.h, _ptr(tokens), _ptr(labels), _ptr(cand), B, S, seed, step,
                                       eps, lr, sc[0:1].data_ptr(), sc[1:2].data_ptr(),
                                       sc[2:3].data_ptr(), _stream()))
        return sc[:3]

    def set_sparse_storage(self, fmt, out=None):
        """Sparse values stored in 'bf16' or 'f16' (None or 'f32': off): every update is followed by one rounding to
        the format; `out` (16-bit tensor [k_total]) mirrors the stored form (szo_model_set_sparse_storage)."""
        dt = {None: SZO_F32, "f32": SZO_F32, "bf16": SZO_BF16, "f16": SZO_F16}[fmt]
        self._keep_s16 = out
        _check(lib().szo_model_set_sparse_storage(self.h, dt, _ptr(out), _stream()))

    def zo_step_n(self, tokens, seed, step, n, eps, lr, labels=None, cand=None) -> torch.Tensor:
        """n-sample SPSA step; returns the device tensor [3, n] of (f+_i, f-_i, g_i) (fp64)."""
        B, S = tokens.shape
        out = torch.zeros((3, n), dtype=torch.float64, device=self.S_all.device)
        _check(lib().szo_model_zo_step_n(self.h, _ptr(tokens), _ptr(labels), _ptr(cand), B, S, seed, step, n, eps, lr,
                                         out[0].data_ptr(), out[1].data_ptr(), out[2].data_ptr(), _stream()))
        return out

    def zo_losses(self, tokens, seed, step, eps, labels=None, cand=None, sums=None) -> torch.Tensor:
        """First half of a step on this replica's share of the batch: returns the device tensor
        (sum of losses of f+, of f-, number of positions) (fp64 [3]); z stays in the model."""
        B, S = tokens.shape
        if sums is None:
            sums = torch.zeros(3, dtype=torch.float64, device=self.S_all.device)
        _check(lib().szo_model_zo_losses(self.h, _ptr(tokens), _ptr(labels), _ptr(cand), B, S, seed, step, eps,
                                         _ptr(sums), _stream()))
        return sums

    def zo_apply(self, eps, lr, sums) -> torch.Tensor:
        """Second half: `sums` added up over all replicas; returns the device tensor (f+, f-, g)."""
        sc = self._scalars
        _check(lib().szo_model_zo_apply(self.h, eps, lr, _ptr(sums), sc[0:1].data_ptr(), sc[1:2].data_ptr(),
                                        sc[2:3].data_ptr(), _stream()))
        return sc[:3]

    def zo_step_host(self, tokens_host, seed, step, eps, lr, labels_host=None, cand_host=None):
        """Host-buffer variant: tokens_host etc. are CPU int32 tensors (pinned for speed)."""
        B, S = tokens_host.shape
        out = (C.c_double * 3)()
        hp = lambda t: None if t is None else t.data_ptr()
        _check(lib().szo_model_zo_step_host(self.h, hp(tokens_host), hp(labels_host), hp(cand_host), B, S,
                                            seed, step, eps, lr, C.cast(out, C.c_void_p), _stream()))
        return out[0], out[1], out[2]

    def enable_decode(self):
        _check(lib().szo_model_enable_decode(self.h, _stream()))

    def decode_step(self, tokens, pos0: int, logits=None, S_vals=None) -> torch.Tensor:
        """tokens int32 [B, T] following pos0 cached positions; returns fp32 logits [B, vocab] of the last one."""
        B, T = tokens.shape
        if logits is None:
            logits = torch.empty((B, self.cfg.vocab), dtype=torch.float32, device=tokens.device)
        _check(lib().szo_model_decode_step(self.h, _ptr(tokens), B, T, pos0, _ptr(S_vals), _ptr(logits), _stream()))
        return logits

    def enable_timing(self, on: bool = True):
        _check(lib().szo_model_enable_timing(self.h, 1 if on else 0))

    def linear_time(self):
        """(total ms, launches) of the decoder-block linears since the last call."""
        ms, n = C.c_double(0), C.c_int64(0)
        _check(lib().szo_model_linear_time(self.h, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def last_launches(self) -> int:
        return lib().szo_model_last_launches(self.h)

    def close(self):
        if getattr(self, "h", None):
            lib().szo_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _memcpy_d2d(dst: int, src: int, nbytes: int):
    # torch-only device copy between raw pointers: wrap the source in a tensor view
    src_t = _as_cuda_u8(src, nbytes)
    dst_t = _as_cuda_u8(dst, nbytes)
    dst_t.copy_(src_t)


def _as_cuda_u8(ptr: int, nbytes: int) -> torch.Tensor:
    class _Holder:
        pass
    h = _Holder()
    h.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (ptr, False), "version": 2}
    return torch.as_tensor(h, device="cuda")
