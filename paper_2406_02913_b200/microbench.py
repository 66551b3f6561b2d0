"""Kernel microbenchmarks through the C ABI: one JSON line per case.

    python -m paper_2406_02913_b200.microbench linear --M 8192 [--N 4096 --K 4096 --mode sparse_add]
    python -m paper_2406_02913_b200.microbench sparse --k 6476005
    python -m paper_2406_02913_b200.microbench steady --M 8 --N 11008 --K 4096 --mode auto
    python -m paper_2406_02913_b200.microbench sweep            # the single-linear and k-sweep cases
    python -m paper_2406_02913_b200.microbench step --model opt_13b --batch 8 --seq 512 --loss lm

linear: x bf16 [M,K] ~ N(0,1); W [N,K] int4 group-128 with bf16 scales/zeros quantized (by the
library) from N(0,0.02); 0.1 % sparse entries chosen as the top-k of squared Student-t(3) scores
(by the library); the perturbed forward is timed.  sparse: one perturb pass over k sorted random
indices.  Timing: CUDA events on the launching stream, L2 flushed by writing a 512 MB buffer before
every timed launch, median of the repetitions.  steady: the few-token regime, where a call lasts
microseconds and the time between an event and a lone launch is of the same size: enough plans of the
same shape to exceed L2 several times are called in turn inside one CUDA graph (weights from HBM,
code resident, host out of the loop); the time per call is the graph's time over the calls in it.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2406_02913_b200 import binding as B  # noqa: E402
from paper_2406_02913_b200 import workloads as wl  # noqa: E402


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


_flush = None


def flush_l2():
    global _flush
    if _flush is None:
        _flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    _flush.fill_(1)


def time_call(fn, reps, warmup=3, flush=True):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        if flush:
            flush_l2()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return statistics.median(ts), min(ts)


def linear_case(M, N, K, G, mode, rho, reps, out_dtype=torch.bfloat16):
    W = torch.from_numpy(wl.gaussian_matrix(N, K, 0.02, seed=0, i=1)).cuda()
    g = torch.from_numpy(wl.student_t_gradient(N * K, 3.0, seed=0, i=2)).cuda()
    nnz = int(rho * N * K)
    idx = B.szo_select_mask(g * g, nnz)
    S = W.view(-1)[idx].contiguous()
    W.view(-1)[idx] = 0.0
    plan_args, lut = None, None
    if G > 0:
        codes, sc, ze = B.szo_quantize(W, G, "bf16")
        plan_args = (codes, sc, ze)
    elif G < 0:    # non-uniform 4-bit format: random codes into per-row tables of 16 fp16 values
        plan_args = (torch.from_numpy(wl.random_codes(N, K, seed=0, i=4)).cuda(), None, None)
        lut = torch.from_numpy(wl.random_lut(N, seed=0, i=5)).cuda().to(torch.float16)
    else:
        plan_args = (W.to(torch.bfloat16), None, None)
    plan = B.Linear(N, K, G, plan_args[0], plan_args[1], plan_args[2], "bf16", idx, lut=lut)
    x = torch.from_numpy(wl.activation(M, K, seed=0, i=3)).cuda().to(torch.bfloat16)
    S_pert = torch.empty_like(S)
    B.szo_perturb(S, S_pert, idx, 0, 1234, 0, 1e-3)
    y = torch.empty((M, N), dtype=out_dtype, device="cuda")
    md = MODES[mode]
    med, best = time_call(lambda: plan.fwd(x, S_pert, md, out_dtype, y=y), reps)
    hbm, tf, src = peaks()
    flops = 2.0 * M * N * K
    w_bytes = N * K / 2 + 4 * N * K / G if G > 0 else (N * K / 2 + 32 * N if G < 0 else 2 * N * K)
    byts = w_bytes + 2 * M * K + y.element_size() * M * N + 8 * nnz
    t_roof = max(flops / (tf * 1e12), byts / (hbm * 1e9))
    line = {"case": "linear", "M": M, "N": N, "K": K, "G": G, "mode": mode, "nnz": nnz, "ms_median": med,
            "ms_min": best, "tflops": flops / (med * 1e-3) / 1e12, "gbs": byts / (med * 1e-3) / 1e9,
            "bound": "tensor" if flops / (tf * 1e12) >= byts / (hbm * 1e9) else "hbm",
            "roofline_ms": t_roof * 1e3, "frac_of_roofline": t_roof * 1e3 / med, "peaks": src,
            "status": B.device_status()}
    print(json.dumps(line), flush=True)
    plan.close()
    return line


MODES = {"auto": B.MODE_AUTO, "sparse_add": B.MODE_SPARSE_ADD, "spmm": B.MODE_SPMM, "fp32": B.MODE_FP32_VALIDATE}


def steady_case(M, N, K, G, mode, rho, reps, total_bytes=400e6):
    W = torch.from_numpy(wl.gaussian_matrix(N, K, 0.02, seed=0, i=1)).cuda()
    g = torch.from_numpy(wl.student_t_gradient(N * K, 3.0, seed=0, i=2)).cuda()
    nnz = int(rho * N * K)
    idx = B.szo_select_mask(g * g, nnz)
    S = W.view(-1)[idx].contiguous()
    W.view(-1)[idx] = 0.0
    n_plans = max(2, int(total_bytes / (N * K / 2)) + 1)
    if G > 0:
        codes, sc, ze = B.szo_quantize(W, G, "bf16")
        keep = [(codes.clone(), sc.clone(), ze.clone(), idx.clone(), S.clone()) for _ in range(n_plans)]
        plans = [B.Linear(N, K, G, c, s_, z_, "bf16", i_) for (c, s_, z_, i_, _) in keep]
    else:          # non-uniform 4-bit format: random codes into per-row tables of 16 fp16 values
        codes = torch.from_numpy(wl.random_codes(N, K, seed=0, i=4)).cuda()
        lut = torch.from_numpy(wl.random_lut(N, seed=0, i=5)).cuda().to(torch.float16)
        keep = [(codes.clone(), lut.clone(), None, idx.clone(), S.clone()) for _ in range(n_plans)]
        plans = [B.Linear(N, K, G, c, None, None, "bf16", i_, lut=l_) for (c, l_, _, i_, _) in keep]
    x = torch.from_numpy(wl.activation(M, K, seed=0, i=3)).cuda().to(torch.bfloat16)
    ys = [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(n_plans)]
    rounds = 4

    def run_all():
        for r in range(n_plans):
            plans[r].fwd(x, keep[r][4], MODES[mode], torch.bfloat16, y=ys[r])

    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        for _ in range(3):
            run_all()                                   # workspaces and function attributes exist before the capture
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=st):
            for _ in range(rounds):
                run_all()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / (rounds * n_plans))
    med = statistics.median(ts)
    hbm, _, src = peaks()
    byts = N * K / 2 + (4 * N * K / G if G > 0 else 32 * N) + 2 * M * K + 2 * M * N + 8 * nnz
    line = {"case": "linear_steady", "M": M, "N": N, "K": K, "G": G, "mode": mode, "nnz": nnz, "plans": n_plans,
            "us_per_call_median": med * 1e3, "us_per_call_min": min(ts) * 1e3, "gbs": byts / (med * 1e-3) / 1e9,
            "frac_of_hbm": byts / (med * 1e-3) / 1e9 / hbm, "peaks": src, "status": B.device_status()}
    print(json.dumps(line), flush=True)
    for pl in plans:
        pl.close()
    return line


def sparse_case(k, reps, n_total=12_582_912_000):
    g = torch.Generator(device="cuda")
    g.manual_seed(k % 1000003)
    idx = torch.sort(torch.randint(0, n_total, (k,), generator=g, device="cuda", dtype=torch.int64)).values
    S = torch.randn(k, generator=g, device="cuda") * 0.02
    out = torch.empty_like(S)
    hbm, _, src = peaks()
    res = {}
    for name, dst, fl in (("out_of_place_cold", out, True), ("in_place_cold", S, True), ("in_place_warm", S, False)):
        med, best = time_call(lambda: B.szo_perturb(S, dst, idx, 0, 1234, 1, 1e-3), reps, flush=fl)
        res[name] = {"ms_median": med, "gbs_moved": 16.0 * k / (med * 1e-3) / 1e9,
                     "frac_hbm_moved": 16.0 * k / (med * 1e-3) / 1e9 / hbm,
                     "frac_hbm_algorithmic": 12.0 * k / (med * 1e-3) / 1e9 / hbm}
    # z kept by the first pass of a step: that pass writes 4 more bytes per entry, the other three
    # passes stream 12 bytes per entry
    z = torch.empty_like(S)
    med, _ = time_call(lambda: B.szo_perturb_keep_z(S, S, idx, 0, 1234, 1, 1e-3, z), reps, flush=True)
    res["keep_z_first_pass_cold"] = {"ms_median": med, "frac_hbm_moved": 20.0 * k / (med * 1e-3) / 1e9 / hbm,
                                     "frac_hbm_algorithmic": 12.0 * k / (med * 1e-3) / 1e9 / hbm}
    med, _ = time_call(lambda: B.szo_perturb_kept_z(S, S, z, -2e-3), reps, flush=True)
    res["kept_z_pass_cold"] = {"ms_median": med, "gbs": 12.0 * k / (med * 1e-3) / 1e9,
                               "frac_hbm_algorithmic": 12.0 * k / (med * 1e-3) / 1e9 / hbm}
    line = {"case": "sparse_perturb", "k": k, "bytes_per_entry_algorithmic": 12, "bytes_per_entry_moved_regenerating": 16,
            "peaks": src, **res}
    print(json.dumps(line), flush=True)
    return line


def cold_case(N, K, G, reps):
    """The two one-off steps: szo_quantize of one [N, K] fp32 weight and szo_select_mask of its
    N*K scores (k = 0.1 %).  Reported, not part of the step."""
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    W = torch.randn(N, K, generator=g, device="cuda") * 0.02
    hbm, _, src = peaks()
    med, _ = time_call(lambda: B.szo_quantize(W, G, "bf16"), reps)
    q_bytes = 4.0 * N * K + 0.5 * N * K + 4.0 * N * K / G
    scores = (W * W).reshape(-1).contiguous()
    k = N * K // 1000
    med_s, _ = time_call(lambda: B.szo_select_mask(scores, k), reps)
    line = {"case": "cold", "N": N, "K": K, "G": G, "peaks": src,
            "quantize": {"ms_median": med, "gbs": q_bytes / (med * 1e-3) / 1e9, "frac_hbm": q_bytes / (med * 1e-3) / 1e9 / hbm},
            "select_mask": {"ms_median": med_s, "n": N * K, "k": k,
                            "gbs_one_pass_equivalent": 4.0 * N * K / (med_s * 1e-3) / 1e9}}
    print(json.dumps(line), flush=True)
    return line


def attention_case(Bn, S, H, Hkv, hd, reps):
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    q = torch.randn(Bn * S, H * hd, generator=g, device="cuda").to(torch.bfloat16)
    k = torch.randn(Bn * S, Hkv * hd, generator=g, device="cuda").to(torch.bfloat16)
    v = torch.randn(Bn * S, Hkv * hd, generator=g, device="cuda").to(torch.bfloat16)
    med, best = time_call(lambda: B.szo_attention(q, k, v, Bn, S, H, Hkv, hd), reps)
    flops = 4.0 * Bn * H * S * S * hd / 2          # causal
    print(json.dumps({"case": "attention", "B": Bn, "S": S, "H": H, "Hkv": Hkv, "hd": hd, "ms_median": med,
                      "tflops_causal": flops / (med * 1e-3) / 1e12}), flush=True)


def attention_paired_case(Bn, S, H, Hkv, hd, reps):
    """Causal attention of both forwards of a step as centre and half-difference rows (szo_attention_paired)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    M = Bn * S
    row0 = B.paired_row0(M)

    def rows(width):
        t = torch.randn(row0 + M, width, generator=g, device="cuda")
        t[row0:] *= 1e-3
        return t.to(torch.bfloat16)

    q, k, v = rows(H * hd), rows(Hkv * hd), rows(Hkv * hd)
    med, best = time_call(lambda: B.szo_attention_paired(q, k, v, row0, Bn, S, H, Hkv, hd), reps)
    flops = 4 * 4.0 * Bn * H * S * S * hd / 2          # causal; four products per term
    print(json.dumps({"case": "attention_paired", "B": Bn, "S": S, "H": H, "Hkv": Hkv, "hd": hd, "ms_median": med,
                      "ms_min": best, "tflops_causal": flops / (med * 1e-3) / 1e12}), flush=True)


def paired_case(M, N, K, G, rho, reps):
    """One linear in the paired form (szo_linear_fwd_paired): M centre rows and M half-difference rows
    in one call: weight pass, SparseAdd scatter, one tensor-core launch over both kinds of rows, the
    sparse product pass.  Timed whole, L2 flushed between repetitions."""
    g = torch.Generator(device="cuda")
    g.manual_seed(0)
    codes = torch.randint(0, 256, (N, K // 2), generator=g, device="cuda", dtype=torch.uint8)
    sc = (0.004 + 0.002 * torch.rand(N, K // G, generator=g, device="cuda")).to(torch.bfloat16)
    ze = (-7.5 * sc.float()).to(torch.bfloat16)
    nnz = int(rho * N * K)
    idx = torch.from_numpy(wl.sorted_random_indices(N * K, nnz, seed=1)).cuda()
    plan = B.Linear(N, K, G, codes, sc, ze, "bf16", idx)
    S = torch.randn(nnz, generator=g, device="cuda") * 0.02
    z = torch.randn(nnz, generator=g, device="cuda")
    row0 = B.paired_row0(M)
    x = torch.randn(row0 + M, K, generator=g, device="cuda").to(torch.bfloat16)
    x[row0:] *= 1e-3
    ms, ms_min = time_call(lambda: plan.fwd_paired(x, M, S, z, 1e-3), reps)
    flops = 2 * 2 * M * N * K
    print(json.dumps({"case": "paired_linear", "M": M, "N": N, "K": K, "G": G, "rho": rho, "nnz": nnz, "ms": ms,
                      "ms_min": ms_min, "tflops_both_row_kinds": flops / ms / 1e9, "device_status": B.device_status()}))
    plan.close()


def step_case(name, Bn, S, loss, steps, eps, lr, profile_range=False, form="paired"):
    """A full ZO step of a whole decoder shape (random-init weights in device memory), timed like
    bench.py: CUDA events around `steps` back-to-back steps after three warm-up steps; the weights
    streamed per forward exceed L2."""
    shape = wl.MODEL_SHAPES[name]
    tensors, S_all = wl.device_decoder_tensors(shape, seed=0)
    loss_kind = B.LOSS_CLS2 if loss == "cls2" else B.LOSS_LM
    model = B.Model(shape, wl.linear_names(shape), tensors, S_all, act_dtype=B.SZO_BF16,
                    linear_mode=B.MODE_PAIRED if form == "paired" else B.MODE_SPARSE_ADD, loss_kind=loss_kind,
                    max_batch=Bn, max_seq=S)
    n = 3 + steps
    toks = [torch.from_numpy(wl.token_batch(shape["vocab"], Bn, S, 0, wl.PURPOSE_TRAIN_BATCH, i)).cuda() for i in range(n)]
    labs = [torch.from_numpy(wl.binary_labels(Bn, 0, i)).cuda() for i in range(n)] if loss == "cls2" else [None] * n
    cand = torch.tensor([9906, 13], dtype=torch.int32).cuda() if loss == "cls2" else None
    for i in range(3):
        model.zo_step(toks[i], 1234, i, eps, lr, labs[i], cand)
    torch.cuda.synchronize()
    model.enable_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if profile_range:       # for ncu --profile-from-start off: exactly the timed steps are listed
        torch.cuda.profiler.start()
    e0.record()
    for i in range(3, n):
        model.zo_step(toks[i], 1234, i, eps, lr, labs[i], cand)
    e1.record()
    torch.cuda.synchronize()
    if profile_range:
        torch.cuda.profiler.stop()
    ms = e0.elapsed_time(e1) / steps
    lin_ms, lin_launches = model.linear_time()
    model.enable_timing(False)
    M = Bn * S
    flops = 2 * steps * shape["n_layers"] * sum(2 * M * nn * kk for nn, kk in
                                                 (wl.linear_shape(shape, nm) for nm in wl.linear_names(shape)))
    sus = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))).get("bf16_tflops_sustained") \
        if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else 1400.0
    last = model._scalars[:3].cpu().numpy()
    ach = flops / (lin_ms * 1e-3) / 1e12
    print(json.dumps({"case": "step", "model": name, "form": form, "batch": Bn, "seq": S, "loss": loss, "k": int(model.k_total),
                      "ms_per_step": ms, "steps_per_s": 1e3 / ms, "tokens_per_s": 1e3 / ms * M,
                      "linear_ms_per_step": lin_ms / steps, "linear_launches_per_step": lin_launches / steps,
                      "linear_tflops": ach, "frac_of_sustained_peak": ach / sus,
                      "roofline_ms_per_step": flops / steps / sus / 1e9, "device_status": B.device_status(),
                      "f_plus": float(last[0]), "f_minus": float(last[1]), "g": float(last[2])}))
    model.close()


def decode_case(name, Bn, prompt, gen):
    """Token generation with a KV cache (szo_model_decode_step): a prompt of `prompt` tokens in one
    call, then `gen` calls of one token per sequence, timed with CUDA events over the generation loop.
    Every step streams all linear weights once, so the roofline is the weight bytes over the HBM
    bandwidth."""
    shape = wl.MODEL_SHAPES[name]
    tensors, S_all = wl.device_decoder_tensors(shape, seed=0)
    model = B.Model(shape, wl.linear_names(shape), tensors, S_all, act_dtype=B.SZO_BF16, linear_mode=B.MODE_SPARSE_ADD,
                    loss_kind=B.LOSS_LM, max_batch=Bn, max_seq=prompt + gen)
    model.enable_decode()
    g = torch.Generator(device="cuda")
    g.manual_seed(1)
    toks = torch.randint(0, shape["vocab"], (Bn, prompt), generator=g, device="cuda", dtype=torch.int32)
    logits = torch.empty((Bn, shape["vocab"]), dtype=torch.float32, device="cuda")
    nxt = torch.empty((Bn, 1), dtype=torch.int32, device="cuda")

    def run():
        model.decode_step(toks, 0, logits)
        for i in range(gen):
            nxt.copy_(torch.argmax(logits, dim=1, keepdim=True))          # greedy choice, on the device
            model.decode_step(nxt, prompt + i, logits)

    stream = torch.cuda.Stream()          # a token step is replayed as a CUDA graph on a non-default stream
    with torch.cuda.stream(stream):
        run()
        stream.synchronize()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record(stream)
        model.decode_step(toks, 0, logits)
        e1.record(stream)
        for i in range(gen):
            nxt.copy_(torch.argmax(logits, dim=1, keepdim=True))
            model.decode_step(nxt, prompt + i, logits)
        e2.record(stream)
        stream.synchronize()
    ms_gen = e1.elapsed_time(e2)
    weight_bytes = 0
    for nm in wl.linear_names(shape):
        N, K = wl.linear_shape(shape, nm)
        G = shape["group"]
        weight_bytes += (N * K // 2 + 4 * N * K // G) if G > 0 else ((N * K // 2 + 32 * N) if G < 0 else 2 * N * K)
    weight_bytes = weight_bytes * shape["n_layers"] + 2 * shape["vocab"] * shape["d_model"]
    hbm = peaks()[0]
    per_step_ms = ms_gen / gen
    print(json.dumps({"case": "decode", "model": name, "batch": Bn, "prompt": prompt, "generated": gen,
                      "prompt_ms": e0.elapsed_time(e1), "ms_per_token_step": per_step_ms,
                      "tokens_per_s": Bn * gen / ms_gen * 1e3, "weight_bytes_per_step": weight_bytes,
                      "roofline_ms_per_step": weight_bytes / hbm / 1e6, "frac_of_hbm": weight_bytes / hbm / 1e6 / per_step_ms,
                      "device_status": B.device_status()}))
    model.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["linear", "paired", "steady", "sparse", "sweep", "attention", "step", "decode"])
    ap.add_argument("--prompt", type=int, default=16)
    ap.add_argument("--gen", type=int, default=128)
    ap.add_argument("--model", default="mistral_7b", choices=sorted(wl.MODEL_SHAPES))
    ap.add_argument("--batch", type=int, default=8)
    ap.add_argument("--seq", type=int, default=512)
    ap.add_argument("--loss", default="lm", choices=["lm", "cls2"])
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--eps", type=float, default=1e-3)
    ap.add_argument("--lr", type=float, default=1e-6)
    ap.add_argument("--profile-range", action="store_true",
                    help="step: bracket the timed steps with cudaProfilerStart/Stop")
    ap.add_argument("--M", type=int, default=8192)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--G", type=int, default=128, help="group size; 0: dense bf16 weight; -1: non-uniform 4-bit (table) format")
    ap.add_argument("--rho", type=float, default=1e-3)
    ap.add_argument("--mode", default="sparse_add")
    ap.add_argument("--form", default="paired", choices=["paired", "sparse_add"],
                    help="step: both forwards in one paired pass (centre / half-difference), or two bf16 forwards")
    ap.add_argument("--k", type=int, default=6_476_005)
    ap.add_argument("--reps", type=int, default=20)
    a = ap.parse_args()
    B.lib()
    if a.what == "linear":
        linear_case(a.M, a.N, a.K, a.G, a.mode, a.rho, a.reps)
    elif a.what == "decode":
        decode_case(a.model, a.batch, a.prompt, a.gen)
    elif a.what == "paired":
        paired_case(a.M, a.N, a.K, a.G, a.rho, a.reps)
    elif a.what == "steady":
        steady_case(a.M, a.N, a.K, a.G, a.mode, a.rho, a.reps)
    elif a.what == "sparse":
        sparse_case(a.k, a.reps)
    elif a.what == "step":
        step_case(a.model, a.batch, a.seq, a.loss, a.steps, a.eps, a.lr, a.profile_range, a.form)
    elif a.what == "attention":
        attention_case(16, 256, 32, 32, 128, a.reps)
        attention_case(8, 512, 32, 8, 128, a.reps)
        attention_paired_case(16, 256, 32, 32, 128, a.reps)
        attention_paired_case(8, 512, 32, 8, 128, a.reps)
    else:
        for M in (16, 256, 8192):
            for mode in ("sparse_add", "spmm"):
                linear_case(M, 4096, 4096, 128, mode, 1e-3, a.reps)
        for N, K in ((4096, 4096), (11008, 4096), (4096, 11008)):
            linear_case(4096, N, K, 128, "sparse_add", 1e-3, a.reps)
        for k in (100_000, 1_000_000, 6_476_005, 12_582_912, 100_000_000):
            sparse_case(k, a.reps)
        cold_case(11008, 4096, 128, a.reps)
        attention_case(16, 256, 32, 32, 128, a.reps)
        for N, K in ((4096, 4096), (11008, 4096), (4096, 11008)):       # few tokens, steady state
            for M, mode in ((1, "auto"), (8, "auto"), (16, "auto"), (16, "sparse_add"), (64, "auto")):
                steady_case(M, N, K, 128, mode, 1e-3, 10)


if __name__ == "__main__":
    main()
