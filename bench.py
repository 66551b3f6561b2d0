#!/usr/bin/env python
"""Benchmark: sensitive-sparse ZO-SGD steps per second on a Llama-2-7B-shaped 4-bit decoder.

One step = draw z, both perturbed losses f+ and f- on the same batch, projected gradient, update of
the k sensitive values, all through the C ABI (szo_model_zo_step).  Prints ONE JSON line (rank 0).

    python bench.py --gpus 1 --steps 5 --warmup 3
    python bench.py --gpus 4                  # starts 4 processes itself (or run it under torchrun)
    python bench.py --impl reference          # the CPU oracle on a bounded sample of the same work

--mode paired (default) evaluates f+ and f- in one pass that carries centre and half-difference of
every activation: the form whose projected gradient is tested against the oracle; --mode sparse_add
runs two bf16 forwards (faster, but their loss difference is lost in bf16 rounding).

Multi-GPU: the step holds the whole model on one GPU.  --parallel replicas (default) runs N
independent replicas and reports their aggregate; --parallel dp runs N data-parallel replicas of one
run (same weights and z, own batches, one 24-byte all-reduce of loss sums per step).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "llama2_7b"
BATCH, SEQ = 16, 256
EPS, LR, SEED = 1e-3, 1e-6, 1234
# ncu summary that holds the DRAM traffic of one launch of the dominant kernel, and the sources it was taken from
TRAFFIC_PROFILE = os.path.join(ROOT, "profiles", "szo_linear_tc2_kernel_paired_gate_up_M8192.md")
KERNEL_SOURCES = [os.path.join(ROOT, "paper_2406_02913_b200", "csrc", f) for f in ("gemm_tc2.cu", "tc_common.cuh")]
ORACLE_TOKENS_SAMPLE, ORACLE_K_SAMPLE = 4096, 6_476_005


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        h.update(open(f, "rb").read())
    return h.hexdigest()[:16]


def profiled_traffic():
    """(bytes per launch, note) read from the ncu summary; None once the kernel sources differ from the
    ones the counters were taken from."""
    if not os.path.exists(TRAFFIC_PROFILE):
        return None, "no ncu summary for this kernel"
    text = open(TRAFFIC_PROFILE).read()
    m_hash = re.search(r"kernel_source_sha256_16:\s*([0-9a-f]{16})", text)
    m_bytes = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", text)
    if not (m_hash and m_bytes):
        return None, "ncu summary lacks the traffic record"
    if m_hash.group(1) != kernel_source_hash():
        return None, "kernel sources changed since the counters in " + os.path.relpath(TRAFFIC_PROFILE, ROOT) + " were taken"
    return float(m_bytes.group(1)), os.path.relpath(TRAFFIC_PROFILE, ROOT)


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop = index, [], threading.Event()
        self._t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                parts = [p.strip() for p in out.strip().split(",")]
                if len(parts) >= 6:
                    self.rows.append(parts)
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
        sm = [float(r[0]) for r in self.rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows)}


def linear_flops_per_forward(shape, M):
    from paper_2406_02913_b200 import workloads as wl
    per_layer = sum(2 * M * n * k for n, k in (wl.linear_shape(shape, nm) for nm in wl.linear_names(shape)))
    return per_layer * shape["n_layers"]


# ------------------------------------------------------------------------------------ oracle leg
def oracle_sample(shape, tokens_sample=ORACLE_TOKENS_SAMPLE, k_sample=ORACLE_K_SAMPLE):
    """Times the CPU oracle, as it stands, on a bounded sample of the step: the seven linears of one
    decoder layer (dequantize, add the sparse values, fp64 product) for `tokens_sample` tokens, and
    one sparse perturb pass over `k_sample` entries.  Extrapolated to a whole step by the layer
    count, the token count and the total k."""
    import numpy as np
    from oracle import szo_oracle as so
    from paper_2406_02913_b200 import workloads as wl

    G, fmt = shape["group"], shape["sz_fmt"]
    t_lin, t_prep = 0.0, 0.0
    for j, nm in enumerate(wl.linear_names(shape)):
        N, K = wl.linear_shape(shape, nm)
        codes = wl.random_codes(N, K, seed=1, i=j)
        sc = (0.004 + 0.002 * wl.rng(1, wl.PURPOSE_WEIGHTS, 50 + j).random((N, K // G))).astype(np.float32)
        sb, scv = so.round_to_16(sc, fmt)
        zb, _ = so.round_to_16(-7.5 * scv, fmt)
        idx = wl.sorted_random_indices(N * K, int(shape["rho"] * N * K), seed=1, i=j)
        S = wl.rng(1, wl.PURPOSE_WEIGHTS, 80 + j).normal(0, 0.02, idx.size).astype(np.float32)
        x = wl.activation(tokens_sample, K, seed=1, i=j)
        t0 = time.perf_counter()
        deq = so.dequantize(codes, sb, zb, G, fmt)
        t1 = time.perf_counter()
        so.effective_weight(deq, idx, S)
        t2 = time.perf_counter()
        so.linear_fwd(x, deq, idx, S)
        t3 = time.perf_counter()
        t_prep += (t1 - t0) + (t2 - t1)
        t_lin += max((t3 - t2) - (t2 - t1), 0.0)
    gidx = wl.sorted_random_indices(6_476_005_376, k_sample, seed=2)
    Sv = np.zeros(k_sample, np.float32)
    t0 = time.perf_counter()
    so.perturb(Sv, gidx, SEED, 0, np.float32(EPS))
    t_pert = time.perf_counter() - t0
    M = BATCH * SEQ
    d_lin = sum(n * k for n, k in (wl.linear_shape(shape, nm) for nm in wl.linear_names(shape))) * shape["n_layers"]
    k_total = int(shape["rho"] * d_lin)
    # the weight preparation (dequantize, add the sparse values) does not depend on the token count;
    # the fp64 product does
    step_s = 2 * shape["n_layers"] * (t_prep + t_lin * (M / tokens_sample)) + 4 * t_pert * (k_total / k_sample)
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    sample = (f"extrapolated from one decoder layer's 7 linears (weight preparation {t_prep:.2f} s + fp64 product at "
              f"{tokens_sample} tokens {t_lin:.2f} s) and one perturb pass over {k_sample} entries ({t_pert:.2f} s): "
              f"x{shape['n_layers']} layers x2 forwards, product x{M // tokens_sample} token blocks, + 4 passes over "
              f"k={k_total}; attention and norms not included")
    return dict(value=1.0 / step_s, unit="steps/s", cores=cores, kind="oracle", sample=sample), step_s


def oracle_small_configs():
    """The oracle on the two small workloads, in full (no extrapolation): the tiny decoder's 10 ZO steps
    and one 4096 x 4096 int4 linear at 16 and 256 tokens."""
    import numpy as np
    from oracle import model_oracle as mo
    from oracle import szo_oracle as so
    from paper_2406_02913_b200 import workloads as wl
    from tests.fixtures import DecoderFixture

    fx = DecoderFixture("tiny", seed=0, mask="random", B=4, S=64)
    om = fx.oracle_model()
    t0 = time.perf_counter()
    for step in range(10):
        mo.zo_step(om, fx.batch(step), SEED, step, 1e-3, 1e-5)
    t_tiny = time.perf_counter() - t0
    N = K = 4096
    codes = wl.random_codes(N, K, seed=3)
    sc = (0.004 + 0.002 * wl.rng(3, wl.PURPOSE_WEIGHTS, 1).random((N, K // 128))).astype(np.float32)
    sb, scv = so.round_to_16(sc, "bf16")
    zb, _ = so.round_to_16(-7.5 * scv, "bf16")
    idx = wl.sorted_random_indices(N * K, 16777, seed=3)
    S = wl.rng(3, wl.PURPOSE_WEIGHTS, 2).normal(0, 0.02, idx.size).astype(np.float32)
    out = {"tiny_decoder_10_steps_s": round(t_tiny, 3)}
    deq = so.dequantize(codes, sb, zb, 128, "bf16")
    for M in (16, 256):
        x = wl.activation(M, K, seed=3, i=M)
        t0 = time.perf_counter()
        so.linear_fwd(x, deq, idx, so.perturb(S, idx, SEED, 0, np.float32(EPS)))
        out[f"linear_4096x4096_M{M}_perturbed_forward_s"] = round(time.perf_counter() - t0, 3)
    return out


def run_reference(args):
    from paper_2406_02913_b200 import workloads as wl
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shape = wl.MODEL_SHAPES[WORKLOAD]
    vals = []
    for i in range(args.warmup + args.steps):
        cb, step_s = oracle_sample(shape)
        if i >= args.warmup:
            vals.append(step_s)
    ms = 1e3 * sum(vals) / len(vals)
    value = 1e3 / ms
    cb["value"] = value
    cb["measured_repeats"] = len(vals)
    cb["note"] = ("each 'step' of this arm is one timing of the bounded sample, extrapolated to a whole step; "
                  "ms_per_step is that extrapolation, not elapsed time")
    line = {"impl": "reference", "metric": "zo_steps_per_s", "value": value, "unit": "steps/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(shape, "n/a", "n/a"), "cpu_baseline": cb,
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def workload_config(shape, mode, parallel):
    return {"workload": "llama2_7b-shaped decoder, int4 group-128 + 0.1% fp32 sparse, full ZO step",
            "batch": BATCH, "seq_len": SEQ, "tokens_per_step": BATCH * SEQ, "n_layers": shape["n_layers"],
            "d_model": shape["d_model"], "d_ff": shape["d_ff"], "loss": "last-token 2-candidate CE",
            "eps": EPS, "lr": LR, "step_form": mode,
            "l2": "inputs larger than L2 (3.4 GB of weights streamed per step)", "parallelism": parallel}


# ------------------------------------------------------------------------------------ sparse passes
def sparse_pass_roofline(B, torch, k, peaks, launches=100):
    """The sparse perturb / update passes at the workload's k, each as `launches` back-to-back launches
    inside one CUDA graph (a single launch is shorter than the gap between two host launches), timed
    with CUDA events; 12 algorithmic bytes per entry (4 index + 4 read + 4 write)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    # consecutive launches work on different buffer sets, 6 sets of 52-78 MB: more than the 126 MB L2,
    # so that every launch streams its entries from HBM
    n_sets = 6
    idx = [torch.sort(torch.randint(0, 6_476_005_376, (k,), generator=g, device="cuda", dtype=torch.int64)).values.contiguous()
           for _ in range(n_sets)]
    S = [(torch.randn(k, generator=g, device="cuda") * 0.02).contiguous() for _ in range(n_sets)]
    z = [torch.empty(k, device="cuda") for _ in range(n_sets)]
    out = {"k": k, "algorithmic_bytes_per_entry": 12, "launches_per_graph": launches, "peak_gbs": peaks["hbm_gbs"],
           "peak_source": peaks["source"] + " (copy bandwidth)",
           "l2": f"{n_sets} buffer sets in rotation ({n_sets * 12 * k / 1e6:.0f} MB), larger than L2"}
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for i in range(n_sets):                                            # warm-up, and z for the kept passes
            B.szo_perturb_keep_z(S[i], S[i], idx[i], 0, SEED, 0, 1e-3, z[i])
            B.szo_perturb_kept_z(S[i], S[i], z[i], -1e-3)
        stream.synchronize()
        for name, call in (("regenerating", lambda i: B.szo_perturb(S[i], S[i], idx[i], 0, SEED, 0, 1e-3)),
                           ("kept_z", lambda i: B.szo_perturb_kept_z(S[i], S[i], z[i], 1e-3)),
                           ("three_passes_in_one", lambda i: B.szo_perturb3_keep_z(S[i], S[i], idx[i], 0, SEED, 0, 1e-3, z[i]))):
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for j in range(launches):
                    call(j % n_sets)
            graph.replay()
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            us = 1e3 * e0.elapsed_time(e1) / launches
            passes = 3 if name == "three_passes_in_one" else 1          # logical passes of 12 algorithmic bytes per entry
            gbs = passes * 12.0 * k / us / 1e3
            out[name] = {"us_per_launch": us, "achieved_gbs": gbs, "frac": gbs / peaks["hbm_gbs"]}
    out["three_passes_in_one"]["note"] = ("+eps, -2 eps, +eps of one (seed, step) in one launch: 36 algorithmic bytes per entry, "
                                          "20 moved (index 8, S read and written, z written)")
    sep = out["regenerating"]["us_per_launch"] + 3 * out["kept_z"]["us_per_launch"]
    out["four_passes_one_launch_each"] = {"us": sep, "achieved_gbs": 4 * 12.0 * k / sep / 1e3,
                                          "frac": 4 * 12.0 * k / sep / 1e3 / peaks["hbm_gbs"]}
    # what the paired step launches: the three perturbation passes in one, then the update from the kept z
    four = out["three_passes_in_one"]["us_per_launch"] + out["kept_z"]["us_per_launch"]
    out["four_passes_of_a_step"] = {"us": four, "achieved_gbs": 4 * 12.0 * k / four / 1e3,
                                    "frac": 4 * 12.0 * k / four / 1e3 / peaks["hbm_gbs"],
                                    "launches": 2, "bytes_moved_per_entry": 32}
    return out


# ------------------------------------------------------------------------------------ token generation
def token_generation(B, torch, model, shape, peaks, prompt=16, gen=128):
    """Outside the timed steps, on the same model: a prompt of `prompt` tokens, then `gen` single-token steps of one
    sequence with a KV cache (szo_model_decode_step, replayed as a CUDA graph), timed with CUDA events; every step
    streams all weights once, so the roofline is the weight bytes over the HBM bandwidth."""
    from paper_2406_02913_b200 import workloads as wl
    model.enable_decode()
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    toks = torch.randint(0, shape["vocab"], (1, prompt), generator=g, device="cuda", dtype=torch.int32)
    logits = torch.empty((1, shape["vocab"]), dtype=torch.float32, device="cuda")
    nxt = torch.empty((1, 1), dtype=torch.int32, device="cuda")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        times = []
        for rep_i in range(2):                                              # the first pass captures the graphs
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            model.decode_step(toks, 0, logits)
            e0.record(stream)
            for i in range(gen):
                nxt.copy_(torch.argmax(logits, dim=1, keepdim=True))
                model.decode_step(nxt, prompt + i, logits)
            e1.record(stream)
            stream.synchronize()
            times.append(e0.elapsed_time(e1) / gen)
    weight_bytes = 0
    for nm in wl.linear_names(shape):
        N, K = wl.linear_shape(shape, nm)
        weight_bytes += N * K // 2 + 4 * N * K // shape["group"]
    weight_bytes = weight_bytes * shape["n_layers"] + 2 * shape["vocab"] * shape["d_model"]
    ms = times[-1]
    return {"batch": 1, "prompt": prompt, "generated": gen, "ms_per_token_step": ms, "tokens_per_s": 1e3 / ms,
            "weight_bytes_per_step": weight_bytes, "roofline_ms_per_step": weight_bytes / peaks["hbm_gbs"] / 1e6,
            "frac_of_hbm": weight_bytes / peaks["hbm_gbs"] / 1e6 / ms, "device_status": B.device_status()}


# ------------------------------------------------------------------------------------ GPU leg
def run_ours(args):
    import torch
    from paper_2406_02913_b200 import binding as B
    from paper_2406_02913_b200 import build as build_mod
    from paper_2406_02913_b200 import workloads as wl
    from paper_2406_02913_b200.replicas import Replicas

    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    rep = Replicas("nccl")
    world, rank, local = rep.world, rep.rank, rep.local_rank
    if rank == 0:
        build_mod.build()
    if rep.dist is not None:
        rep.dist.barrier()
    B.lib()

    dp = args.parallel == "dp" and world > 1
    shape = wl.MODEL_SHAPES[WORKLOAD]
    # data-parallel replicas hold the same weights, mask and S; independent replicas their own
    tensors, S_all = wl.device_decoder_tensors(shape, seed=0 if dp else rank)
    mode = {"paired": B.MODE_PAIRED, "sparse_add": B.MODE_SPARSE_ADD}[args.mode]
    model = B.Model(shape, wl.linear_names(shape), tensors, S_all, act_dtype=B.SZO_BF16,
                    linear_mode=mode, loss_kind=B.LOSS_CLS2, max_batch=BATCH, max_seq=SEQ)
    n_steps = args.warmup + args.steps
    toks_host = [torch.from_numpy(wl.token_batch(shape["vocab"], BATCH, SEQ, rank, wl.PURPOSE_TRAIN_BATCH, i)).pin_memory()
                 for i in range(n_steps)]
    labs_host = [torch.from_numpy(wl.binary_labels(BATCH, rank, i)).pin_memory() for i in range(n_steps)]
    cand_host = torch.tensor([9906, 13], dtype=torch.int32).pin_memory()
    toks_dev = [t.cuda() for t in toks_host]
    labs_dev = [t.cuda() for t in labs_host]
    cand_dev = cand_host.cuda()
    barrier, max_over_ranks = rep.barrier, rep.max_over_ranks
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")

    def step_dev(i):
        if dp:
            rep.data_parallel_step(lambda: model.zo_losses(toks_dev[i], SEED, i, EPS, labs_dev[i], cand_dev, sums),
                                   lambda s: model.zo_apply(EPS, LR, s))
        else:
            model.zo_step(toks_dev[i], SEED, i, EPS, LR, labs_dev[i], cand_dev)

    # ---- device-resident inputs (the headline value)
    for i in range(args.warmup):
        step_dev(i)
    barrier()
    model.enable_timing(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clk:
        if args.profile_range:
            torch.cuda.profiler.start()
        ev0.record()
        for i in range(args.warmup, n_steps):
            step_dev(i)
        ev1.record()
        barrier()
        if args.profile_range:
            torch.cuda.profiler.stop()
    ms_total = max_over_ranks(ev0.elapsed_time(ev1))
    lin_ms, lin_groups = model.linear_time()
    model.enable_timing(False)
    launches = model.last_launches() * args.steps
    last = model._scalars[:3].cpu().numpy()

    # ---- host-resident inputs through the same API (end to end)
    if not dp:
        for i in range(min(args.warmup, 1)):
            model.zo_step_host(toks_host[i], SEED, n_steps + i, EPS, LR, labs_host[i], cand_host)
        barrier()
        t0 = time.perf_counter()
        for i in range(args.warmup, n_steps):
            model.zo_step_host(toks_host[i], SEED, n_steps + i, EPS, LR, labs_host[i], cand_host)
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0))
    else:
        barrier()
        t0 = time.perf_counter()
        for i in range(args.warmup, n_steps):
            td, ld = toks_host[i].cuda(non_blocking=True), labs_host[i].cuda(non_blocking=True)
            cd = cand_host.cuda(non_blocking=True)
            out = rep.data_parallel_step(lambda: model.zo_losses(td, SEED, n_steps + i, EPS, ld, cd, sums),
                                         lambda s: model.zo_apply(EPS, LR, s))
            out.cpu()
        torch.cuda.synchronize()
        e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0))

    if rank != 0:
        rep.close()
        return 0
    peaks = measured_peaks()
    M = BATCH * SEQ
    ms_per_step = ms_total / args.steps
    steps_per_s = rep.whole_job_rate(1.0, ms_per_step)
    flops_fwd = linear_flops_per_forward(shape, M)
    lin_flops_total = 2 * flops_fwd * args.steps
    achieved = lin_flops_total / (lin_ms * 1e-3) / 1e12 if lin_ms > 0 else 0.0
    peak = peaks["bf16_tflops_sustained"]
    traffic, traffic_of = profiled_traffic()
    k_total = int(model.k_total)
    sparse = sparse_pass_roofline(B, torch, k_total, peaks)
    decode = token_generation(B, torch, model, shape, peaks)
    cb, _ = oracle_sample(shape)
    cb["other_configs"] = oracle_small_configs()
    per_group = {"paired": "weight pass (int4 -> bf16), SparseAdd scatter of S, ONE szo_linear_tc2_kernel launch over "
                           "centre and half-difference rows, pair_cross_kernel",
                 "sparse_add": "weight pass, two SparseAdd scatters, two szo_linear_tc2_kernel launches"}[args.mode]
    line = {
        "metric": "zo_steps_per_s", "value": steps_per_s, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": workload_config(shape, args.mode, args.parallel if world > 1 else "one GPU"),
        "tokens_per_s": steps_per_s * M,
        "e2e": {"value": rep.whole_job_rate(args.steps, e2e_ms), "unit": "steps/s",
                "h2d_bytes_per_step": BATCH * SEQ * 4 + BATCH * 4 + 8, "d2h_bytes_per_step": 24},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor", "kernel": "szo_linear_tc2_kernel", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak, "traffic": traffic, "traffic_of": traffic_of,
                     "peak_source": f"{peaks['source']} (sustained cuBLAS bf16)",
                     "timed": "CUDA events around every decoder-block linear GROUP inside the timed steps; a group is: " + per_group,
                     "linear_groups": int(lin_groups), "avg_group_ms": lin_ms / max(lin_groups, 1),
                     "linear_ms_per_step": lin_ms / args.steps,
                     "algorithmic_flops_per_step": 2 * flops_fwd},
        "roofline_sparse": sparse,
        "token_generation": decode,
        "cpu_baseline": cb,
        "clocks": clk.summary(),
        "last_step": {"f_plus": float(last[0]), "f_minus": float(last[1]), "g": float(last[2])},
    }
    print(json.dumps(line))
    rep.close()
    return 0


def spawn_ranks(args) -> int:
    """--gpus N without a launcher: start N processes of this script, one per GPU, with the rendezvous
    on 127.0.0.1, and pass rank 0's line through."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, WORLD_SIZE=str(args.gpus), RANK=str(r), LOCAL_RANK=str(r), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env,
                                      stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL, text=True))
    out, _ = procs[0].communicate()
    rc = procs[0].returncode
    for p in procs[1:]:
        rc = rc or p.wait()
    sys.stdout.write(out)
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="paired", choices=["paired", "sparse_add"],
                    help="paired: both forwards of a step in one pass as centre / half-difference (the default: "
                         "the form whose projected gradient meets the tested bound); sparse_add: two bf16 forwards")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "dp"],
                    help="with several GPUs: independent replicas, or data-parallel replicas of one run")
    ap.add_argument("--profile-range", action="store_true",
                    help="bracket the timed region with cudaProfilerStart/Stop (for ncu --profile-from-start off)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_ranks(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
