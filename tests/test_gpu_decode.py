"""GPU parity of token generation with a KV cache (szo_model_decode_step) against the oracle's
incremental decode, which tests/test_oracle_model_pins.py pins to the full forward."""
import numpy as np
import pytest
import torch

from oracle import model_oracle as mo
from tests.fixtures import DecoderFixture

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2406_02913_b200 import binding
    binding.lib()
    return binding


@pytest.mark.parametrize("name", ["tiny", "tiny_gqa", "tiny_opt", "tiny_lut"])
@pytest.mark.parametrize("act", ["f32", "bf16"])
def test_decode_steps_match_the_oracle(B, name, act):
    """A prompt of 5 tokens in one call, a chunk of 3, then single tokens, for 3 sequences: the logits of
    every stop against the oracle (fp32 validation path: 1e-4 of the largest logit; bf16 path with the
    few-token kernels: 2e-2), the sparse values perturbed as inside a ZO step."""
    fx = DecoderFixture(name, seed=6, mask="random", B=3, S=32)
    om = fx.oracle_model()
    S_np = om.S + np.float32(1e-3)                              # any values: the sparse term must be live
    toks = fx.batch(0)[:, :24]
    lin_W = om.lin_W(S_np)
    cache = mo.KVCache(om.cfg.n_layers)
    a, md = (B.SZO_F32, B.MODE_FP32_VALIDATE) if act == "f32" else (B.SZO_BF16, B.MODE_SPARSE_ADD)
    t = fx.gpu_tensors(torch, None)
    S = torch.from_numpy(S_np.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=a, linear_mode=md, max_batch=fx.B, max_seq=fx.S)
    m.enable_decode()
    tol = 1e-4 if act == "f32" else 2e-2
    at = 0
    for T in (5, 3, 1, 1, 1, 1):
        ref = mo.decode_step(om.cfg, om.params, lin_W, toks[:, at:at + T], cache).numpy()
        got = m.decode_step(torch.from_numpy(np.ascontiguousarray(toks[:, at:at + T])).cuda(), at).cpu().numpy()
        at += T
        assert np.max(np.abs(got - ref)) <= tol * np.max(np.abs(ref)), (name, act, at)
        if act == "f32":
            assert np.array_equal(np.argmax(got, axis=1), np.argmax(ref, axis=1))
    assert B.device_status() == 0
    # a fresh prompt after the old one: the cache is simply overwritten from position 0
    cache2 = mo.KVCache(om.cfg.n_layers)
    ref = mo.decode_step(om.cfg, om.params, lin_W, toks[:, 4:8], cache2).numpy()
    got = m.decode_step(torch.from_numpy(np.ascontiguousarray(toks[:, 4:8])).cuda(), 0).cpu().numpy()
    assert np.max(np.abs(got - ref)) <= tol * np.max(np.abs(ref))
    # a prompt of more than 16 tokens (rotation, cache append and attention as separate launches), then
    # one token on top of it (the fused launch reading that cache)
    cache3 = mo.KVCache(om.cfg.n_layers)
    at = 0
    for T in (20, 1):
        ref = mo.decode_step(om.cfg, om.params, lin_W, toks[:, at:at + T], cache3).numpy()
        got = m.decode_step(torch.from_numpy(np.ascontiguousarray(toks[:, at:at + T])).cuda(), at).cpu().numpy()
        at += T
        assert np.max(np.abs(got - ref)) <= tol * np.max(np.abs(ref)), (name, act, "long prompt", T)
    assert B.device_status() == 0
    m.close()


@pytest.mark.parametrize("name", ["small_gqa", "small_gqa_lut"])
def test_token_steps_of_a_wider_grouped_query_decoder(B, name):
    """Two layers of width 1024 with 16 query and 4 key/value heads (the q/k/v launch of the 16-row-group kernel
    holds a 1024-row and two 256-row matrices; K = 1024 and 2816: 8 and 22 column steps for seven warps), uniform
    int4 and table-coded weights: a prompt of 3, single tokens and a pair of tokens, for two sequences (cluster
    kernel at 6 rows, the other kernel at 2) and for one, against the oracle's incremental decode."""
    fx = DecoderFixture(name, seed=12, mask="random", B=2, S=16)
    om = fx.oracle_model()
    S_np = om.S + np.float32(1e-3)
    lin_W = om.lin_W(S_np)
    toks = fx.batch(0)[:, :8]
    t = fx.gpu_tensors(torch, None)
    S = torch.from_numpy(S_np.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=B.SZO_BF16, linear_mode=B.MODE_SPARSE_ADD, max_batch=fx.B, max_seq=fx.S)
    m.enable_decode()
    for nseq in (2, 1):
        cache = mo.KVCache(om.cfg.n_layers)
        at = 0
        for T in (3, 1, 1, 2):
            tk = np.ascontiguousarray(toks[:nseq, at:at + T])
            ref = mo.decode_step(om.cfg, om.params, lin_W, tk, cache).numpy()
            got = m.decode_step(torch.from_numpy(tk).cuda(), at).cpu().numpy()
            at += T
            assert np.max(np.abs(got - ref)) <= 2e-2 * np.max(np.abs(ref)), (name, nseq, at)
    assert B.device_status() == 0
    m.close()


def test_decode_argument_errors(B):
    fx = DecoderFixture("tiny", seed=6, mask="random", B=2, S=16, n_layers=1)
    t = fx.gpu_tensors(torch, None)
    S = torch.from_numpy(fx.S_init.copy()).cuda()
    m = B.Model(fx.shape, fx.names, t, S, act_dtype=B.SZO_BF16, linear_mode=B.MODE_SPARSE_ADD, max_batch=fx.B, max_seq=fx.S)
    toks = torch.zeros((2, 4), dtype=torch.int32, device="cuda")
    with pytest.raises(B.SzoError):                      # no cache yet
        m.decode_step(toks, 0)
    m.enable_decode()
    with pytest.raises(B.SzoError) as ei:                # beyond max_seq
        m.decode_step(toks, 14)
    assert ei.value.name == "SZO_ERR_SHAPE"
    m.decode_step(toks, 12)
    m.close()


def test_graph_replay_of_token_steps_equals_the_launch_by_launch_form(B):
    """On a non-default stream a token step is captured once and replayed with the position read from
    device memory; the logits must be the bits of the launch-by-launch form (default stream), for a
    prompt, several single-token steps and a second prompt that reuses the captured graphs."""
    fx = DecoderFixture("tiny", seed=7, mask="random", B=2, S=32)
    t = fx.gpu_tensors(torch, None)
    toks = torch.from_numpy(np.ascontiguousarray(fx.batch(0)[:, :10])).cuda()
    outs = []
    for use_stream in (False, True):
        S = torch.from_numpy(fx.S_init.copy()).cuda()
        m = B.Model(fx.shape, fx.names, t, S, act_dtype=B.SZO_BF16, linear_mode=B.MODE_SPARSE_ADD, max_batch=fx.B, max_seq=fx.S)
        m.enable_decode()
        stream = torch.cuda.Stream() if use_stream else torch.cuda.current_stream()
        got = []
        with torch.cuda.stream(stream):
            for rep in range(2):
                got.append(m.decode_step(toks[:, :4].contiguous(), 0).clone())
                for i in range(4, 10):
                    got.append(m.decode_step(toks[:, i:i + 1].contiguous(), i).clone())
            stream.synchronize()
        outs.append(torch.stack(got).cpu())
        assert B.device_status() == 0
        m.close()
    assert torch.equal(outs[0], outs[1])
    assert torch.equal(outs[0][:7], outs[0][7:])             # the second pass over the same prompt repeats the first


_SWITCH_SCRIPT = r"""
import sys, numpy as np, torch
from paper_2406_02913_b200 import binding as B, workloads as wl
shape = dict(wl.MODEL_SHAPES["llama2_7b"], n_layers=2)
tensors, S_all = wl.device_decoder_tensors(shape, seed=3)
m = B.Model(shape, wl.linear_names(shape), tensors, S_all, act_dtype=B.SZO_BF16, linear_mode=B.MODE_SPARSE_ADD,
            loss_kind=B.LOSS_LM, max_batch=2, max_seq=16)
m.enable_decode()
g = torch.Generator(device="cuda"); g.manual_seed(5)
toks = torch.randint(0, shape["vocab"], (2, 8), generator=g, device="cuda", dtype=torch.int32)
outs = [m.decode_step(toks[:, :3].contiguous(), 0).clone()]
for i in range(3, 8):
    outs.append(m.decode_step(toks[:, i:i + 1].contiguous(), i).clone())
assert B.device_status() == 0
np.save(sys.argv[1], torch.stack(outs).cpu().numpy())
"""


def test_switches_of_the_token_step_leave_the_bits_alone(tmp_path):
    """The token step at the Llama-2-7B width (two layers, two sequences: the 16-row-group kernel with the norms
    inside the projections, launched as a chain) against the same step with the norms in a kernel of their own
    and with ordinary launches: the fused norm repeats the separate kernel's arithmetic and reduction tree, and a
    chained launch changes when a kernel starts, not what it computes, so the logits must be the same bits.  The
    switches are read once per process: one child process per setting."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = {}
    for name, extra in (("default", {}), ("separate_norm", {"SZO_DECODE_FUSED_NORM": "0"}), ("no_chain", {"SZO_DECODE_CHAIN": "0"})):
        out = str(tmp_path / (name + ".npy"))
        r = subprocess.run([sys.executable, "-c", _SWITCH_SCRIPT, out], cwd=root, env=dict(os.environ, **extra),
                           capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, name + ": " + r.stdout[-2000:] + r.stderr[-2000:]
        res[name] = np.load(out)
    assert np.isfinite(res["default"]).all()
    assert np.array_equal(res["default"], res["separate_norm"])
    assert np.array_equal(res["default"], res["no_chain"])
