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
