"""The N > 1 path of the benchmark on CPU: two gloo ranks run the replica plumbing (barrier,
max-over-ranks time, whole-job rate) that bench.py uses with NCCL on GPUs."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, time
sys.path.insert(0, %r)
from paper_2406_02913_b200.replicas import Replicas
rep = Replicas("gloo")
assert rep.world == 2 and rep.device.type == "cpu"
rep.barrier()
mine = 10.0 + 5.0 * rep.rank                     # rank 1 is the slow replica
slowest = rep.max_over_ranks(mine)
assert slowest == 15.0, slowest
rate = rep.whole_job_rate(3.0, slowest)          # 3 steps per rank in 15 ms -> 2 * 3 / 0.015 steps/s
assert abs(rate - 400.0) < 1e-9, rate
t0 = time.perf_counter()
if rep.rank == 0:
    time.sleep(0.3)                              # the barrier holds rank 1 until rank 0 arrives
rep.barrier()
waited = time.perf_counter() - t0
assert waited >= 0.25, waited
rep.close()
print("rank", rep.rank, "ok")
''' % ROOT


DP_WORKER = r'''
import os, sys
sys.path.insert(0, %r)
import numpy as np, torch
from oracle import model_oracle as mo, szo_oracle as so
from paper_2406_02913_b200.replicas import Replicas
from tests.fixtures import DecoderFixture
rep = Replicas("gloo")
fx = DecoderFixture("tiny", seed=0, mask="random", B=4, S=16, n_layers=1)
toks = fx.batch(0)
eps, lr, seed, step = np.float32(1e-3), np.float32(1e-3), 77, 5
# the whole batch on one replica: the oracle's step
full = fx.oracle_model()
fp, fm, g = mo.zo_step(full, toks, seed, step, eps, lr)
# this rank's half of the batch, same S, same (seed, step)
mine = fx.oracle_model()
half = toks[2 * rep.rank: 2 * rep.rank + 2]
count = half.shape[0] * (half.shape[1] - 1)
state = {}
def losses():
    S1 = so.perturb(mine.S, mine.gidx, seed, step, eps)
    lp = mine.loss(S1, half)
    S2 = so.perturb(S1, mine.gidx, seed, step, np.float32(-2.0) * eps)
    lm = mine.loss(S2, half)
    state["S"] = so.perturb(S2, mine.gidx, seed, step, eps)
    return torch.tensor([lp * count, lm * count, count], dtype=torch.float64)
def apply(sums):
    f_plus, f_minus = float(sums[0] / sums[2]), float(sums[1] / sums[2])
    gg = so.projected_gradient(f_plus, f_minus, eps)
    state["S"] = so.perturb(state["S"], mine.gidx, seed, step, so.zo_update_scale(f_plus, f_minus, eps, lr))
    return f_plus, f_minus, gg
f_plus, f_minus, gg = rep.data_parallel_step(losses, apply)
assert abs(f_plus - fp) <= 1e-13 * abs(fp) and abs(f_minus - fm) <= 1e-13 * abs(fm), (f_plus, fp)
assert abs(gg - g) <= 1e-9 * abs(g), (gg, g)
assert np.allclose(state["S"], full.S, rtol=0, atol=1e-9)
rep.close()
print("rank", rep.rank, "ok")
''' % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_agree_on_the_slowest_replica():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=120)
        except subprocess.TimeoutExpired:
            p.kill()
            out, _ = p.communicate()
        outs.append(out)
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, f"rank {rank} failed:\n{out}"
        assert f"rank {rank} ok" in out


def test_two_gloo_ranks_reproduce_the_full_batch_step_from_half_batches():
    """Data-parallel replicas: each of two ranks runs the ORACLE on half of the batch, the ranks add up
    (sum f+, sum f-, count), and every rank obtains the full-batch step of the oracle: same f+, f-, g
    (to fp64 rounding) and the same updated S."""
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, WORLD_SIZE="2", RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, "-c", DP_WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for rank, p in enumerate(procs):
        try:
            out, _ = p.communicate(timeout=300)
        except subprocess.TimeoutExpired:
            p.kill()
            out, _ = p.communicate()
        assert p.returncode == 0, f"rank {rank} failed:\n{out}"
        assert f"rank {rank} ok" in out


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2406_02913_b200.replicas import Replicas
    env = {k: os.environ.pop(k) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK") if k in os.environ}
    try:
        rep = Replicas("gloo")
        assert rep.world == 1 and rep.dist is None
        rep.barrier()
        assert rep.max_over_ranks(7.5) == 7.5
        assert rep.whole_job_rate(2.0, 100.0) == 20.0
    finally:
        os.environ.update(env)
