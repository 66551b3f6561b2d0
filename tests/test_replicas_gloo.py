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
