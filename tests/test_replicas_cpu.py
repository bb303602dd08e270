"""N > 1 path of the benchmark on the CPU: two `gloo` ranks reduce replica timings (max) and work
(sum); `bench.py --impl reference` under two ranks prints one line from rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_16190_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert replicas.dist_env() == (rank, world, rank)
    replicas.barrier(world)
    ms_local = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    work_local = 100.0 * (rank + 1)
    rate, ms = replicas.job_throughput(work_local, ms_local, world, "cpu")
    out[rank] = (rate, ms, replicas.replica_seed(4, rank))
    dist.destroy_process_group()


def test_two_ranks_take_max_time_and_sum_work():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        rate, ms, seed = res[rank]
        assert ms == 15.0                               # the slowest replica
        assert abs(rate - 300.0 / 15e-3) < 1e-6         # all replicas' work over that time
        assert seed == 4 + 100 * rank                   # distinct synthetic layers


def test_single_rank_is_identity():
    assert replicas.job_throughput(50.0, 5.0, 1, "cpu") == (50.0 / 5e-3, 5.0)


def test_reference_arm_under_two_ranks_prints_one_line():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "1", "--warmup", "0", "--workload", "tiny"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "TFLOP/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
