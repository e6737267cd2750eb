"""The N > 1 path of the benchmark is "replicas only": a barrier around the timed region and the
maximum of the per-rank times.  Exercised here with two gloo ranks on CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2609_19758_b200 import replicas
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    mine = [0.040 + 0.005 * rank, 4.0 - rank, 2.5]          # probe ms, step ms, e2e ms of this rank
    mx = replicas.max_over_ranks(mine, dist)
    dist.barrier()
    if rank == 0:
        torch.save(mx, out)
    dist.destroy_process_group()


def test_max_over_ranks_and_weak_scaling_value(tmp_path):
    from paper_2609_19758_b200 import replicas
    out = str(tmp_path / "mx.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    mx = torch.load(out)
    assert mx == [0.045, 4.0, 2.5]
    # whole-job value: both replicas move their bytes in the time of the slower one
    v = replicas.whole_job_throughput(134217728 / 1e9, mx[0] * 1e-3, 2)
    assert abs(v - 2 * 0.134217728 / 0.045e-3) < 1e-6 * v
    # without a process group the helper is the identity
    assert replicas.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]
