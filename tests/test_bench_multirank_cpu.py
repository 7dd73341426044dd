"""The N > 1 protocol of bench.py (replicas only): every rank times its own replica, a barrier brackets the
timed region and the reported time is the maximum over ranks.  Exercised here with world_size 2 on the gloo
backend (CPU); the data path itself has no collective."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    """One replica: its own per-sequence timings go through bench.py's reduction (the code the benchmark runs)."""
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    steps = 7
    # three timed sequences and the end-to-end time of this replica; rank 1 is slower on the device, rank 0 end to end
    local = torch.tensor([10.0 + 5.0 * rank, 12.0 + 5.0 * rank, 11.0 + 5.0 * rank, 20.0 - 3.0 * rank], dtype=torch.float64)
    red = bench.max_over_ranks(local, world)
    if rank == 0:
        med, mn = bench.per_token_stats([float(t) for t in red[:-1]], steps, world)
        out.put(([float(t) for t in red], med, mn))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    red, med, mn = q.get(timeout=10)
    assert red == [15.0, 17.0, 16.0, 20.0]               # slowest replica decides, entry by entry
    assert med == pytest.approx(16.0 / 14)               # median sequence; 2 replicas x 7 steps = 14 tokens per sequence
    assert mn == pytest.approx(15.0 / 14)


def test_single_rank_reduction_is_the_identity():
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    t = torch.tensor([3.0, 1.0, 2.0], dtype=torch.float64)
    assert bench.max_over_ranks(t, 1) is t
    assert bench.per_token_stats([3.0, 1.0, 2.0], 2, 1) == (1.0, 0.5)


def test_reference_arm_line_on_tiny_config():
    import json
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.check_output([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "tiny",
                                   "--steps", "1", "--warmup", "0"], text=True, timeout=300)
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "ms/token" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert set(line["config"]) == {"workload", "replicas", "l2", "seed"}          # the same keys as the CUDA arm's line
    assert line["value"] > 0
