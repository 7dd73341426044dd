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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    local_ms = torch.tensor([10.0 + 5.0 * rank, 20.0 - 3.0 * rank], dtype=torch.float64)   # (device ms, e2e ms) of this replica
    dist.all_reduce(local_ms, op=dist.ReduceOp.MAX)
    steps = 7
    tokens = steps * world
    if rank == 0:
        out.put((float(local_ms[0]), float(local_ms[1]), local_ms[0].item() / tokens))
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
        p.join(60)
        assert p.exitcode == 0
    dev_ms, e2e_ms, per_token = q.get(timeout=10)
    assert dev_ms == 15.0 and e2e_ms == 20.0            # slowest replica decides
    assert per_token == pytest.approx(15.0 / 14)        # aggregate ms per token over both replicas


def test_reference_arm_line_on_tiny_config():
    import json
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.check_output([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--config", "tiny",
                                   "--steps", "1", "--warmup", "0"], text=True, timeout=300)
    line = json.loads(out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "ms/token" and line["higher_is_better"] is False
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["value"] > 0
