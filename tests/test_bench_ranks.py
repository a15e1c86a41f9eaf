"""The multi-rank leg of bench.py on CPU: two gloo ranks stand in for two GPUs.  Ranks are independent replicas (no
collective on the data path); the only exchange is the final gathering of the result, checked here: the job's time is the
slowest rank's and its units are the sum over ranks."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from tests.conftest import ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seconds, units = bench.reduce_over_ranks(0.010 * (rank + 1), 1000.0 + rank, torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        out.put((seconds, units))
    dist.destroy_process_group()


def test_two_ranks_report_max_time_and_summed_units():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    seconds, units = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert abs(seconds - 0.020) < 1e-12 and units == 2001.0


def test_gpus_flag_starts_its_own_ranks():
    """`bench.py --gpus 2` outside a torchrun launch starts two ranks itself; here with the CPU-only plumbing mode, so that
    the start-up and the gathering run without a GPU."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-plumbing-only"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    d = json.loads(line)
    assert d["n_gpus"] == 2 and abs(d["seconds"] - 0.020) < 1e-12 and d["units"] == 2001.0
