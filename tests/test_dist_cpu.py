"""The multi-rank plumbing on CPU: two gloo ranks, no data-path collective, timing
reduced by max over ranks, whole-job rate from per-rank units."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2410_17765_b200 import dist_util, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert dist_util.env_rank_world() == (rank, world, rank)
    assert dist_util.init("gloo")
    cpu = torch.device("cpu")
    # each rank has its own batch (different seeds), nothing is exchanged on the data path
    inp = synth.make_inputs(synth.Shape(4, 64, 16, 2, 2), seed=dist_util.shard_seed(0, rank))
    digest = float(inp.h.float().sum())
    dist_util.barrier()
    slowest = dist_util.max_over_ranks(10.0 * (rank + 1), cpu)
    rate = dist_util.whole_job_rate(units_per_rank=4, steps=5, world=world, elapsed_ms_max=slowest)
    torch.save({"slowest": slowest, "rate": rate, "digest": digest}, os.path.join(out_dir, f"r{rank}.pt"))
    dist_util.barrier()
    dist_util.finalize()


def test_two_gloo_ranks(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(os.path.join(tmp_path, f"r{r}.pt")) for r in range(world)]
    assert all(r["slowest"] == 20.0 for r in res)
    assert all(abs(r["rate"] - 4 * 2 * 5 / 0.020) < 1e-9 for r in res)
    assert res[0]["digest"] != res[1]["digest"]


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert dist_util.env_rank_world() == (0, 1, 0)
    assert dist_util.init("gloo") is False
    assert dist_util.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    assert dist_util.whole_job_rate(10, 2, 1, 100.0) == 200.0
