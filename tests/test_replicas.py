"""The N > 1 bookkeeping of the benchmark (replicas only: no exchange on the data
path), run as two gloo ranks on the CPU."""
import json
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_08524_b200.replicas import Replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    reps = Replicas(dist, "cpu")
    reps.barrier()
    ms_local = 10.0 + 5.0 * rank          # rank 1 is the slow one
    units_local = 255 * (rank + 1)        # unequal on purpose
    res = (reps.rank, reps.world, reps.max_ms(ms_local), reps.total_units(units_local),
           reps.throughput(units_local, ms_local))
    with open(os.path.join(out, f"rank{rank}.json"), "w") as f:
        json.dump(res, f)
    reps.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_job_totals_over_the_slowest_rank(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    res = {r: json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)}
    for rank in range(world):
        r, w, ms, units, tput = res[rank]
        assert (r, w) == (rank, world)
        assert ms == 15.0                                   # max over ranks, on every rank
        assert units == 255 * 3
        assert abs(tput - 255 * 3 / 15e-3) < 1e-6


def test_single_process_is_the_one_rank_case():
    reps = Replicas(None, "cpu")
    assert (reps.rank, reps.world) == (0, 1)
    reps.barrier()
    assert reps.max_ms(2.5) == 2.5 and reps.total_units(7) == 7
    assert reps.throughput(100, 50.0) == 2000.0
