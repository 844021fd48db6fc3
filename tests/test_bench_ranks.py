"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own batch (weak scaling, no
data-path collective); the job time is the maximum over ranks and the rows are summed."""
import os
import socket
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2605_28396_b200 import synth
    # every rank generates its own windows, as bench.py does with its rank-dependent seed
    w, r = synth.windows_for(2, 8, 1024, seed=synth.SEED_BASE + 100000 * rank)
    rows = int(torch.minimum(w, r).sum())
    times, total = bench.aggregate_over_ranks([10.0 + rank, 5.0 - rank], rows, "cpu", world)
    dist.barrier()
    if rank == 0:
        torch.save({"times": times, "total": total, "rows0": rows}, out)
    dist.destroy_process_group()


def test_two_rank_aggregation_is_max_time_and_summed_rows(tmp_path):
    world, port, out = 2, _free_port(), tmp_path / "agg.pt"
    mp.spawn(_rank_main, args=(world, port, str(out)), nprocs=world, join=True)
    got = torch.load(out)
    sys.path.insert(0, str(ROOT))
    from paper_2605_28396_b200 import synth
    rows = []
    for rank in range(world):
        w, r = synth.windows_for(2, 8, 1024, seed=synth.SEED_BASE + 100000 * rank)
        rows.append(int(torch.minimum(w, r).sum()))
    assert rows[0] != rows[1]                      # the ranks really hold different batches
    assert got["times"] == [11.0, 5.0]             # max over ranks of each timing
    assert got["total"] == float(sum(rows)) and got["rows0"] == rows[0]


def test_single_rank_aggregation_needs_no_process_group():
    sys.path.insert(0, str(ROOT))
    import bench
    times, total = bench.aggregate_over_ranks([3.5], 42, "cpu", 1)
    assert times == [3.5] and total == 42.0
