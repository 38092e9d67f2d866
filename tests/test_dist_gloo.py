"""The N > 1 path on CPU: two gloo ranks agree on the slowest time, shard rows without gaps or
overlap, and report whole-job throughput; a rank that raises is seen by the parent."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out_dir, fail_rank):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2607_20501_b200 import dist as D
    assert D.env_world() == (rank, rank, world)
    assert D.init("gloo") is True
    if rank == fail_rank:
        raise RuntimeError("injected failure on the host")
    D.barrier()
    t = D.max_over_ranks([1.0 + rank, 5.0 - rank, 2.5])
    lo, hi = D.shard_rows(103, rank, world)
    thr = D.aggregate_throughput(10.0, world, t[0])
    with open(os.path.join(out_dir, f"r{rank}.txt"), "w") as f:
        f.write(repr((t, lo, hi, thr)))
    D.barrier()
    torch.distributed.destroy_process_group()


def test_two_ranks_agree(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path), -1), nprocs=world, join=True)
    res = [eval(open(tmp_path / f"r{r}.txt").read()) for r in range(world)]
    assert res[0][0] == res[1][0] == [2.0, 5.0, 2.5]            # element-wise max over ranks
    assert (res[0][1], res[0][2], res[1][1], res[1][2]) == (0, 52, 52, 103)   # contiguous, no gap, no overlap
    assert res[0][3] == res[1][3] == 10.0 * 2 / 2.0            # whole-job units / slowest rank's time


def test_a_failing_rank_is_reported(tmp_path):
    world, port = 2, _free_port()
    with pytest.raises(Exception):
        mp.spawn(_worker, args=(world, port, str(tmp_path), 1), nprocs=world, join=True)


def test_single_process_defaults():
    sys.path.insert(0, ROOT)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    from paper_2607_20501_b200 import dist as D
    assert D.env_world() == (0, 0, 1) and D.init("gloo") is False
    assert D.max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert [D.shard_rows(10, r, 3) for r in range(3)] == [(0, 4), (4, 7), (7, 10)]
