"""The N > 1 path on CPU: two gloo ranks exercise the sharding and the max/sum-over-ranks plumbing
that bench.py uses under torchrun (no GPU, no attention arithmetic)."""
import os
import socket

import pytest

from paper_2609_10937_b200 import multirank


def test_shard_is_a_balanced_partition():
    for n, world in [(128, 8), (7, 2), (1, 4), (0, 3), (129, 8)]:
        parts = [multirank.shard(n, r, world) for r in range(world)]
        flat = [i for p in parts for i in p]
        assert flat == list(range(n))
        sizes = [len(p) for p in parts]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        multirank.shard(4, 2, 2)
    assert len({multirank.rank_seed(0, r) for r in range(8)}) == 8


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch.distributed as dist

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dist.barrier()
        ms = 1.0 + rank                      # rank 1 is the slow one
        work = 10.0 * (rank + 1)
        slowest = multirank.max_over_ranks(ms, dist)
        total = multirank.sum_over_ranks(work, dist)
        rate = multirank.whole_job_rate(work, ms, dist)
        mine = list(multirank.shard(7, rank, world))
        with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as fh:
            fh.write(f"{slowest} {total} {rate} {mine}\n")
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_aggregates(tmp_path):
    import torch.multiprocessing as mp

    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    lines = [open(tmp_path / f"rank{r}.txt").read().split(" ", 3) for r in range(world)]
    for slowest, total, rate, _ in lines:
        assert float(slowest) == 2.0            # max over ranks of (1.0, 2.0)
        assert float(total) == 30.0             # 10 + 20
        assert float(rate) == 15.0              # all work over the slowest rank's time
    assert lines[0][3].strip() == "[0, 1, 2]" and lines[1][3].strip() == "[3, 4, 5, 6]"


def test_without_a_process_group_the_helpers_are_identities():
    assert multirank.max_over_ranks(3.5) == 3.5
    assert multirank.whole_job_rate(8.0, 2.0) == 4.0
