"""The N > 1 host logic on CPU: two gloo ranks, one cluster partition each."""

import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_1802_04819_b200.partition import max_over_ranks, partition_seed_offset, rank_info, whole_job_rate
    from workloads import make_workload
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert rank_info() == (rank, rank, world)
        wl = make_workload(1, seed_offset=partition_seed_offset(rank))
        dist.barrier()
        mine = [10.0 + rank, 3.0 - rank]                      # pretend step times: rank 1 slower on the first
        worst = max_over_ranks(mine)
        sums = torch.tensor([float(wl.losses.sum())], dtype=torch.float64)
        gathered = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(gathered, sums)
        out[rank] = dict(worst=worst, rate=whole_job_rate(wl.n_jobs, world, worst[0]), n_jobs=wl.n_jobs,
                         checksums=[float(g[0]) for g in gathered])
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_ranks_partition_and_timing():
    world, port = 2, 29531 + os.getpid() % 400
    manager = mp.get_context("spawn").Manager()
    out = manager.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    a, b = out[0], out[1]
    assert a["worst"] == b["worst"] == [11.0, 3.0]            # every rank ends with the slowest rank's times
    assert a["rate"] == b["rate"] == 2 * a["n_jobs"] / 11e-3  # whole-job rate: all ranks' jobs over the slowest time
    assert a["checksums"] == b["checksums"]
    assert a["checksums"][0] != a["checksums"][1]             # the two partitions hold different jobs


def _exchange_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_1802_04819_b200.sharded import N_BINS, ProcessGroupExchange
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ex = ProcessGroupExchange(device="cpu")
        hist = torch.arange(N_BINS, dtype=torch.int64) * (rank + 1)
        ex.sum_histograms([hist])
        out[rank] = dict(total=ex.sum_ints([10 + rank]), ties=ex.gather_ints([7 * (rank + 1)]), ranks=ex.ranks(1),
                         hist_ok=bool((hist == torch.arange(N_BINS) * 3).all()))
    finally:
        dist.destroy_process_group()


def test_shard_exchange_over_a_process_group():
    """What the shards of one cluster exchange per epoch (sums of histograms and counts, gathered tie counts),
    over gloo on CPU; on GPUs the same calls run over NCCL."""
    world, port = 2, 29931 + os.getpid() % 400
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_exchange_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        assert out[rank]["total"] == [21]
        assert out[rank]["ties"] == [[7, 14]]
        assert out[rank]["ranks"] == [rank]
        assert out[rank]["hist_ok"]
    # the local exchange used on one GPU gives every shard the same answers
    from paper_1802_04819_b200.sharded import LocalExchange
    ex = LocalExchange()
    assert ex.sum_ints([10, 11]) == [21, 21] and ex.gather_ints([7, 14]) == [[7, 14], [7, 14]] and ex.ranks(2) == [0, 1]
    a, b = torch.arange(4), torch.arange(4) * 2
    ex.sum_histograms([a, b])
    assert (a == torch.arange(4) * 3).all() and (b == a).all()


def test_single_process_is_identity():
    from paper_1802_04819_b200.partition import max_over_ranks, whole_job_rate
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert whole_job_rate(100_000, 1, 10.0) == 1e7
    np.testing.assert_allclose(whole_job_rate(100_000, 8, 10.0), 8e7)
