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
        before = ex.ties_before([torch.tensor([7 * (rank + 1)], dtype=torch.int64)])
        out[rank] = dict(total=ex.sum_ints([10 + rank]), before=[int(b.item()) for b in before],
                         hist_ok=bool((hist == torch.arange(N_BINS) * 6).all()))
    finally:
        dist.destroy_process_group()


def test_shard_exchange_over_a_process_group():
    """What the shards of one cluster exchange per epoch (sums of histograms and counts, the tie counts of the
    shards before each), over gloo on CPU; on GPUs the same calls run over NCCL."""
    world, port = 3, 29931 + os.getpid() % 400
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_exchange_worker, args=(world, port, out), nprocs=world, join=True)
    for rank in range(world):
        assert out[rank]["total"] == [33]
        assert out[rank]["before"] == [[0], [7], [21]][rank]          # 7, 14, 21 ties: exclusive prefix over ranks
        assert out[rank]["hist_ok"]
    # the local exchange used on one GPU gives every shard the same answers
    from paper_1802_04819_b200.sharded import LocalExchange
    ex = LocalExchange()
    assert ex.sum_ints([10, 11]) == [21, 21]
    before = ex.ties_before([torch.tensor([7]), torch.tensor([14]), torch.tensor([21])])
    assert [int(b.item()) for b in before] == [0, 7, 21]
    a, b = torch.arange(4), torch.arange(4) * 2
    ex.sum_histograms([a, b])
    assert (a == torch.arange(4) * 3).all() and (b == a).all()


class _StubShard:
    """Stands in for a Scheduler: records the calls of one sharded epoch and plays a shard whose histograms and
    tie count are simple functions of its rank, so that what comes back from the exchange can be checked."""

    def __init__(self, rank, active, cap):
        self.rank, self.active, self.max_cores_per_job, self.calls, self.imported = rank, active, cap, [], {}

    def get_active_count(self):
        self.calls.append(("active",))
        return self.active

    def set_param(self, key, value):
        self.calls.append(("param", key, value))

    def shard_predict(self, T, with_floor):
        self.calls.append(("predict", T, bool(with_floor)))

    def shard_pass(self, p):
        self.calls.append(("pass", p))

    def shard_histogram(self, p, buf, import_it):
        self.calls.append(("import" if import_it else "export", p))
        if import_it:
            self.imported[p] = buf.clone()
        else:
            buf.copy_(torch.arange(buf.numel(), dtype=torch.int64) * (self.rank + 1) + p)

    def shard_pick(self, p, want):
        self.calls.append(("pick", p, want))

    def shard_count_device(self, t):
        self.calls.append(("count",))
        t.fill_(5 + self.rank)

    def shard_finalise_device(self, before):
        self.calls.append(("finalise", int(before.item())))
        return np.full(self.active, self.rank, np.int32)


def _protocol_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_1802_04819_b200.sharded import N_BINS, ProcessGroupExchange, schedule_sharded
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shard = _StubShard(rank, active=100 + rank, cap=8)
        alloc = schedule_sharded([shard], ProcessGroupExchange(device="cpu"), 2.5, 1000)
        want_sum = [torch.arange(N_BINS, dtype=torch.int64) * sum(r + 1 for r in range(world)) + world * p
                    for p in range(6)]
        out[rank] = dict(calls=shard.calls, alloc_ok=bool((alloc[0] == rank).all()),
                         sums_ok=all(bool((shard.imported[p] == want_sum[p]).all()) for p in range(6)))
    finally:
        dist.destroy_process_group()


def test_sharded_epoch_runs_the_protocol_in_order_on_every_rank():
    """schedule_sharded under a process group, with stub shards: every rank makes the calls of the protocol in the
    documented order with the same cluster-wide numbers, imports the sum of all ranks' histograms in every pass,
    and is told the tie count of the ranks before it."""
    world, port = 3, 30331 + os.getpid() % 400
    out = mp.get_context("spawn").Manager().dict()
    mp.spawn(_protocol_worker, args=(world, port, out), nprocs=world, join=True)
    n_jobs = 100 + 101 + 102
    want = 1000 - n_jobs                                   # floor of one core each, cap 8: 1000 < 8 * 303
    from paper_1802_04819_b200.binding import P_FIT_CLUSTER_JOBS
    expected = [("active",), ("param", P_FIT_CLUSTER_JOBS, n_jobs), ("predict", 2.5, True)]
    for p in range(6):
        if p > 0:
            expected.append(("pass", p))
        expected += [("export", p), ("import", p), ("pick", p, want)]
    expected.append(("count",))
    for rank in range(world):
        assert out[rank]["calls"][:-1] == expected, out[rank]["calls"]
        assert out[rank]["calls"][-1] == ("finalise", sum(5 + r for r in range(rank)))
        assert out[rank]["sums_ok"] and out[rank]["alloc_ok"]


def test_single_process_is_identity():
    from paper_1802_04819_b200.partition import max_over_ranks, whole_job_rate
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert whole_job_rate(100_000, 1, 10.0) == 1e7
    np.testing.assert_allclose(whole_job_rate(100_000, 8, 10.0), 8e7)
