"""One cluster sharded over several GPUs: the driver of the step-by-step calls.

Shard r holds a contiguous block of the cluster's job ids (block r, in global order) in its
own ``Scheduler``.  The driver below runs the protocol of ``include/slaq.h`` ("One cluster
sharded over several GPUs"): per radix pass one sum of a 2048-entry histogram over the shards,
at the end one gather of each shard's number of threshold-equal gains.  Two ways to exchange:

* ``ProcessGroupExchange``: one shard per process, ``torch.distributed`` (NCCL) does the sums;
* ``LocalExchange``: several shards in one process on one GPU, summed directly - the same
  steps in the same order, used to check the protocol where only one GPU is available.
"""

from __future__ import annotations

from .binding import P_FIT_CLUSTER_JOBS

N_PASSES = 6
N_BINS = 2048


class LocalExchange:
    """All shards live in this process, on the current CUDA device."""

    device = "cuda"

    def sum_ints(self, values):
        total = sum(int(v) for v in values)
        return [total] * len(values)

    def sum_histograms(self, buffers):
        total = buffers[0].clone()
        for b in buffers[1:]:
            total += b
        for b in buffers:
            b.copy_(total)

    def ties_before(self, ties):
        """ties: one 1-entry int64 tensor per shard.  Returns per shard the sum over the shards before it."""
        import torch
        stacked = torch.cat(ties)
        before = torch.cumsum(stacked, 0) - stacked
        return [before[i:i + 1].contiguous() for i in range(len(ties))]


class ProcessGroupExchange:
    """One shard per process; ``torch.distributed`` must be initialised (NCCL for GPU tensors)."""

    def __init__(self, group=None, device="cuda"):
        import torch.distributed as dist
        self.dist, self.group, self.device = dist, group, device

    def sum_ints(self, values):
        import torch
        assert len(values) == 1
        t = torch.tensor([int(values[0])], dtype=torch.int64, device=self.device)
        self.dist.all_reduce(t, group=self.group)
        return [int(t.item())]

    def sum_histograms(self, buffers):
        assert len(buffers) == 1
        self.dist.all_reduce(buffers[0], group=self.group)

    def ties_before(self, ties):
        import torch
        assert len(ties) == 1
        world, rank = self.dist.get_world_size(self.group), self.dist.get_rank(self.group)
        out = [torch.zeros_like(ties[0]) for _ in range(world)]
        self.dist.all_gather(out, ties[0], group=self.group)
        return [torch.cat(out)[:rank].sum().reshape(1)]


def schedule_sharded(shards, exchange, epoch_seconds: float, total_cores: int):
    """One epoch of one cluster whose jobs are split over ``shards`` (list of ``Scheduler``; one entry
    per process with ``ProcessGroupExchange``).  Returns the list of per-shard allocations.

    Every shard works on torch's current stream, on which torch orders its collectives as well: the
    exchanges between the steps are stream-ordered, and the host waits for the device only twice, for
    the cluster's job count before anything is queued and for the allocation at the end."""
    import torch
    on_gpu = str(exchange.device).startswith("cuda")
    if on_gpu:
        stream = torch.cuda.current_stream()
        for s in shards:
            if getattr(s, "_sharded_stream", None) != stream.cuda_stream:
                s.set_stream(stream)
                s._sharded_stream = stream.cuda_stream
    cap = shards[0].max_cores_per_job
    assert all(s.max_cores_per_job == cap for s in shards)
    n_jobs = exchange.sum_ints([s.get_active_count() for s in shards])[0]
    with_floor = total_cores >= n_jobs
    for s in shards:                      # every shard fits with the lanes per job the undivided cluster would use
        s.set_param(P_FIT_CLUSTER_JOBS, n_jobs)
    want = min(total_cores, n_jobs * cap) - (n_jobs if with_floor else 0)
    for s in shards:
        s.shard_predict(epoch_seconds, with_floor)
    buffers = [torch.zeros(N_BINS, dtype=torch.int64, device=exchange.device) for _ in shards]
    for p in range(N_PASSES):
        if p > 0:
            for s in shards:
                s.shard_pass(p)
        for s, b in zip(shards, buffers):
            s.shard_histogram(p, b, import_it=False)
        exchange.sum_histograms(buffers)
        for s, b in zip(shards, buffers):
            s.shard_histogram(p, b, import_it=True)
            s.shard_pick(p, want)
    ties = [torch.zeros(1, dtype=torch.int64, device=exchange.device) for _ in shards]
    for s, t in zip(shards, ties):
        s.shard_count_device(t)
    before = exchange.ties_before(ties)
    return [s.shard_finalise_device(b) for s, b in zip(shards, before)]
