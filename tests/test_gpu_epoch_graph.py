"""The epoch replayed as one CUDA graph (SLAQ_P_EPOCH_GRAPH) gives what the plain launches give."""

import numpy as np
import pytest
import torch

from gpu_common import make_scheduler
from workloads import make_workload

pytestmark = pytest.mark.gpu


def _epochs(slaq, wl, graph, stream=None, selection=0):
    """Four scheduling epochs (the second captures the graph when it is on), then one new loss per job and
    three more, then another epoch length: allocations, predictions and statistics of every call."""
    sched = make_scheduler(wl, packed=False)
    if stream is not None:
        sched.set_stream(stream)
    sched.set_param(slaq.binding.P_EPOCH_GRAPH, graph)
    sched.set_param(slaq.binding.P_SELECTION, selection)
    ids = np.arange(wl.n_jobs, dtype=np.int32)
    out = []

    def run(T):
        alloc, rc = sched.schedule(T, wl.total_cores)
        pred = sched.get_predictions()
        st = sched.get_stats()
        assert st.ms_total > 0.0 and st.launches >= 15
        assert st.ms_fit > 0.0 or graph != 0          # a replayed graph has no stage times
        out.append((alloc.copy(), pred["gain"].copy(), pred["R"].copy(), rc, st.launches))

    for _ in range(4):
        run(wl.epoch_seconds)
    last = wl.losses[wl.offsets[1:] - 1]
    sched.append_losses(ids, 0.97 * last, wl.s + wl.w)
    for _ in range(3):
        run(wl.epoch_seconds)
    for _ in range(2):
        run(2.0 * wl.epoch_seconds)
    sched.close()
    return out


@pytest.mark.parametrize("cfg,n_jobs", [(1, None), (2, 1500)])
def test_graph_replay_equals_plain_launches(cfg, n_jobs):
    import paper_1802_04819_b200 as slaq
    wl = make_workload(cfg, n_jobs=n_jobs)
    plain = _epochs(slaq, wl, 0)
    own = torch.cuda.Stream()
    for graph, stream in ((1, None), (1, own.cuda_stream), (-1, None)):
        replay = _epochs(slaq, wl, graph, stream)
        assert len(replay) == len(plain)
        for a, b in zip(plain, replay):
            np.testing.assert_array_equal(a[0], b[0])
            np.testing.assert_array_equal(a[1].view(np.int64), b[1].view(np.int64))
            np.testing.assert_array_equal(a[2].view(np.int64), b[2].view(np.int64))
            assert a[3] == b[3] and a[4] == b[4]
    assert not np.array_equal(plain[3][0], plain[4][0]) or not np.array_equal(plain[3][1], plain[4][1])


def test_graph_replay_without_a_gain_table():
    """Selection without a table inside a replayed graph: the gain rows asked for after every epoch are written on
    request and belong to that epoch, also after new losses arrived between two replays of the same graph."""
    import paper_1802_04819_b200 as slaq
    wl = make_workload(1)
    plain = _epochs(slaq, wl, 0, selection=1)
    replay = _epochs(slaq, wl, 1, selection=1)
    table = _epochs(slaq, wl, 0, selection=0)
    for a, b, c in zip(plain, replay, table):
        np.testing.assert_array_equal(a[0], b[0])
        np.testing.assert_array_equal(a[1].view(np.int64), b[1].view(np.int64))
        np.testing.assert_array_equal(a[2].view(np.int64), b[2].view(np.int64))
        np.testing.assert_array_equal(a[1].view(np.int64), c[1].view(np.int64))     # the rows are the table's rows
        assert a[0].sum() == c[0].sum()


def test_the_parameter_is_checked():
    import paper_1802_04819_b200 as slaq
    wl = make_workload(0)
    sched = make_scheduler(wl)
    assert sched.get_param(slaq.binding.P_EPOCH_GRAPH) == -1
    with pytest.raises(slaq.SlaqError):
        sched.set_param(slaq.binding.P_EPOCH_GRAPH, 2)
    sched.close()
