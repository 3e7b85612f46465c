"""The allocation-free entry point against the handle-based one.

Some callers may not allocate device memory once they are running (a scheduler loop
beside other GPU work that cannot take cudaMalloc's device-wide synchronisation, a
plug-in with a fixed budget).  slaq_allocate_static serves them from a scratch array
inside the library image.  Here it must hand out exactly the cores that
slaq_allocate_only hands out for the same gain rows, twice in a row, because the second
call starts from whatever the first left in the shared scratch.
"""

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def test_static_allocation_equals_handle_allocation_twice():
    import torch
    assert torch.cuda.is_available()
    import paper_1802_04819_b200 as slaq
    slaq.build()
    rng = np.random.default_rng(12)
    J, cap = 5000, 48
    gain_a = -np.sort(-rng.uniform(0, 1, (J, cap)) * rng.uniform(0.01, 2, (J, 1)), axis=1)
    gain_b = -np.sort(-rng.integers(0, 5, (J, cap)).astype(float) / 4.0, axis=1)     # many exact ties
    with slaq.Scheduler(J, 8, cap) as sched:
        sched.append_losses(np.arange(J), np.ones(J))                                # every row an active job
        d_alloc = torch.empty(J, dtype=torch.int32, device="cuda")
        d_red = torch.empty(J, dtype=torch.float64, device="cuda")
        stream = torch.cuda.current_stream()
        for gain, C in ((gain_a, 4 * J), (gain_b, 3 * J + 17), (gain_a, J - 5), (gain_b, J * cap + 9)):
            sched.set_gains(gain)
            want, want_rc = sched.allocate_only(C)
            want_red = sched.get_predictions(want_gain=False)["R"]
            d_gain = torch.from_numpy(gain).cuda()
            d_alloc.fill_(-7)
            rc = slaq.allocate_static(d_gain, C, d_alloc, d_red, stream)
            stream.synchronize()
            assert rc == want_rc
            np.testing.assert_array_equal(d_alloc.cpu().numpy(), want)               # integer work: bit-exact
            np.testing.assert_array_equal(d_red.cpu().numpy(), want_red)             # same kernel, same order of sums


def test_static_allocation_rejects_sizes_beyond_its_scratch():
    import torch
    import paper_1802_04819_b200 as slaq
    slaq.build()
    J = slaq.STATIC_MAX_JOBS + 1
    d_gain = torch.zeros((J, 2), dtype=torch.float64, device="cuda")
    d_alloc = torch.full((J,), -1, dtype=torch.int32, device="cuda")
    d_red = torch.zeros(J, dtype=torch.float64, device="cuda")
    with pytest.raises(slaq.SlaqError) as e:
        slaq.allocate_static(d_gain, J, d_alloc, d_red)
    assert e.value.code == -2
    torch.cuda.synchronize()
    assert (d_alloc == -1).all()          # nothing ran
