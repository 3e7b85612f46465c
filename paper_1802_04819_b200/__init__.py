"""B200-native per-epoch scheduling path of a quality-driven ML-job scheduler.

A thin binding over the C ABI in ``include/slaq.h``: every step (normalise, fit,
predict, allocate) runs in the CUDA kernels of ``libslaq.so``; Python only marshals
arguments.  Importing this package does not need a GPU; creating a ``Scheduler`` does.
"""

from .binding import (  # noqa: F401
    JOB_FIT_FAILED, JOB_FITTED, JOB_FLAT, JOB_INACTIVE, JOB_NEW, JOB_NO_TIME, JOB_NONFINITE, JOB_SHORT,
    EXPORTED_SYMBOLS, STATIC_MAX_JOBS, Scheduler, SlaqError, Stats, allocate_static, load_library, workspace_bytes,
)
from .build import build  # noqa: F401
from .sharded import LocalExchange, ProcessGroupExchange, schedule_sharded  # noqa: F401
