"""Gradient Agreement Filtering (arxiv 2412.18052) hot path for B200: CUDA library + thin binding.

``binding`` wraps the C ABI of ``include/gaf.h``; ``workloads`` draws the seeded
synthetic micro-gradients used by the tests and the benchmark; ``build``
compiles the library in-tree.
"""
from . import binding, workloads  # noqa: F401
from .binding import (  # noqa: F401
    GAF_BF16, GAF_F32, GAF_SCHED_AUTO, GAF_SCHED_GRAM, GAF_SCHED_GRAM_FUSED, GAF_SCHED_STEPWISE,
    GAF_STATUS_ILL_CONDITIONED, GAF_STATUS_NONFINITE, GAF_STATUS_TIMEOUT, GAF_STATUS_ZERO_NORM, GafError,
    gaf_cosdist, gaf_cosdist_static, gaf_filter_accumulate, gaf_filter_accumulate_any_seed, gaf_filter_accumulate_bucketed, gaf_filter_accumulate_host, gaf_filter_accumulate_repeat, gaf_host_staging_bytes,
    gaf_last_gram_loader, gaf_last_launch_count, gaf_last_schedule, gaf_pairwise_cosdist, gaf_read_status, gaf_workspace_bytes,
    gaf_stream_begin, gaf_stream_end, gaf_stream_push, gaf_test_set_wait_fault, gaf_workspace_init, new_workspace,
)
