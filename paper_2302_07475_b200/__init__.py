"""S3GD-MV step (top-K sign compression, majority vote, update) for NVIDIA B200.

The compute path is the CUDA library ``libs3gd.so`` (sources in ``csrc/``, C ABI in
``include/s3gd.h``); ``binding`` marshals torch tensors into it.  ``workloads``
draws the seeded synthetic gradient batches used by tests and benchmarks.
"""
from . import workloads  # noqa: F401
from .binding import (  # noqa: F401
    S3gdError, alloc_workspace, load, s3gd_apply, s3gd_device_status, s3gd_majority_vote, s3gd_majority_vote_noalloc, s3gd_noalloc_max_d,
    s3gd_profile_begin, s3gd_profile_begin_filter, s3gd_profile_begin_filter_every, s3gd_profile_end, s3gd_status_string, s3gd_apply_momentum, s3gd_step, s3gd_step_ex, s3gd_topk_sign, s3gd_workspace_bytes,
    s3gd_randk_sign, s3gd_step_randk, s3gd_last_device_status, s3gd_debug_topk_sign, s3gd_debug_step,
    s3gd_vote_apply, s3gd_vote_counts, s3gd_encode_vote2, s3gd_apply_vote2,
    s3gd_sparse_workspace_bytes, s3gd_encode_vote_sparse, s3gd_apply_vote_sparse,
)
