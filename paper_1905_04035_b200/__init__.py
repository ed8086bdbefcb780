"""B200-native densification of assumed-sparse (IndexedSlices) gradients.

Thin binding over the C-ABI library declared in ``include/dst.h``: the Python
functions carry the same names as the C entry points and only marshal
arguments.  PyTorch supplies device memory and streams; every step of the
operation runs in the library's CUDA kernels.  There is no CPU fallback: if
the library has not been built, calls raise.
"""
from .binding import (  # noqa: F401
    DST_ACC_PROPOSED,
    DST_ACC_SPARSE_AS_DENSE,
    DST_ACC_STOCK,
    DST_OPT_ADAM,
    DST_OPT_MOMENTUM,
    DST_OPT_SGD,
    DST_STATUS,
    Densifier,
    DstError,
    dst_accumulate,
    dst_accumulate_plan,
    dst_bytes_report,
    dst_densify,
    dst_densify_apply,
    dst_densify_batch,
    dst_densify_apply_sgd,
    dst_densify_concat,
    dst_densify_concat_host,
    dst_densify_static,
    dst_host_staging_bytes,
    dst_kernel_launches,
    dst_profile_events,
    dst_profile_ranges,
    dst_selftest_wait_limit,
    dst_status_string,
    dst_version,
    dst_workspace_bytes,
    library_path,
    load_library,
)
