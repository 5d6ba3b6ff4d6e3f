"""BigBird block-sparse attention forward for NVIDIA B200 (sm_100a).

A thin ctypes binding over the C-ABI library built from ``csrc/`` (see
``include/bigbird.h``).  PyTorch is used for device memory and streams only;
every step of the attention runs in the library's CUDA kernels.  There is no
CPU or PyTorch fallback: if the shared library is missing, importing the
binding raises.
"""
from .binding import (  # noqa: F401
    BIGBIRD_BF16,
    BIGBIRD_ETC,
    BIGBIRD_FP32,
    BIGBIRD_ITC,
    BigBirdError,
    Layout,
    bigbird_attn_bwd,
    bigbird_attn_fwd,
    bigbird_attn_fwd_simt,
    bigbird_attn_fwd_static,
    bigbird_build_layout,
    bigbird_last_launch_count,
    bigbird_last_status,
    bigbird_last_status_static,
    bigbird_selftest_wait_expiry,
    bigbird_strerror,
    lib,
    library_path,
)
