"""Overlap-Local-SGD hot path for m simulated workers on one B200.

The work is done by hand-written sm_100a CUDA kernels behind the C ABI declared
in include/olsgd.h (built in-tree as libolsgd.so); `binding` marshals arguments
to it.  PyTorch supplies device memory and streams only.
"""
from .binding import (OverlapLocalSGD, OlsgdError, class_pairs, class_pairs_noalloc,  # noqa: F401
                      lib_path, load_library, set_launch_overlap, set_gemm_pairs, tensor_core_launches,
                      KERNEL_CLASSES,
                      NOALLOC_MAX_WORKERS)
