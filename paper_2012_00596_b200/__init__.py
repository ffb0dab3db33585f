"""B200-native block-punched CONV / block-based GEMM library (thin Python binding over a C ABI).

``inputs`` draws the seeded synthetic workloads; everything else is the ctypes binding over
``libnpas.so`` (see ``include/npas.h``).  Importing the package does not load the library; the
first call does, and fails loudly when it has not been built.
"""
from . import inputs  # noqa: F401
from .binding import (BF16, F32, BbBlob, BpBlob, NpasError, blob_check, check_device_status, conv2d_bp, conv2d_bp_maxpool, conv2d_bp_static_ws,  # noqa: F401
                      launch_count, linear_bb, load, mask_bb_from_dense, mask_bp_from_dense, mask_to_numpy,
                      maxpool2d, pack_bb, pack_bp, conv2d_bp_kernel, conv2d_bp_workspace, linear_bb_kernel, tune_conv2d_bp, tune_linear_bb, PlanCache,
                      CONV_KERNELS, LINEAR_KERNELS, prune_bb_magnitude, prune_bp_magnitude, prune_bp_magnitude_global, status_string, subsample2d, unpack_bb, unpack_bp, workspace)
