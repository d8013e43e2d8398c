"""B200 (sm_100a) gated subspace linear layer: Python binding of the C ABI.

The arithmetic lives in ``csrc/`` (CUDA).  This package only loads
``libgsi_b200.so``, marshals arguments and keeps device memory alive through
torch tensors.  There is no CPU path: importing works anywhere (the library is
cross-compiled), running needs a B200.
"""
from .binding import (  # noqa: F401
    lib, lib_path, GsiError, Layer, Stack,
    gsi_build_image, gsi_workspace_bytes, gsi_status_string, gsi_forward_static,
    GSI_BF16, GSI_F32, GSI_FLAG_NONE, GSI_FLAG_STATIC_PROJECTION, GSI_FLAG_DENSE, GSI_FLAG_FP8_IMAGE,
    GSI_MAX_MAPS, GSI_MAX_TOKENS, EXPORTED,
)
