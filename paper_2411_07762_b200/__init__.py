"""B200 (sm_100a) library for the forward pass of an ASER-quantized linear layer
(arXiv 2411.07762): thin Python binding over the C ABI declared in include/aser.h.

Every step of the path runs in the library's CUDA kernels; this package only marshals
torch device pointers and the current stream.  There is no CPU or PyTorch fallback: if
libaser.so is missing, importing `paper_2411_07762_b200.binding` raises.
"""
from .binding import (  # noqa: F401
    AserError, lib, lib_path, version, last_error,
    pack_w4, repack_w4, unrepack_w4, repacked_bytes, quant_act,
    linear_w4a8_lr, linear_w4a8, linear_w4a8_lr_simt,
    workspace_bytes, new_workspace, check_status, forward_host,
    AserLinear, EXPORTED_SYMBOLS,
)
