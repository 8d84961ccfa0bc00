"""B200 (sm_100a) library for the forward pass of an ASER-quantized linear layer
(arXiv 2411.07762): thin Python binding over the C ABI declared in include/aser.h.

Every step of the path runs in the library's CUDA kernels; this package only marshals
torch device pointers and the current stream.  There is no CPU or PyTorch fallback: the
first use of any binding name loads libaser.so and raises ImportError if it has not been
built (`python -m paper_2411_07762_b200.build`).
"""
import importlib

_BINDING_NAMES = (
    "AserError", "lib", "lib_path", "version", "last_error",
    "pack_w4", "repack_w4", "unrepack_w4", "repacked_bytes", "quant_act",
    "linear_w4a8_lr", "linear_w4a8", "linear_w4a8_lr_simt", "linear_w4a8_lr_static",
    "workspace_bytes", "new_workspace", "check_status", "forward_host",
    "AserLinear", "EXPORTED_SYMBOLS", "pad_rank", "pair_up_projection", "quant_act_ws", "quant_workspace_bytes", "quant_act_ws_launches", "forward_act_launches",
    "linear_w4a8_lr_ld", "AserSharedInput", "AserSharedInputCat", "construct",
)


def __getattr__(name):
    if name in _BINDING_NAMES or name == "binding":
        binding = importlib.import_module(__name__ + ".binding")
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(name)
