"""Host-side checks of the C ABI: the library loads without a GPU, exports every declared
symbol, and rejects bad arguments with an error code before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2411_07762_b200 import build
    build.build()
    from paper_2411_07762_b200 import binding
    return binding.lib


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "aser.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aser_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2411_07762_b200 import binding
    names = declared_symbols()
    assert len(names) >= 14
    for nm in names:
        assert getattr(lib, nm) is not None
    assert set(names) == set(binding.EXPORTED_SYMBOLS)


def test_version_and_sizes(lib):
    assert lib.aser_version() >= 1000
    assert lib.aser_repacked_bytes(128, 128) == 8192
    assert lib.aser_repacked_bytes(129, 256) == 2 * 2 * 8192     # rows padded to 128
    assert lib.aser_repacked_bytes(0, 128) == 0
    assert lib.aser_workspace_bytes(8, 4096, 4096, 64) >= 256
    assert lib.aser_workspace_bytes(8, 4096, 4100, 64) == 0      # bad K


def test_bad_arguments_are_rejected_before_launch(lib):
    OK, NULL, ALIGN, SHAPE, WORKSPACE = 0, -1, -2, -3, -4
    good = C.c_void_p(0x1000)
    odd = C.c_void_p(0x1004)
    # shape errors
    assert lib.aser_pack_w4(good, None, 128, 100, good, good, None) == SHAPE
    assert lib.aser_quant_act(good, None, good, 4, 256, 24, good, good, good, None) == SHAPE
    assert lib.aser_quant_act(good, None, good, 4, 256, 512, good, good, good, None) == SHAPE
    assert lib.aser_linear_w4a8(good, good, good, good, -1, 128, 128, good, None, good, 1 << 20, None) == SHAPE
    # empty problems are no-ops
    assert lib.aser_quant_act(None, None, None, 0, 256, 16, None, None, None, None) == OK
    assert lib.aser_pack_w4(None, None, 0, 256, None, None, None) == OK
    assert lib.aser_linear_w4a8(None, None, None, None, 0, 128, 128, None, None, None, 0, None) == OK
    # null / misaligned pointers
    assert lib.aser_pack_w4(None, None, 128, 128, good, good, None) == NULL
    assert lib.aser_pack_w4(good, None, 128, 128, odd, good, None) == ALIGN
    assert lib.aser_quant_act(good, odd, None, 4, 256, 0, good, good, None, None) == ALIGN
    assert lib.aser_quant_act(good, None, None, 4, 256, 16, good, good, good, None) == NULL
    assert lib.aser_linear_w4a8_lr(good, good, good, good, None, good, 4, 128, 128, 16, good, None,
                                   good, 1 << 20, None) == NULL
    # workspace missing or too small
    assert lib.aser_linear_w4a8(good, good, good, good, 4, 128, 128, good, None, None, 0, None) == WORKSPACE
    assert lib.aser_linear_w4a8(good, good, good, good, 4, 128, 128, good, None, good, 8, None) == WORKSPACE
    assert lib.aser_workspace_init(None, 1024, None) == WORKSPACE
    assert lib.aser_last_error() != b""
    # a fused shared-input group: layer count, N a multiple of 128, one rank within the stacked limit
    i3 = (C.c_int * 3)(256, 128, 128)
    bad_n = (C.c_int * 2)(256, 136)
    i5 = (C.c_int * 5)(128, 128, 128, 128, 128)
    cat = lambda n, N, r, ws=good, nbytes=1 << 24: lib.aser_linear_w4a8_lr_cat(
        good, good, good, good, good, good, n, N, r, 64, 256, good, ws, nbytes, None)
    assert cat(5, i5, 16) == SHAPE
    assert cat(2, bad_n, 16) == SHAPE
    assert cat(3, i3, 192) == SHAPE                 # 3 x 192 stacked rows of T
    assert cat(0, i3, 16) == SHAPE
    assert cat(3, None, 16) == SHAPE
    assert cat(3, i3, 16, None, 0) == WORKSPACE
    assert lib.aser_forward_shared_cat_workspace_bytes(3, i3, 16, 64, 256) >= lib.aser_workspace_bytes(64, 512, 256, 16)
    assert lib.aser_forward_shared_cat_workspace_bytes(2, bad_n, 16, 64, 256) == 0
    assert lib.aser_forward_shared_cat(good, None, good, 3, good, good, good, i3, 16, 64, 256, good, good, good,
                                       None, good, 1 << 24, None) == NULL      # Y missing


def test_binding_refuses_cpu_tensors(lib):
    import torch
    import paper_2411_07762_b200 as aser
    with pytest.raises(TypeError):
        aser.pack_w4(torch.zeros(128, 128, dtype=torch.float16), None)
