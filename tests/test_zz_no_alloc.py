"""aser_linear_w4a8_lr_static: the linear kernel for callers that have no device memory to
spare for a workspace and are not in a position to allocate one (a process whose memory budget
was fixed at start-up, or a point in a step where cudaMalloc's device synchronisation is not
acceptable).  Its scratch is an 8 MiB array built into the library, shared by all calls.

Checked here through the C ABI: calls in a row (different token counts and inputs, so each
call meets whatever the previous one left in the array) give the same output as
aser_linear_w4a8_lr with a caller-provided workspace, and a problem that does not fit the
built-in array is refused without launching anything.

This file is collected last on purpose: if it fails, a run that stops at the first failure has
already run every other test.
"""
import numpy as np
import pytest
import torch

import aser_synth as synth
from gpu_util import to_dev, oracle_layer, assert_rows_close
from oracle import forward as F

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aser(cuda_device):
    import paper_2411_07762_b200 as aser
    return aser


def _run_both(aser, M, N, K, r, seed):
    lay = synth.make_layer(M, N, K, seed=seed, n_cal=16)
    s, Wq_ref, w_scale_ref, L_A, L_B = oracle_layer(lay, r, construct=False)
    ds = to_dev(s)
    Wq, wsc = aser.pack_w4(to_dev(lay.W), ds)
    Wk = aser.repack_w4(Wq)
    dLA, dLB = to_dev(L_A), to_dev(L_B)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA)
    ws = aser.new_workspace(M, N, K, r)
    acc_a = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    acc_b = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y_ws = aser.linear_w4a8_lr(Xq, sc, Wk, wsc, T, dLB, N, ws, acc_debug=acc_a)
    aser.check_status(ws)
    Y_static = aser.linear_w4a8_lr_static(Xq, sc, Wk, wsc, T, dLB, N, acc_debug=acc_b)
    torch.cuda.synchronize()
    # same inputs (at M <= 16 the workspace call runs the streaming kernel, the static one always
    # the tensor-core kernel): integer accumulators identical, outputs within the suite's bound
    assert torch.equal(acc_a, acc_b)
    y_ws = Y_ws.cpu().numpy().astype(np.float64)
    assert_rows_close(Y_static.cpu().numpy(), y_ws)
    # and both agree with the CPU oracle
    ref = F.forward(lay.X, s, Wq_ref, w_scale_ref, L_A, L_B, use_dgemm=True)
    assert np.array_equal(acc_b.cpu().numpy(), ref.acc)
    assert_rows_close(Y_static.cpu().numpy(), ref.y)


def test_static_scratch_matches_workspace_version_calls_in_a_row(aser):
    _run_both(aser, 8, 1024, 2048, 64, seed=901)    # several CTAs share each tile
    _run_both(aser, 19, 384, 1024, 32, seed=902)    # different shape: stale contents must not matter
    _run_both(aser, 8, 1024, 2048, 64, seed=903)


def test_static_scratch_refuses_problems_beyond_its_size(aser):
    M, N, K, r = 64, 256, 512, 16
    assert aser.workspace_bytes(M, N, K, r) > 8 << 20
    Xq = torch.zeros((M, K), dtype=torch.int8, device="cuda")
    sc = torch.ones((M,), dtype=torch.float32, device="cuda")
    Wk = torch.zeros((aser.repacked_bytes(N, K),), dtype=torch.uint8, device="cuda")
    wsc = torch.ones((N,), dtype=torch.float32, device="cuda")
    T = torch.zeros((M, r), dtype=torch.bfloat16, device="cuda")
    LB = torch.zeros((N, r), dtype=torch.float16, device="cuda")
    Y = torch.full((M, N), 7.0, dtype=torch.float16, device="cuda")
    with pytest.raises(aser.AserError) as err:
        aser.linear_w4a8_lr_static(Xq, sc, Wk, wsc, T, LB, N, Y=Y)
    assert err.value.code == -4 and "8388608" in str(err.value)
    torch.cuda.synchronize()
    assert bool((Y == 7.0).all())                   # nothing was launched
