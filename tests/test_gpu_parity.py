"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same
seeded inputs.  Integer stages bit-exact; fp16 outputs within 2e-3 * max|y_ref| per row."""
import numpy as np
import pytest
import torch

import aser_synth as synth
from oracle import forward as F
from gpu_util import to_dev, oracle_layer, assert_rows_close, assert_T_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aser(cuda_device):
    import paper_2411_07762_b200 as aser
    return aser


def bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


# ---------------------------------------------------------------------------
# aser_pack_w4 / repack
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("N,K,smooth", [(512, 512, True), (136, 1024, True), (8, 128, False),
                                        (1024, 4096, True), (264, 14336, True)])
def test_pack_w4_bit_exact(aser, N, K, smooth):
    lay = synth.make_layer(1, N, K, seed=100 + N + K, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 11.5) if smooth else None
    W = lay.W.copy()
    if N >= 136:
        W[3] = 0                        # zero row: scale 0, codes 0
        W[5, :] = 0
        W[5, 7] = np.float16(3.5)       # single element: code 7 and exact ties elsewhere
        W[6, :8] = np.array([7, .5, 1.5, 2.5, -2.5, 6.5, -6.5, -7], np.float16)
        W[6, 8:] = 0
    q, w_scale = F.quant_w4(W, s)
    Wq, wsc = aser.pack_w4(to_dev(W), None if s is None else to_dev(s))
    assert np.array_equal(Wq.cpu().numpy(), F.pack_w4(q))
    assert np.array_equal(bits(wsc.cpu().numpy()), bits(w_scale))
    Wk = aser.repack_w4(Wq)
    assert Wk.numel() == aser.repacked_bytes(N, K)
    back = aser.unrepack_w4(Wk, N, K)
    assert torch.equal(back, Wq)


def test_repack_layout_by_definition(aser):
    """Word w of sub-block `sub`, row `row` covers columns 32*sub + 8*w .. +7 with column
    c0+i in nibble 2i and column c0+4+i in nibble 2i+1."""
    N, K = 256, 384
    rng = np.random.default_rng(5)
    q = rng.integers(-8, 8, (N, K)).astype(np.int8)
    Wq = to_dev(F.pack_w4(q))
    Wk = aser.repack_w4(Wq).cpu().numpy().view(np.uint32).reshape(N // 128, K // 128, 4, 128, 4)
    for (nb, kb, sub, row, w) in [(0, 0, 0, 0, 0), (1, 2, 3, 127, 3), (0, 1, 2, 77, 1), (1, 0, 1, 5, 2)]:
        word = int(Wk[nb, kb, sub, row, w])
        c0 = kb * 128 + sub * 32 + w * 8
        n = nb * 128 + row
        for i in range(4):
            assert (word >> (8 * i)) & 0xF == int(q[n, c0 + i]) & 0xF
            assert (word >> (8 * i + 4)) & 0xF == int(q[n, c0 + 4 + i]) & 0xF


# ---------------------------------------------------------------------------
# aser_quant_act
# ---------------------------------------------------------------------------
ACT_CASES = [  # M, K, r
    (1, 512, 16), (3, 4096, 64), (8, 4096, 64), (16, 512, 16), (17, 1024, 0), (32, 8192, 32),
    (33, 512, 16), (127, 1024, 64), (129, 4096, 128), (300, 2048, 256), (64, 14336, 64),
    # cluster kernel: one stage per CTA, r = 0, ranks that leave accumulator rows unused, ragged
    # last token tile, every cluster size
    (65, 128, 0), (200, 128, 48), (96, 8192, 32), (1000, 2048, 112), (2049, 512, 16), (40, 28672, 64),
]


@pytest.mark.parametrize("M,K,r", ACT_CASES)
def test_quant_act_parity(aser, M, K, r):
    lay = synth.make_layer(M, 8, K, seed=200 + M + K + r, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 13.0)
    X = lay.X.copy()
    if M >= 3:
        X[1] = 0                                   # zero token: scale 0, codes 0
        X[2, :] = 0
        X[2, :6] = np.array([127, .5, 1.5, 2.5, -2.5, -126.5], np.float16)   # exact ties
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0] if r else None
    xs = F.smooth_act(X, s)
    Xq_ref, sc_ref = F.quant_act(xs)
    Xq, sc, T = aser.quant_act(to_dev(X), to_dev(s), None if L_A is None else to_dev(L_A))
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
    if r:
        T_ref = F.down_proj(xs, L_A)
        assert_T_close(T.float().cpu().numpy(), T_ref)


@pytest.mark.parametrize("M,K,r", [(8, 1024, 16), (300, 1024, 64), (2048, 512, 32)])
def test_quant_act_dense_smoothing_vector(aser, M, K, r):
    """Every divisor differs from 1 (a SmoothQuant-style vector): the division path everywhere,
    including divisors below 1."""
    lay = synth.make_layer(M, 8, K, seed=400 + M + K + r, n_cal=8)
    rng = np.random.default_rng(M + K)
    s = rng.uniform(0.25, 6.0, size=K).astype(np.float32)
    s[::7] = 1.0
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0]
    xs = F.smooth_act(lay.X, s)
    Xq_ref, sc_ref = F.quant_act(xs)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), to_dev(s), to_dev(L_A))
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
    assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A))


def test_quant_act_without_smoothing_vector(aser):
    lay = synth.make_layer(5, 8, 256, seed=9, n_cal=8)
    Xq, sc, _ = aser.quant_act(to_dev(lay.X), None, None)
    Xq_ref, sc_ref = F.quant_act(F.smooth_act(lay.X, None))
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref) and np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))


# ---------------------------------------------------------------------------
# whole path: quant_act -> linear
# ---------------------------------------------------------------------------
def run_path(aser, lay, s, Wq_ref, w_scale_ref, L_A, L_B, impl, rows=None, use_dgemm=False,
             large_lowrank_term=False):
    M, K = lay.X.shape
    N = lay.W.shape[0]
    r = 0 if L_A is None else L_A.shape[0]
    dW, ds = to_dev(lay.W), to_dev(s)
    Wq, wsc = aser.pack_w4(dW, ds)
    assert np.array_equal(Wq.cpu().numpy(), Wq_ref)
    assert np.array_equal(bits(wsc.cpu().numpy()), bits(w_scale_ref))
    dLA = None if r == 0 else to_dev(L_A)
    dLB = None if r == 0 else to_dev(L_B)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA)
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    if impl == "simt":
        Y = aser.linear_w4a8_lr_simt(Xq, sc, Wq, wsc, T, dLB, acc_debug=acc)
    else:
        Wk = aser.repack_w4(Wq)
        ws = aser.new_workspace(M, N, K, r)
        if r:
            Y = aser.linear_w4a8_lr(Xq, sc, Wk, wsc, T, dLB, N, ws, acc_debug=acc)
        else:
            Y = aser.linear_w4a8(Xq, sc, Wk, wsc, N, ws, acc_debug=acc)
        aser.check_status(ws)
    torch.cuda.synchronize()
    ref = F.forward(lay.X, s, Wq_ref, w_scale_ref, L_A, L_B, rows=rows, use_dgemm=use_dgemm)
    assert np.array_equal(Xq.cpu().numpy(), ref.Xq)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(ref.a_scale))
    acc_h = acc.cpu().numpy()
    assert np.array_equal(acc_h if rows is None else acc_h[rows], ref.acc)
    if large_lowrank_term:
        # The bound 2e-3 * max|y_ref| budgets the bf16 rounding of T (2^-9 relative) for a low-rank
        # term that is a few per cent of y.  Where the factors carry whole weight columns that no
        # longer holds; the rounding of T then adds up to 2^-9 * sum_j |L_B[n,j]| |T[m,j]| (2^-8
        # with the fp16 rounding of x~ in the tensor-core projection), which is allowed on top.
        y_gpu = Y.cpu().numpy().astype(np.float64)
        if rows is not None:
            y_gpu = y_gpu[rows]
        slack = 2.0 ** -8 * (np.abs(ref.T) @ np.abs(L_B.astype(np.float64)).T)
        bound = 2e-3 * np.abs(ref.y).max(axis=1, keepdims=True) + slack
        assert np.all(np.abs(y_gpu - ref.y) <= bound)
    else:
        assert_rows_close(Y.cpu().numpy(), ref.y, rows)
    return Y


PATH_CASES = [  # M, N, K, r
    (16, 512, 512, 16), (1, 256, 512, 16), (7, 136, 1024, 32), (33, 264, 512, 0),
    (130, 384, 1024, 64), (257, 520, 2048, 128), (40, 128, 384, 256),
]


@pytest.mark.parametrize("impl", ["simt", "tc"])
@pytest.mark.parametrize("M,N,K,r", PATH_CASES)
def test_path_parity_small(aser, impl, M, N, K, r):
    lay = synth.make_layer(M, N, K, seed=300 + M + N + K + r, n_cal=64,
                           n_out=max(1, K // 100))
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=(K <= 1024 and r > 0))
    if r == 0:
        L_A = L_B = None
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl)


@pytest.mark.parametrize("impl", ["simt", "tc"])
def test_config1_tiny_with_constructed_factors(aser, impl):
    lay, r = synth.config1_tiny()
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=True)
    Y = run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl)
    # the compensated output is closer to the fp product than the plain W4A8 one
    plain = run_path(aser, lay, s, Wq, w_scale, None, None, impl)
    ref = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    e_lr = np.linalg.norm(Y.cpu().numpy().astype(np.float64) - ref)
    e_plain = np.linalg.norm(plain.cpu().numpy().astype(np.float64) - ref)
    assert e_lr < e_plain


@pytest.mark.parametrize("impl", ["tc"])
@pytest.mark.parametrize("M", [1, 8])
def test_config2_decode_full_size(aser, impl, M):
    lay, r = synth.config2_decode(M)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=(M == 8))
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl, use_dgemm=True)


@pytest.mark.parametrize("impl", ["tc"])
@pytest.mark.parametrize("which", ["gate_up", "down"])
def test_config3_prefill_full_size_sampled_rows(aser, impl, which):
    lay, r = synth.config3_prefill(which)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    rows = np.array([0, 1, 127, 128, 1000, 1023, 1024, 2046, 2047])
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl, rows=rows, use_dgemm=True)


FORWARD_CASES = [  # M, N, K, r
    (8, 512, 4096, 64), (1, 256, 512, 16), (33, 264, 512, 0), (130, 384, 1024, 64),
    (300, 1152, 2048, 128), (2048, 512, 4096, 64),
]


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,r", FORWARD_CASES)
def test_forward_overlapped_is_bit_identical_to_separate_calls(aser, M, N, K, r):
    """aser_forward launches the linear kernel as a programmatic dependent of the quantization
    kernel; every output must equal that of the two plain calls, on repeated back-to-back runs
    with alternating inputs (a missing wait would show as stale Xq, a_scale or T)."""
    lay = synth.make_layer(M, N, K, seed=900 + M + N + K + r, n_cal=8, n_out=max(1, K // 100))
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 9.0)
    L_A, L_B = synth.standin_factors(N, K, r, seed=M + r, scale_a=0.02, scale_b=0.02) if r else (None, None)
    layer = aser.AserLinear(to_dev(lay.W), to_dev(s), None if r == 0 else to_dev(L_A),
                            None if r == 0 else to_dev(L_B), M)
    X0 = to_dev(lay.X)
    X1 = torch.roll(X0, shifts=3, dims=1).contiguous() * 0.5
    want = []
    for X in (X0, X1):
        layer.quant(X)
        layer.linear(M)
        want.append((layer.Y[:M].clone(), layer.Xq[:M].clone(), layer.a_scale[:M].clone(),
                     layer.T[:M].clone()))
    aser.check_status(layer.ws)
    for it in range(12):
        X = (X0, X1)[it & 1]
        Y = layer(X)
        got = (Y, layer.Xq[:M], layer.a_scale[:M], layer.T[:M])
        for g, w in zip(got, want[it & 1]):
            assert torch.equal(g.view(torch.uint8), w.view(torch.uint8)), it
    aser.check_status(layer.ws)


@pytest.mark.parametrize("name", ["k", "gate", "down"])
def test_config4_block_linears_full_size_sampled_rows(aser, name):
    """Decoder-block linears at 4096 tokens, rank 128 (the GQA projection, the widest and the
    deepest layer): every int8 code and scale, and Y on sampled token rows."""
    lay, r = synth.config4_block_layer(name)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    rows = np.array([0, 63, 64, 2047, 2048, 4031, 4095])
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, "tc", rows=rows, use_dgemm=True)


@pytest.mark.parametrize("M,N,r", [(16, 8192, 32), (16, 28672, 64), (128, 28672, 256), (1024, 8192, 128), (4096, 8192, 0)])
def test_config5_sweep_points_sampled_rows(aser, M, N, r):
    """Points of the 70B-class sweep (K = 8192): 16 tokens on both few-token paths (streaming
    kernel up to 64 MB of packed weights, tensor-core kernel above), rank 256 (two launches of the
    quantization cluster kernel) and rank 0 (plain W4A8)."""
    lay = synth.config5_point(M, N)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    if r == 0:
        L_A = L_B = None
    rows = np.unique(np.array([0, 1, M // 2, M - 2, M - 1]).clip(0, M - 1))
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, "tc", rows=rows, use_dgemm=True)


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,r", [(8, 256, 1024, 40), (200, 384, 2048, 72)])
def test_rank_not_a_multiple_of_16_is_padded_with_zeros(aser, M, N, K, r):
    """A per-layer rank from the singular-value threshold (Sec. 4.1) is any integer: pad_rank
    appends zero rows / columns; the result must match the oracle run on the UNPADDED factors."""
    lay = synth.make_layer(M, N, K, seed=700 + r, n_cal=8)
    s, Wq_ref, w_scale_ref, L_A, L_B = oracle_layer(lay, r, construct=False)
    dLA, dLB = aser.pad_rank(to_dev(L_A), to_dev(L_B))
    assert dLA.shape[0] % 16 == 0 and dLB.shape[1] == dLA.shape[0]
    ds = to_dev(s)
    Wq, wsc = aser.pack_w4(to_dev(lay.W), ds)
    Wk = aser.repack_w4(Wq)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA)
    ws = aser.new_workspace(M, N, K, dLA.shape[0])
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = aser.linear_w4a8_lr(Xq, sc, Wk, wsc, T, dLB, N, ws, acc_debug=acc)
    aser.check_status(ws)
    torch.cuda.synchronize()
    ref = F.forward(lay.X, s, Wq_ref, w_scale_ref, L_A, L_B)
    assert np.array_equal(acc.cpu().numpy(), ref.acc)
    assert bool((T[:, r:] == 0).all())
    assert_rows_close(Y.cpu().numpy(), ref.y)


@pytest.mark.gpu
def test_paper_smoothing_rule_with_outlier_split_runs_through_the_same_path(aser):
    """The paper's own variant (Sec. 4.2): m_i = X-bar_i / min over the f outlier channels, and the
    outlier columns W_o kept out of the int4 matrix and carried by the low-rank factors.  For the
    GPU this is the same path with different inputs: the caller zeroes the outlier columns of W
    before packing.  Packed weights and accumulators bit-exact; the output within the bound plus
    the bf16 rounding of T, whose term is now as large as the outlier columns' contribution; and
    the split layer's output is closer to the fp product than plain W4A8 on the same codes."""
    from oracle import construct as Cn
    lay, r = synth.config1_tiny()
    s, idx = Cn.smoothing_vector_paper(lay.X_cal, lay.W, f=4)
    assert np.array_equal(idx, lay.outlier_idx)
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r, split_outliers=idx)
    W_split = lay.W.copy()
    W_split[:, idx] = 0
    lay_split = synth.LayerInputs(X=lay.X, W=W_split, X_cal=lay.X_cal, outlier_idx=lay.outlier_idx,
                                  outlier_gain=lay.outlier_gain, meta=lay.meta)
    Y = run_path(aser, lay_split, s, L.Wq, L.w_scale, L.L_A, L.L_B, "tc", large_lowrank_term=True)
    plain = run_path(aser, lay_split, s, L.Wq, L.w_scale, None, None, "tc")
    ref = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    e_lr = np.linalg.norm(Y.cpu().numpy().astype(np.float64) - ref)
    e_plain = np.linalg.norm(plain.cpu().numpy().astype(np.float64) - ref)
    assert e_lr < 0.5 * e_plain        # without the factors the outlier columns are simply missing


# ---------------------------------------------------------------------------
# 6-bit activation codes (the W4A6 setting): same kernels, narrower code range
# ---------------------------------------------------------------------------
@pytest.mark.gpu
@pytest.mark.parametrize("M,K,r", [(5, 1024, 16), (33, 512, 0), (200, 2048, 64), (300, 2048, 256),
                                   (129, 4096, 128)])
def test_quant_act_6bit_parity(aser, M, K, r):
    lay = synth.make_layer(M, 8, K, seed=600 + M + K + r, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 13.0)
    X = lay.X.copy()
    X[1] = 0                                       # zero token: scale 0, codes 0
    X[2, :] = 0
    X[2, :6] = np.array([31, .5, 1.5, 2.5, -2.5, -30.5], np.float16)   # exact ties at scale 1
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0] if r else None
    xs = F.smooth_act(X, s)
    Xq_ref, sc_ref = F.quant_act(xs, act_bits=6)
    Xq, sc, T = aser.quant_act(to_dev(X), to_dev(s), None if L_A is None else to_dev(L_A), act_bits=6)
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
    assert int(Xq.abs().max()) == 31
    if r:
        assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A))


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,r", [(8, 256, 1024, 16), (130, 384, 1024, 64)])
def test_w4a6_path_parity(aser, M, N, K, r):
    """W4A6: 6-bit codes through the unchanged linear kernels; accumulators bit-exact, output
    within the bound, against the oracle run with act_bits = 6."""
    lay = synth.make_layer(M, N, K, seed=650 + M, n_cal=8)
    s, Wq_ref, w_scale_ref, L_A, L_B = oracle_layer(lay, r, construct=False)
    ds, dLA, dLB = to_dev(s), to_dev(L_A), to_dev(L_B)
    Wq, wsc = aser.pack_w4(to_dev(lay.W), ds)
    Wk = aser.repack_w4(Wq)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA, act_bits=6)
    ws = aser.new_workspace(M, N, K, r)
    acc = torch.zeros((M, N), dtype=torch.int32, device="cuda")
    Y = aser.linear_w4a8_lr(Xq, sc, Wk, wsc, T, dLB, N, ws, acc_debug=acc)
    aser.check_status(ws)
    torch.cuda.synchronize()
    ref = F.forward(lay.X, s, Wq_ref, w_scale_ref, L_A, L_B, act_bits=6)
    assert np.array_equal(Xq.cpu().numpy(), ref.Xq)
    assert np.array_equal(acc.cpu().numpy(), ref.acc)
    assert_rows_close(Y.cpu().numpy(), ref.y)


@pytest.mark.gpu
def test_quant_act_bits_rejects_other_widths(aser):
    X = torch.zeros((4, 128), dtype=torch.float16, device="cuda")
    for bad in (1, 9, 0):
        with pytest.raises(aser.AserError) as err:
            aser.quant_act(X, None, None, act_bits=bad)
        assert err.value.code == -3
