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
    import os
    import paper_2411_07762_b200 as aser
    # the oracle's row loops are independent: all host cores for the full-size cases
    F.set_threads(len(os.sched_getaffinity(0)))
    yield aser
    F.set_threads(1)


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
        assert_T_close(T.float().cpu().numpy(), T_ref, xs, L_A)


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
    assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A), xs, L_A)


@pytest.mark.parametrize("path,M,K,r", [("cluster", 4096, 4096, 64), ("ws", 4800, 8192, 16)])
def test_quant_act_dense_smoothing_long_slices(aser, path, M, K, r):
    """Every divisor differs from 1 on slices long enough that a CTA meets more units with a
    divisor than it keeps in shared memory (the cluster kernel keeps 62 of its 128, the
    projection kernel 254 of its 256): the rest read their divisors from global memory."""
    lay = synth.make_layer(M, 8, K, seed=430 + M + K + r, n_cal=8)
    rng = np.random.default_rng(M + K + 1)
    s = rng.uniform(0.25, 6.0, size=K).astype(np.float32)
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0]
    xs = F.smooth_act(lay.X, s)
    Xq_ref, sc_ref = F.quant_act(xs)
    fn = aser.quant_act if path == "cluster" else aser.quant_act_ws
    Xq, sc, T = fn(to_dev(lay.X), to_dev(s), to_dev(L_A))
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
    assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A), xs, L_A)


def test_quant_act_without_smoothing_vector(aser):
    lay = synth.make_layer(5, 8, 256, seed=9, n_cal=8)
    Xq, sc, _ = aser.quant_act(to_dev(lay.X), None, None)
    Xq_ref, sc_ref = F.quant_act(F.smooth_act(lay.X, None))
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref) and np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))


WS_ACT_CASES = [  # M, K, r, t_pair
    (33, 512, 16, False), (127, 1024, 64, False), (129, 4096, 128, False), (300, 2048, 256, False),
    (64, 14336, 64, False), (200, 128, 48, False), (65, 256, 0, False), (1000, 2048, 112, False),
    (2049, 512, 16, False), (40, 28672, 64, False),
    # stacked down projections of several layers (more than 256 rows), the pair storage of T,
    # and enough tokens at K = 14336 for the pass to be cut into chunks
    (700, 4096, 384, False), (260, 1024, 512, False), (300, 2048, 96, True), (4096, 14336, 128, False),
]


@pytest.mark.parametrize("M,K,r,t_pair", WS_ACT_CASES)
def test_quant_act_ws_parity(aser, M, K, r, t_pair):
    """aser_quant_act_ws (two kernels, caller's scratch): codes and scales bit-exact against the
    oracle, T within the derived bound, on ragged token tiles, zero rows and exact ties."""
    lay = synth.make_layer(M, 8, K, seed=250 + M + K + r, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 13.0)
    X = lay.X.copy()
    X[1] = 0
    X[2, :] = 0
    X[2, :6] = np.array([127, .5, 1.5, 2.5, -2.5, -126.5], np.float16)
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0] if r else None
    xs = F.smooth_act(X, s)
    Xq_ref, sc_ref = F.quant_act(xs)
    Xq, sc, T = aser.quant_act_ws(to_dev(X), to_dev(s), None if L_A is None else to_dev(L_A), t_pair=t_pair)
    assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
    if r:
        T_ref = F.down_proj(xs, L_A)
        if t_pair:
            assert_T_close(T[:, :r].float().cpu().numpy(), T_ref, xs, L_A)
            T_sum = T[:, :r].double().cpu().numpy() + T[:, r:].double().cpu().numpy()
            xs64, la64 = xs.astype(np.float64), L_A.astype(np.float64)
            tol = 2.0 ** -16 * np.abs(T_ref) + 2.0 ** -9.2 * np.sqrt((xs64 ** 2) @ (la64 ** 2).T) + \
                2.0 ** -20 * (np.abs(xs64) @ np.abs(la64).T) + 1e-30
            assert np.all(np.abs(T_sum - T_ref) <= tol)
        else:
            assert_T_close(T.float().cpu().numpy(), T_ref, xs, L_A)


def test_quant_act_ws_dense_smoothing_and_6_bits(aser):
    """Every divisor differs from 1, and 6-bit codes, through the two-kernel path."""
    M, K, r = 300, 1024, 64
    lay = synth.make_layer(M, 8, K, seed=471, n_cal=8)
    rng = np.random.default_rng(M + K)
    s = rng.uniform(0.25, 6.0, size=K).astype(np.float32)
    s[::7] = 1.0
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0]
    xs = F.smooth_act(lay.X, s)
    for bits_ in (8, 6):
        Xq_ref, sc_ref = F.quant_act(xs, act_bits=bits_)
        Xq, sc, T = aser.quant_act_ws(to_dev(lay.X), to_dev(s), to_dev(L_A), act_bits=bits_)
        assert np.array_equal(Xq.cpu().numpy(), Xq_ref)
        assert np.array_equal(bits(sc.cpu().numpy()), bits(sc_ref))
        assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A), xs, L_A)


# ---------------------------------------------------------------------------
# whole path: quant_act -> linear
# ---------------------------------------------------------------------------
def run_path(aser, lay, s, Wq_ref, w_scale_ref, L_A, L_B, impl, rows=None, use_dgemm=False,
             t_pair=False, timed_config=False, ws=None, ref=None):
    """Pack, quantize and multiply on the GPU, run the oracle on the same arrays, compare every
    stage.  `rows`: the oracle's products cover these token rows only (None = all).
    `t_pair`: T as bf16 pairs with the up projection written twice.  `timed_config`: the linear
    kernel runs once more without the accumulator dump (the configuration that is timed) and
    that output is compared with the oracle as well.  `ws`: a caller-owned workspace (reuse
    across calls).  `ref`: a precomputed oracle result for these inputs."""
    M, K = lay.X.shape
    N = lay.W.shape[0]
    r = 0 if L_A is None else L_A.shape[0]
    dW, ds = to_dev(lay.W), to_dev(s)
    Wq, wsc = aser.pack_w4(dW, ds)
    assert np.array_equal(Wq.cpu().numpy(), Wq_ref)
    assert np.array_equal(bits(wsc.cpu().numpy()), bits(w_scale_ref))
    del dW
    dLA = None if r == 0 else to_dev(L_A)
    dLB = None if r == 0 else to_dev(L_B)
    Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA, t_pair=t_pair)
    if t_pair:
        dLB = aser.pair_up_projection(dLB)
    r_lin = 2 * r if t_pair else r
    acc = torch.full((M, N), -7, dtype=torch.int32, device="cuda")
    Y_timed = None
    if impl == "simt":
        Y = aser.linear_w4a8_lr_simt(Xq, sc, Wq, wsc, T, dLB, acc_debug=acc)
    else:
        Wk = aser.repack_w4(Wq)
        if ws is None:
            ws = aser.new_workspace(M, N, K, r_lin)

        def call(acc_debug):
            if r:
                return aser.linear_w4a8_lr(Xq, sc, Wk, wsc, T, dLB, N, ws, acc_debug=acc_debug)
            return aser.linear_w4a8(Xq, sc, Wk, wsc, N, ws, acc_debug=acc_debug)
        Y = call(acc)
        if timed_config:
            Y_timed = call(None)
        aser.check_status(ws)
    torch.cuda.synchronize()
    if ref is None:
        ref = F.forward(lay.X, s, Wq_ref, w_scale_ref, L_A, L_B, rows=rows, use_dgemm=use_dgemm)
    assert np.array_equal(Xq.cpu().numpy(), ref.Xq)
    assert np.array_equal(bits(sc.cpu().numpy()), bits(ref.a_scale))
    acc_h = acc.cpu().numpy()
    assert np.array_equal(acc_h if rows is None else acc_h[rows], ref.acc)
    assert_rows_close(Y.cpu().numpy(), ref.y, rows)
    if Y_timed is not None:
        assert_rows_close(Y_timed.cpu().numpy(), ref.y, rows)
    return Y


PATH_CASES = [  # M, N, K, r
    (16, 512, 512, 16), (1, 256, 512, 16), (7, 136, 1024, 32), (33, 264, 512, 0),
    (130, 384, 1024, 64), (257, 520, 2048, 128), (40, 128, 384, 256),
    # 17..32 tokens: the 32-token tile of the tensor-core kernel
    (19, 264, 1024, 32), (32, 384, 512, 16), (17, 1152, 2048, 64),
]


@pytest.mark.parametrize("impl", ["simt", "tc"])
@pytest.mark.parametrize("M,N,K,r", PATH_CASES)
def test_path_parity_small(aser, impl, M, N, K, r):
    lay = synth.make_layer(M, N, K, seed=300 + M + N + K + r, n_cal=64,
                           n_out=max(1, K // 100))
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=(K <= 1024 and r > 0))
    if r == 0:
        L_A = L_B = None
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl, timed_config=(impl == "tc"))


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
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl, use_dgemm=True, timed_config=True)


@pytest.mark.parametrize("impl", ["tc"])
@pytest.mark.parametrize("which", ["gate_up", "down"])
def test_config3_prefill_full_size_all_rows(aser, impl, which):
    """Both prefill layers at full size: every accumulator bit-exact and every output element
    within the bound, with and without the accumulator dump (the timed configuration)."""
    lay, r = synth.config3_prefill(which)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, impl, use_dgemm=True, timed_config=True)


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


@pytest.mark.parametrize("name", ["q", "k", "gate", "down"])
def test_config4_block_linears_full_size_all_rows(aser, name):
    """Decoder-block linears at 4096 tokens, rank 128 (the square projection with eight whole
    tiles per CTA, the GQA projection, the widest and the deepest layer): every code, scale,
    accumulator and output element.  The widest layer also runs a 32-token call first on the
    workspace sized for 4096 tokens: one workspace serves calls of different shapes in turn."""
    lay, r = synth.config4_block_layer(name)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    ref = F.forward(lay.X, s, Wq, w_scale, L_A, L_B, use_dgemm=True)
    M, K = lay.X.shape
    N = lay.W.shape[0]
    ws = aser.new_workspace(M, N, K, r)
    if name == "gate":
        m = 32
        small = synth.LayerInputs(X=lay.X[:m], W=lay.W, X_cal=lay.X_cal, outlier_idx=lay.outlier_idx,
                                  outlier_gain=lay.outlier_gain, meta=lay.meta)
        ref_small = F.ForwardResult(xs=ref.xs[:m], Xq=ref.Xq[:m], a_scale=ref.a_scale[:m],
                                    acc=ref.acc[:m], T=ref.T[:m], y=ref.y[:m], rows=None)
        run_path(aser, small, s, Wq, w_scale, L_A, L_B, "tc", ws=ws, ref=ref_small)
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, "tc", ws=ws, ref=ref, timed_config=True)
    if name == "gate":     # and back to the small shape on the same workspace
        run_path(aser, small, s, Wq, w_scale, L_A, L_B, "tc", ws=ws, ref=ref_small)


C5_POINTS = [  # M, N, r, all rows?
    (1, 8192, 64, True), (16, 8192, 32, True), (16, 28672, 64, True), (128, 8192, 0, True),
    (128, 28672, 256, True), (1024, 8192, 128, True), (1024, 28672, 32, False),
    (4096, 8192, 128, True), (4096, 8192, 0, False), (4096, 28672, 64, True), (4096, 8192, 256, False),
]


@pytest.mark.parametrize("M,N,r,full", C5_POINTS)
def test_config5_sweep_points(aser, M, N, r, full):
    """Points of the 70B-class sweep (K = 8192): few tokens on both few-token paths (streaming
    kernel up to 64 MB of packed weights, tensor-core kernel above), rank 256 (two launches of
    the quantization cluster kernel), rank 0 (plain W4A8), and 4096 tokens at both widths
    compared on every row (the remaining points on token rows spread over every 128-token tile)."""
    lay = synth.config5_point(M, N)
    s, Wq, w_scale, L_A, L_B = oracle_layer(lay, r, construct=False)
    if r == 0:
        L_A = L_B = None
    rows = None
    if not full:
        base = np.arange(0, M, 128)
        rows = np.unique(np.concatenate([base, base + 127, base + 61]).clip(0, M - 1))
    run_path(aser, lay, s, Wq, w_scale, L_A, L_B, "tc", rows=rows, use_dgemm=True,
             timed_config=(M == 4096))


@pytest.mark.gpu
@pytest.mark.parametrize("M,N,K,r", [(4096, 8192, 8192, 256), (4096, 4096, 4096, 128), (2048, 1024, 14336, 192)])
def test_many_chunks_on_long_tiles_repeated_launches(aser, M, N, K, r):
    """Several low-rank chunks per 128-token tile on tiles long enough for the mid-tile schedule,
    several tiles per CTA, launched back to back: no bounded wait may give up (a chunk that is
    late must never make a role wait for something only a stalled role can provide) and every
    launch must give the same bits."""
    lay = synth.make_layer(M, N, K, seed=900 + r, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 16.0)
    L_A, L_B = synth.standin_factors(N, K, r, seed=3, scale_a=0.01, scale_b=0.01)
    L = aser.AserLinear(to_dev(lay.W), to_dev(s), to_dev(L_A), to_dev(L_B), M)
    X = to_dev(lay.X)
    first = L(X).clone()
    aser.check_status(L.ws)
    for rep in range(30):
        L.linear(M, True)
    torch.cuda.synchronize()
    aser.check_status(L.ws)
    assert torch.equal(L.Y[:M], first)
    for rep in range(10):
        Y = L(X)
    torch.cuda.synchronize()
    aser.check_status(L.ws)
    assert torch.equal(Y, first)


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
@pytest.mark.parametrize("M", [16, 200])
def test_paper_smoothing_rule_with_outlier_split_runs_through_the_same_path(aser, M):
    """The paper's own variant (Sec. 4.2): m_i = X-bar_i / min over the f outlier channels
    (Eq. 11), and the outlier columns W_o kept out of the int4 matrix and carried by the low-rank
    factors (Eq. 12).  For the GPU this is the same path with different inputs: the caller zeroes
    the outlier columns of W before packing.  The low-rank term is then as large as the output,
    so T is stored as bf16 pairs (aser_quant_act_ex); with that the output meets the same
    2e-3 * max|y_ref| bound as everywhere else.  Packed weights and accumulators bit-exact; and
    the split layer's output is closer to the fp product than plain W4A8 on the same codes.
    M = 16 takes the few-token kernels, M = 200 the tensor-core kernels."""
    from oracle import construct as Cn
    lay, r = synth.config1_tiny()
    if M != 16:
        lay = synth.make_layer(M, 512, 512, seed=synth.seed_for(1, M), n_out=4, outlier_gain=40.0,
                               sigma_w=0.02, n_cal=128)
    s, idx = Cn.smoothing_vector_paper(lay.X_cal, lay.W, f=4)
    assert np.array_equal(idx, lay.outlier_idx)
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r, split_outliers=idx)
    W_split = lay.W.copy()
    W_split[:, idx] = 0
    lay_split = synth.LayerInputs(X=lay.X, W=W_split, X_cal=lay.X_cal, outlier_idx=lay.outlier_idx,
                                  outlier_gain=lay.outlier_gain, meta=lay.meta)
    Y = run_path(aser, lay_split, s, L.Wq, L.w_scale, L.L_A, L.L_B, "tc", t_pair=True,
                 timed_config=True)
    plain = run_path(aser, lay_split, s, L.Wq, L.w_scale, None, None, "tc")
    ref = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    e_lr = np.linalg.norm(Y.cpu().numpy().astype(np.float64) - ref)
    e_plain = np.linalg.norm(plain.cpu().numpy().astype(np.float64) - ref)
    assert e_lr < 0.5 * e_plain        # without the factors the outlier columns are simply missing


@pytest.mark.gpu
@pytest.mark.parametrize("M,K,r", [(8, 1024, 16), (300, 2048, 64), (129, 4096, 128), (40, 512, 48)])
def test_quant_act_pair_storage_of_T(aser, M, K, r):
    """aser_quant_act_ex with t_pair: hi + lo reproduces the fp64 projection to 2^-16 of each
    entry (plus the fp16 rounding of x~ inside the tensor-core product), codes and scales are
    those of the plain call, and hi is the plain call's T."""
    lay = synth.make_layer(M, 8, K, seed=800 + M + K + r, n_cal=8)
    s = synth.standin_smoothing_vector(K, lay.outlier_idx, 13.0)
    L_A = synth.standin_factors(8, K, r, seed=M, scale_a=0.05)[0]
    dX, ds, dLA = to_dev(lay.X), to_dev(s), to_dev(L_A)
    Xq0, sc0, T0 = aser.quant_act(dX, ds, dLA)
    Xq, sc, T = aser.quant_act(dX, ds, dLA, t_pair=True)
    assert T.shape == (M, 2 * r)
    assert torch.equal(Xq, Xq0) and torch.equal(sc, sc0)
    assert torch.equal(T[:, :r].contiguous().view(torch.int16), T0.view(torch.int16))
    xs = F.smooth_act(lay.X, s)
    T_ref = F.down_proj(xs, L_A)
    T_sum = T[:, :r].double().cpu().numpy() + T[:, r:].double().cpu().numpy()
    xs64, la64 = xs.astype(np.float64), L_A.astype(np.float64)
    rms = np.sqrt((xs64 ** 2) @ (la64 ** 2).T)
    l1 = np.abs(xs64) @ np.abs(la64).T
    tol = 2.0 ** -16 * np.abs(T_ref) + 2.0 ** -9.2 * rms * (M > 32) + 2.0 ** -20 * l1 + 1e-30
    assert np.all(np.abs(T_sum - T_ref) <= tol)
    with pytest.raises(aser.AserError) as err:      # 2 r beyond the kernels' 256
        aser.quant_act(dX, ds, to_dev(synth.standin_factors(8, K, 144, seed=1)[0]), t_pair=True)
    assert err.value.code == -3


@pytest.mark.gpu
def test_rank_from_threshold_end_to_end(aser):
    """Sec. 4.1 Eq. 9 end to end: the oracle picks the rank from the singular-value threshold
    alpha (any integer, here not a multiple of 16), pad_rank brings the factors to the kernels'
    granularity, and the GPU output matches the oracle run on the UNPADDED factors."""
    from oracle import construct as Cn
    lay = synth.make_layer(48, 384, 512, seed=synth.seed_for(1, 77), n_out=5, outlier_gain=40.0, n_cal=256)
    s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
    seen = set()
    for alpha in (0.05, 0.12, 0.3):
        L = Cn.construct_layer(lay.W, lay.X_cal, s, r=None, alpha=alpha)
        r = L.L_A.shape[0]
        assert r == Cn.rank_from_alpha(L.sigma, alpha) and 0 < r < 256
        seen.add(r % 16 != 0)
        dLA, dLB = aser.pad_rank(to_dev(L.L_A), to_dev(L.L_B))
        ds = to_dev(s)
        Wq, wsc = aser.pack_w4(to_dev(lay.W), ds)
        assert np.array_equal(Wq.cpu().numpy(), L.Wq)
        Xq, sc, T = aser.quant_act(to_dev(lay.X), ds, dLA)
        ws = aser.new_workspace(48, 384, 512, dLA.shape[0])
        acc = torch.zeros((48, 384), dtype=torch.int32, device="cuda")
        Y = aser.linear_w4a8_lr(Xq, sc, aser.repack_w4(Wq), wsc, T, dLB, 384, ws, acc_debug=acc)
        aser.check_status(ws)
        ref = F.forward(lay.X, s, L.Wq, L.w_scale, L.L_A, L.L_B)
        assert np.array_equal(acc.cpu().numpy(), ref.acc)
        assert_rows_close(Y.cpu().numpy(), ref.y)
    assert True in seen                 # at least one rank that needed padding


@pytest.mark.gpu
def test_status_word_reports_a_timeout_and_clears(aser):
    """aser_check_status without any kernel timing out: a status word planted by a memset must
    come back as ASER_ERR_DEVICE_TIMEOUT once, then the workspace is clean (word and counters)."""
    ws = aser.new_workspace(64, 256, 512, 16)
    aser.check_status(ws)
    ws[0] = 1
    ws[256:260] = 3                     # a tile counter left behind by the same launch
    with pytest.raises(aser.AserError) as err:
        aser.check_status(ws)
    assert err.value.code == -6 and "status word" in str(err.value)
    aser.check_status(ws)
    assert int(ws[:1024].to(torch.int32).sum()) == 0


SHARED_CASES = [  # M, K, [(N, r), ...]
    (8, 1024, [(256, 32), (128, 16), (128, 16)]),
    (8, 1024, [(256, 32), (128, 32), (384, 32), (128, 32)]),
    (16, 2048, [(1024, 64), (256, 64)]),
    (200, 1024, [(384, 64), (128, 64)]),
    (1100, 1024, [(256, 128), (128, 128), (128, 128)]),
    (200, 1024, [(384, 64), (136, 48), (128, 0)]),
    (300, 2048, [(512, 128), (256, 128), (256, 128)]),
]


@pytest.mark.gpu
@pytest.mark.parametrize("M,K,spec", SHARED_CASES)
def test_forward_shared_matches_oracle_per_layer(aser, M, K, spec):
    """aser_forward_shared: one activation pass for layers that read the same X.  Codes and
    scales bit-exact; every layer's output within the bound of the oracle run on that layer
    alone; and the stacked T agrees with the per-layer T of each layer's own activation step."""
    check_shared_group(aser, M, K, spec, seed0=1200 + M + K, construct=False)


def check_shared_group(aser, M, K, spec, seed0, construct, gain=30.0):
    base = synth.make_layer(M, spec[0][0], K, seed=seed0, n_cal=64, n_out=max(1, K // 100), outlier_gain=gain)
    s = synth.standin_smoothing_vector(K, base.outlier_idx, 11.0)
    ds = to_dev(s)
    layers, refs = [], []
    for li, (N, r) in enumerate(spec):
        rng = np.random.default_rng(seed0 + 17 * li + 1)
        W = (rng.standard_normal((N, K), dtype=np.float32) * np.float32(0.02)).astype(np.float16)
        q, w_scale = F.quant_w4(W, s)
        L_A, L_B = synth.standin_factors(N, K, max(r, 16), seed=seed0 + li, scale_a=0.01, scale_b=0.01)
        L_A, L_B = (L_A[:r], np.ascontiguousarray(L_B[:, :r])) if r else (None, None)
        lay = aser.AserLinear(to_dev(W), ds, None if r == 0 else to_dev(L_A), None if r == 0 else to_dev(L_B), M)
        assert np.array_equal(lay.Wq.cpu().numpy(), F.pack_w4(q))
        layers.append(lay)
        refs.append(F.forward(base.X, s, F.pack_w4(q), w_scale, L_A, L_B, use_dgemm=True))
    group = aser.AserSharedInput(layers, M)
    X = to_dev(base.X)
    for rep in range(2):                    # twice: the workspace is reused
        Ys = group(X)
        aser.check_status(group.ws)
        torch.cuda.synchronize()
        assert np.array_equal(group.Xq[:M].cpu().numpy(), refs[0].Xq)
        assert np.array_equal(bits(group.a_scale[:M].cpu().numpy()), bits(refs[0].a_scale))
        col = 0
        for lay, ref, Y in zip(layers, refs, Ys):
            assert_rows_close(Y.cpu().numpy(), ref.y)
            if lay.r:
                # the layer's own activation step may run other kernels (another summation
                # order): equal up to the last bf16 bit wherever T is not a cancellation
                lay.quant(X)
                a = group.T[:M, col:col + lay.r].float()
                b = lay.T[:M].float()
                assert bool(((a - b).abs() <= 2.0 ** -7 * b.abs() + 2.0 ** -9 * b.abs().max()).all())
                col += lay.r
    # the same group stored as one fused projection (one linear launch over the concatenated N)
    ranks = {r for _, r in spec}
    if len(ranks) == 1 and all(N % 128 == 0 for N, _ in spec) and len(spec) <= 4:
        per_layer = [y.clone() for y in group(X)]
        cat = aser.AserSharedInputCat(layers, M)
        for rep in range(2):
            Ys = cat(X)
            aser.check_status(cat.ws)
            torch.cuda.synchronize()
            assert np.array_equal(cat.Xq[:M].cpu().numpy(), refs[0].Xq)
            for ref, Y, Y1 in zip(refs, Ys, per_layer):
                assert_rows_close(Y.cpu().numpy(), ref.y)
                # same operands, same arithmetic per element as the layer's own launch
                assert torch.equal(Y, Y1)
        Ys = cat.linear(M)                  # the linear step alone on the codes already there
        torch.cuda.synchronize()
        for ref, Y in zip(refs, Ys):
            assert_rows_close(Y.cpu().numpy(), ref.y)


@pytest.mark.gpu
@pytest.mark.parametrize("which", ["qkv", "gate_up"])
def test_forward_shared_decoder_block_groups_full_size(aser, which):
    """The two shared-input groups of the decoder block at 4096 tokens, rank 128: query/key/value
    (384 stacked rows) and gate/up (256)."""
    spec = [(4096, 128), (1024, 128), (1024, 128)] if which == "qkv" else [(14336, 128), (14336, 128)]
    check_shared_group(aser, 4096, 4096, spec, seed0=synth.seed_for(4, 50 + len(spec)), construct=False)


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
        assert_T_close(T.float().cpu().numpy(), F.down_proj(xs, L_A), xs, L_A)


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
