"""Pins for the oracle's forward pass: closed forms, hand-built ties, brute force,
special cases.  None of these re-derive an expected value from the oracle itself."""
import numpy as np
import pytest

from oracle import forward as F
import aser_synth as synth


# ---------------------------------------------------------------------------
# fp16 decoding and smoothing
# ---------------------------------------------------------------------------

def test_f16_decode_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16).reshape(256, 256)
    h = bits.view(np.float16)
    got = F.smooth_act(h, None)
    want = h.astype(np.float32)            # library conversion
    assert np.array_equal(got.view(np.uint32)[~np.isnan(want)], want.view(np.uint32)[~np.isnan(want)])
    assert np.all(np.isnan(got[np.isnan(want)]))


def test_smoothing_divides_each_channel():
    X = np.array([[1.0, 3.0, -10.0, 0.5]], np.float16)
    s = np.array([1.0, 2.0, 4.0, 0.25], np.float32)
    assert np.array_equal(F.smooth_act(X, s), np.array([[1.0, 1.5, -2.5, 2.0]], np.float32))


def test_smoothing_identity_fp64():
    """W diag(s) diag(s)^-1 X = W X  (Eq. 10 of Sec. 4.2)."""
    rng = np.random.default_rng(1)
    X = rng.standard_normal((8, 64)).astype(np.float16)
    W = (rng.standard_normal((32, 64)) * 0.02).astype(np.float16)
    s = np.exp(rng.standard_normal(64)).astype(np.float32)
    X64, W64, s64 = X.astype(np.float64), W.astype(np.float64), s.astype(np.float64)
    ref = X64 @ W64.T
    exact = (X64 / s64) @ (W64 * s64).T
    assert np.max(np.abs(exact - ref)) <= 1e-14 * np.max(np.abs(ref)) * 64
    # the oracle's fp32 smoothed operands reproduce the product to fp32 rounding
    xs = F.smooth_act(X, s)
    _, _, ws = F.quant_w4(W, s, want_ws=True)
    got = xs.astype(np.float64) @ ws.astype(np.float64).T
    assert np.max(np.abs(got - ref)) <= 3e-7 * np.sum(np.abs(X64[:, None, :] * W64[None]), axis=2).max()


# ---------------------------------------------------------------------------
# int8 per-token quantizer
# ---------------------------------------------------------------------------

def test_int8_half_to_even_ties():
    # absmax 127 -> scale exactly 1 -> codes are rne(x)
    row = np.array([127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 126.5, -126.5], np.float32)[None]
    Xq, sc = F.quant_act(row)
    assert sc[0] == np.float32(1.0)
    assert Xq[0].tolist() == [127, 0, 2, 2, 0, -2, -2, 4, 126, -126]


def test_int8_scale_is_one_fp32_division():
    row = np.array([[0.1, -3.3, 2.2]], np.float32)
    _, sc = F.quant_act(row)
    assert sc[0] == np.float32(3.3) / np.float32(127.0)


def test_int8_zero_row_and_range():
    rng = np.random.default_rng(2)
    xs = rng.standard_normal((5, 257)).astype(np.float32) * 7
    xs[3] = 0.0
    Xq, sc = F.quant_act(xs)
    assert sc[3] == 0.0 and not Xq[3].any()
    assert Xq.min() >= -127 and Xq.max() <= 127
    for m in (0, 1, 2, 4):
        k = np.argmax(np.abs(xs[m]))
        assert abs(int(Xq[m, k])) == 127 and np.sign(Xq[m, k]) == np.sign(xs[m, k])
        err = np.abs(xs[m].astype(np.float64) - Xq[m].astype(np.float64) * float(sc[m]))
        assert err.max() <= 0.5 * float(sc[m]) * (1 + 1e-6)


def test_int8_negative_extreme_not_minus_128():
    row = np.array([[-5.0, 1.0]], np.float32)
    Xq, _ = F.quant_act(row)
    assert Xq[0].tolist() == [-127, 25]      # 1/(5/127) = 25.4 -> 25


# ---------------------------------------------------------------------------
# 6-bit activation codes (the W4A6 setting, Sec. 5.2)
# ---------------------------------------------------------------------------

def test_6bit_codes_by_hand():
    # absmax 31 -> scale exactly 1 -> codes are rne(x), half to even
    row = np.array([31.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.5, 30.5, -30.5], np.float32)[None]
    Xq, sc = F.quant_act(row, act_bits=6)
    assert sc[0] == np.float32(1.0)
    assert Xq[0].tolist() == [31, 0, 2, 2, 0, -2, -2, 4, 30, -30]
    # the scale is one fp32 division by 31; the negative extreme maps to -31, never -32
    row = np.array([[-5.0, 1.0, 0.1]], np.float32)
    Xq, sc = F.quant_act(row, act_bits=6)
    assert sc[0] == np.float32(5.0) / np.float32(31.0)
    assert Xq[0].tolist() == [-31, 6, 1]     # 1/(5/31) = 6.2 -> 6, 0.1/(5/31) = 0.62 -> 1


def test_6bit_range_error_bound_and_8bit_unchanged():
    rng = np.random.default_rng(6)
    xs = rng.standard_normal((4, 300)).astype(np.float32) * 3
    xs[2] = 0.0
    Xq, sc = F.quant_act(xs, act_bits=6)
    assert sc[2] == 0.0 and not Xq[2].any()
    assert Xq.min() >= -31 and Xq.max() <= 31
    for m in (0, 1, 3):
        k = np.argmax(np.abs(xs[m]))
        assert abs(int(Xq[m, k])) == 31
        err = np.abs(xs[m].astype(np.float64) - Xq[m].astype(np.float64) * float(sc[m]))
        assert err.max() <= 0.5 * float(sc[m]) * (1 + 1e-6)
    # 8 bits through the general routine is the W4A8 quantizer bit for bit
    Xq8, sc8 = F.quant_act(xs)
    Xq8b = np.empty_like(Xq8)
    sc8b = np.empty_like(sc8)
    F._lib.aser_oracle_quant_act_bits(F._ptr(xs), xs.shape[0], xs.shape[1], 8, F._ptr(Xq8b), F._ptr(sc8b))
    assert np.array_equal(Xq8, Xq8b) and np.array_equal(sc8.view(np.uint32), sc8b.view(np.uint32))
    # coarser codes, larger error: the 6-bit step is 127/31 of the 8-bit one
    assert np.allclose(sc[[0, 1, 3]] / sc8[[0, 1, 3]], 127.0 / 31.0, rtol=1e-6)


def test_6bit_forward_is_the_same_formula_with_coarser_codes():
    rng = np.random.default_rng(7)
    M, N, K = 3, 8, 64
    X = rng.standard_normal((M, K)).astype(np.float16)
    W = (rng.standard_normal((N, K)) * 0.05).astype(np.float16)
    q, w_scale = F.quant_w4(W, None)
    out = F.forward(X, None, F.pack_w4(q), w_scale, act_bits=6)
    xq, sc = F.quant_act(X.astype(np.float32), act_bits=6)
    brute = np.zeros((M, N))
    for m in range(M):
        for n in range(N):
            acc = sum(int(xq[m, k]) * int(q[n, k]) for k in range(K))
            brute[m, n] = acc * float(sc[m]) * float(w_scale[n])
    assert np.allclose(out.y, brute, rtol=1e-12, atol=1e-12)
    # against the product with the SAME int4 weights (so that only the activation codes differ)
    # the 6-bit pass is the coarser approximation, by about the ratio of the steps
    ref = X.astype(np.float64) @ (q.astype(np.float64) * w_scale.astype(np.float64)[:, None]).T
    out8 = F.forward(X, None, F.pack_w4(q), w_scale)
    e6, e8 = np.linalg.norm(out.y - ref), np.linalg.norm(out8.y - ref)
    assert 2.0 * e8 < e6 < 8.0 * e8


# ---------------------------------------------------------------------------
# int4 per-output-channel quantizer
# ---------------------------------------------------------------------------

def test_int4_half_to_even_ties_and_scale():
    # absmax 7 -> scale exactly 1
    W = np.array([[7.0, 0.5, 1.5, 2.5, -2.5, 6.5, -6.5, -7.0]], np.float16)
    q, sc = F.quant_w4(W, None)
    assert sc[0] == np.float32(1.0)
    assert q[0].tolist() == [7, 0, 2, 2, -2, 6, -6, -7]


def test_int4_smoothing_multiplies_columns():
    W = np.array([[1.0, 1.0, -0.5, 0.25]], np.float16)
    s = np.array([1.0, 7.0, 2.0, 4.0], np.float32)     # ws = [1, 7, -1, 1], scale 1
    q, sc, ws = F.quant_w4(W, s, want_ws=True)
    assert ws[0].tolist() == [1.0, 7.0, -1.0, 1.0]
    assert sc[0] == 1.0 and q[0].tolist() == [1, 7, -1, 1]


def test_int4_range_error_bound_and_extreme():
    lay = synth.make_layer(4, 48, 256, seed=11, n_out=3)
    s = synth.standin_smoothing_vector(256, lay.outlier_idx, 9.0)
    q, sc, ws = F.quant_w4(lay.W, s, want_ws=True)
    assert q.min() >= -8 and q.max() <= 7
    err = np.abs(ws.astype(np.float64) - q.astype(np.float64) * sc.astype(np.float64)[:, None])
    assert np.all(err <= 0.5 * sc.astype(np.float64)[:, None] * (1 + 1e-6))
    k = np.argmax(np.abs(ws), axis=1)
    assert np.all(np.abs(q[np.arange(48), k]) == 7)
    assert np.array_equal(sc, np.abs(ws).max(axis=1) / np.float32(7.0))


def test_int4_quantize_dequantize_idempotent():
    """Q(deq(Q(w))) = Q(w).  Rows are given power-of-two scales so that the
    dequantized values are exactly representable in the fp16 input type."""
    rng = np.random.default_rng(3)
    N, K = 16, 64
    W = np.zeros((N, K), np.float32)
    for n in range(N):
        e = rng.integers(-8, 3)
        row = rng.uniform(-6.9, 6.9, K) * 2.0 ** e
        row[rng.integers(K)] = 7.0 * 2.0 ** e * rng.choice([-1, 1])
        W[n] = row
    W16 = W.astype(np.float16)
    q, sc = F.quant_w4(W16, None)
    deq = (q.astype(np.float32) * sc[:, None]).astype(np.float16)
    assert np.array_equal(deq.astype(np.float32), q.astype(np.float32) * sc[:, None])
    q2, sc2 = F.quant_w4(deq, None)
    assert np.array_equal(q2, q) and np.array_equal(sc2, sc)


def test_int4_zero_row():
    W = np.zeros((2, 8), np.float16)
    W[1, 3] = 1.0
    q, sc = F.quant_w4(W, None)
    assert sc[0] == 0.0 and not q[0].any() and q[1, 3] == 7


def test_pack_layout_and_roundtrip():
    q = np.array([[-8, 7, 1, -1]], np.int8)
    p = F.pack_w4(q)
    assert p.tolist() == [[0x78, 0xF1]]       # low nibble = even k, high nibble = odd k
    allb = np.arange(256, dtype=np.uint8).reshape(4, 64)
    un = F.unpack_w4(allb)
    assert un.min() == -8 and un.max() == 7
    assert np.array_equal(F.pack_w4(un), allb)
    lo = (allb & 0xF).astype(np.int16)
    assert np.array_equal(un[:, 0::2], np.where(lo >= 8, lo - 16, lo))


# ---------------------------------------------------------------------------
# integer product, low-rank branch, dequantisation
# ---------------------------------------------------------------------------

def _brute_int(Xq, q):
    M, K = Xq.shape
    N = q.shape[0]
    out = [[0] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = 0
            for k in range(K):
                acc += int(Xq[m, k]) * int(q[n, k])
            out[m][n] = acc
    return np.array(out, np.int64)


def test_int_matmul_brute_force_tiny():
    rng = np.random.default_rng(4)
    Xq = rng.integers(-127, 128, (5, 37)).astype(np.int8)
    q = rng.integers(-8, 8, (7, 37)).astype(np.int8)
    want = _brute_int(Xq, q)
    assert np.array_equal(F.int_matmul(Xq, q), want)
    assert np.array_equal(F.int_matmul_dgemm(Xq, q), want)
    assert np.array_equal(F.int_matmul(Xq, q, rows=[4, 0]), want[[4, 0]])
    # a transposed-operand mistake would need matching shapes; rule it out explicitly
    sq = rng.integers(-8, 8, (37, 37)).astype(np.int8)
    xsq = rng.integers(-127, 128, (37, 37)).astype(np.int8)
    assert np.array_equal(F.int_matmul(xsq, sq), _brute_int(xsq, sq))


def test_int_matmul_extremes_do_not_overflow():
    K = 28672
    Xq = np.full((1, K), -127, np.int8)
    q = np.full((2, K), -8, np.int8)
    q[1] = 7
    acc = F.int_matmul(Xq, q)
    assert acc.tolist() == [[127 * 8 * K, -127 * 7 * K]]


def test_int_matmul_dgemm_equals_loops_midsize():
    rng = np.random.default_rng(5)
    Xq = rng.integers(-127, 128, (33, 1024)).astype(np.int8)
    q = rng.integers(-8, 8, (130, 1024)).astype(np.int8)
    assert np.array_equal(F.int_matmul(Xq, q), F.int_matmul_dgemm(Xq, q))


def test_down_proj_and_dequant_tiny_by_hand():
    xs = np.array([[1.0, 2.0, -1.0], [0.5, 0.0, 4.0]], np.float32)
    L_A = np.array([[1.0, 0.5, 0.25], [0.0, -2.0, 1.0]], np.float16)      # [r=2, K=3]
    T = F.down_proj(xs, L_A)
    assert T.tolist() == [[1.75, -5.0], [1.5, 4.0]]
    L_B = np.array([[2.0, 1.0], [0.0, 0.5], [-1.0, 0.0]], np.float16)     # [N=3, r=2]
    acc = np.array([[10, -20, 30], [1, 2, 3]], np.int32)
    a_scale = np.array([0.5, 2.0], np.float32)
    w_scale = np.array([1.0, 0.25, 2.0], np.float32)
    y = F.dequant_add(acc, a_scale, w_scale, T, L_B)
    want = [[10 * .5 * 1 + (2 * 1.75 - 5.0), -20 * .5 * .25 + (-2.5), 30 * .5 * 2 - 1.75],
            [1 * 2 * 1 + (3.0 + 4.0), 2 * 2 * .25 + 2.0, 3 * 2 * 2 - 1.5]]
    assert y.tolist() == want
    assert np.array_equal(F.down_proj(xs, L_A, rows=[1]), T[[1]])


def test_down_proj_matches_library_matmul():
    rng = np.random.default_rng(6)
    xs = rng.standard_normal((9, 300)).astype(np.float32)
    L_A = (rng.standard_normal((16, 300)) * 0.1).astype(np.float16)
    want = xs.astype(np.float64) @ L_A.astype(np.float64).T
    assert np.allclose(F.down_proj(xs, L_A), want, rtol=0, atol=1e-12)


def _tiny_layer(r):
    lay = synth.make_layer(6, 24, 64, seed=21, n_out=2, outlier_gain=30.0, n_cal=16)
    s = synth.standin_smoothing_vector(64, lay.outlier_idx, 8.0)
    q, w_scale = F.quant_w4(lay.W, s)
    L_A, L_B = synth.standin_factors(24, 64, r, seed=5)
    return lay, s, F.pack_w4(q), w_scale, L_A, L_B


def test_rank_zero_is_plain_w4a8_bit_for_bit():
    lay, s, Wq, w_scale, _, _ = _tiny_layer(16)
    plain = F.forward(lay.X, s, Wq, w_scale)
    r0 = F.forward(lay.X, s, Wq, w_scale, np.zeros((0, 64), np.float16), np.zeros((24, 0), np.float16))
    assert np.array_equal(plain.y.view(np.uint64), r0.y.view(np.uint64))
    # and the plain product is acc * a_scale * w_scale
    want = plain.acc.astype(np.float64) * plain.a_scale.astype(np.float64)[:, None] \
        * w_scale.astype(np.float64)[None]
    assert np.array_equal(plain.y, want)


def test_forward_row_subset_and_dgemm_agree():
    lay, s, Wq, w_scale, L_A, L_B = _tiny_layer(16)
    full = F.forward(lay.X, s, Wq, w_scale, L_A, L_B)
    sub = F.forward(lay.X, s, Wq, w_scale, L_A, L_B, rows=[5, 2], use_dgemm=True)
    assert np.array_equal(sub.y, full.y[[5, 2]])
    assert np.array_equal(sub.acc, full.acc[[5, 2]])


def test_forward_lowrank_term_is_additive_and_linear():
    lay, s, Wq, w_scale, L_A, L_B = _tiny_layer(16)
    plain = F.forward(lay.X, s, Wq, w_scale)
    lr = F.forward(lay.X, s, Wq, w_scale, L_A, L_B)
    delta = lr.y - plain.y
    want = (lr.xs.astype(np.float64) @ L_A.astype(np.float64).T) @ L_B.astype(np.float64).T
    assert np.allclose(delta, want, rtol=0, atol=1e-9 * np.abs(want).max() + 1e-12)


def test_openmp_threads_do_not_change_results():
    lay, s, Wq, w_scale, L_A, L_B = _tiny_layer(16)
    a = F.forward(lay.X, s, Wq, w_scale, L_A, L_B)
    F.set_threads(min(4, F.max_threads()))
    try:
        b = F.forward(lay.X, s, Wq, w_scale, L_A, L_B)
    finally:
        F.set_threads(1)
    assert np.array_equal(a.y, b.y) and np.array_equal(a.Xq, b.Xq)
