"""Pins for the oracle's construction part (smoothing vector, whitening SVD, rank rule,
overhead model) against closed forms, invariants, hand-written textbook routines and the
paper's printed overhead table."""
import os

import numpy as np
import pytest

from oracle import construct as Cn
from oracle import forward as F
import aser_synth as synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------
# textbook routines written out by hand, used to pin the library calls
# ---------------------------------------------------------------------------

def chol_by_hand(A):
    n = A.shape[0]
    L = np.zeros_like(A)
    for j in range(n):
        d = A[j, j] - sum(L[j, k] ** 2 for k in range(j))
        L[j, j] = d ** 0.5
        for i in range(j + 1, n):
            L[i, j] = (A[i, j] - sum(L[i, k] * L[j, k] for k in range(j))) / L[j, j]
    return L


def jacobi_singular_values(A, sweeps=60):
    """One-sided Jacobi: rotate column pairs until orthogonal; column norms are the sigmas."""
    U = A.astype(np.float64).copy()
    n = U.shape[1]
    for _ in range(sweeps):
        off = 0.0
        for p in range(n - 1):
            for q in range(p + 1, n):
                a, b, c = U[:, p] @ U[:, p], U[:, q] @ U[:, q], U[:, p] @ U[:, q]
                off = max(off, abs(c) / max((a * b) ** 0.5, 1e-300))
                if abs(c) < 1e-300:
                    continue
                zeta = (b - a) / (2 * c)
                t = np.sign(zeta) / (abs(zeta) + (1 + zeta * zeta) ** 0.5) if zeta != 0 else 1.0
                cs = 1 / (1 + t * t) ** 0.5
                sn = cs * t
                up, uq = U[:, p].copy(), U[:, q].copy()
                U[:, p], U[:, q] = cs * up - sn * uq, sn * up + cs * uq
        if off < 1e-15:
            break
    return np.sort(np.linalg.norm(U, axis=0))[::-1]


@pytest.fixture(scope="module")
def small_layer():
    lay = synth.make_layer(8, 40, 48, seed=31, n_out=2, outlier_gain=30.0, n_cal=24)
    s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
    return lay, s


def test_cholesky_and_svd_match_hand_written(small_layer):
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=8)
    G = Cn.gram(F.smooth_act(lay.X_cal, s))
    assert np.allclose(L.S, chol_by_hand(G + L.lam * np.eye(48)), rtol=1e-10, atol=1e-12)
    assert np.allclose(L.sigma, jacobi_singular_values((L.E @ L.S).T if 40 < 48 else L.E @ L.S)[:len(L.sigma)],
                       rtol=1e-9, atol=1e-12)


def test_whitening_makes_identity(small_layer):
    """S^-1 (X X^T) S^-T = I  (Eq. 5), with the damped Gram matrix."""
    lay, s = small_layer
    G = Cn.gram(F.smooth_act(lay.X_cal, s))
    S, lam = Cn.whitening_factor(G)
    assert lam == pytest.approx(0.01 * np.trace(G) / 48)
    Si = np.linalg.inv(S)
    assert np.allclose(Si @ (G + lam * np.eye(48)) @ Si.T, np.eye(48), atol=1e-9)
    assert np.allclose(S, np.tril(S))


def test_gram_orientation_is_channels_by_channels():
    A = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]], np.float32)     # 3 tokens, 2 channels
    assert Cn.gram(A).tolist() == [[35.0, 44.0], [44.0, 56.0]]


@pytest.mark.parametrize("r", [0, 1, 5, 16, 40])
def test_truncation_loss_is_tail_of_singular_values(small_layer, r):
    """Dropping triplet i costs exactly sigma_i in the whitened norm (Eq. 8), hence
    ||(E - L_B L_A) S||_F^2 = sum_{i>r} sigma_i^2, which in data space reads
    ||(E - L_B L_A) X~^T||_F^2 + lambda ||E - L_B L_A||_F^2."""
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
    R = L.E - L.L_B64 @ L.L_A64
    tail = float(np.sum(L.sigma[r:] ** 2))
    assert np.linalg.norm(R @ L.S) ** 2 == pytest.approx(tail, rel=1e-8, abs=1e-18)
    Xs = F.smooth_act(lay.X_cal, s).astype(np.float64)
    data = np.linalg.norm(R @ Xs.T) ** 2 + L.lam * np.linalg.norm(R) ** 2
    assert data == pytest.approx(tail, rel=1e-7, abs=1e-18)


def test_single_triplet_costs_its_singular_value(small_layer):
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=40)
    U, sig, Vt = Cn.whitened_svd(L.E, L.S)
    i = 3
    Si = np.linalg.inv(L.S)
    drop = sig[i] * np.outer(U[:, i], Vt[i]) @ Si
    assert np.linalg.norm(drop @ L.S) == pytest.approx(sig[i], rel=1e-9)


def test_eckart_young_beats_plain_svd_and_random(small_layer):
    lay, s = small_layer
    r = 6
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
    ours = np.linalg.norm((L.E - L.L_B64 @ L.L_A64) @ L.S)
    U, sg, Vt = np.linalg.svd(L.E, full_matrices=False)
    plain = (U[:, :r] * sg[:r]) @ Vt[:r]                  # weight-only truncation
    assert ours <= np.linalg.norm((L.E - plain) @ L.S) * (1 + 1e-12)
    rng = np.random.default_rng(0)
    rand = rng.standard_normal((40, r)) @ rng.standard_normal((r, 48)) * 1e-3
    assert ours <= np.linalg.norm((L.E - rand) @ L.S)
    prev = np.inf
    for rr in range(0, 41, 5):
        Lr = Cn.construct_layer(lay.W, lay.X_cal, s, r=rr)
        cur = np.linalg.norm((Lr.E - Lr.L_B64 @ Lr.L_A64) @ Lr.S)
        assert cur <= prev + 1e-15
        prev = cur


def test_full_rank_recovers_smoothed_weight(small_layer):
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=40)
    deq = L.q.astype(np.float64) * L.w_scale.astype(np.float64)[:, None]
    assert np.allclose(deq + L.L_B64 @ L.L_A64, L.ws.astype(np.float64), rtol=0, atol=1e-10)
    # forward with the (fp16-rounded) full-rank factors ~ smoothed fp product; the remaining
    # error is activation quantization + fp16 rounding of the factors only
    res = F.forward(lay.X, s, L.Wq, L.w_scale, L.L_A, L.L_B)
    plain = F.forward(lay.X, s, L.Wq, L.w_scale)
    ref = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    e_full = np.linalg.norm(res.y - ref)
    e_plain = np.linalg.norm(plain.y - ref)
    assert e_full < 0.25 * e_plain
    assert e_full < 0.02 * np.linalg.norm(ref)


def test_factor_product_independent_of_whitening_root(small_layer):
    """Any S with S S^T = G + lambda I gives the same L_B L_A (sigma_r > sigma_{r+1})."""
    lay, s = small_layer
    r = 7
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
    A = L.S @ L.S.T
    w, Q = np.linalg.eigh(A)
    root = (Q * np.sqrt(w)) @ Q.T                       # symmetric square root
    U, sig, Vt = np.linalg.svd(L.E @ root, full_matrices=False)
    alt = (U[:, :r] * sig[:r]) @ Vt[:r] @ np.linalg.inv(root)
    assert np.allclose(sig, L.sigma, rtol=1e-8)
    assert np.allclose(alt, L.L_B64 @ L.L_A64, atol=1e-8 * np.abs(alt).max())
    # and scaling S leaves it unchanged
    U, sig, Vt = np.linalg.svd(L.E @ (3 * L.S), full_matrices=False)
    alt = (U[:, :r] * sig[:r]) @ Vt[:r] @ np.linalg.inv(3 * L.S)
    assert np.allclose(alt, L.L_B64 @ L.L_A64, atol=1e-8 * np.abs(alt).max())


def test_factor_shapes_dtypes_and_r0(small_layer):
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=16)
    assert L.L_A.shape == (16, 48) and L.L_B.shape == (40, 16)
    assert L.L_A.dtype == np.float16 and L.L_B.dtype == np.float16
    assert L.Wq.shape == (40, 24) and L.Wq.dtype == np.uint8
    L0 = Cn.construct_layer(lay.W, lay.X_cal, s, r=0)
    assert L0.L_A.shape == (0, 48) and L0.L_B.shape == (40, 0)
    # no smoothing reduces to plain round-to-nearest of W (Alg. 1, else branch)
    Ln = Cn.construct_layer(lay.W, lay.X_cal, None, r=0)
    qn, scn = F.quant_w4(lay.W, None)
    assert np.array_equal(Ln.q, qn) and np.array_equal(Ln.w_scale, scn)


# ---------------------------------------------------------------------------
# smoothing vector and outlier set
# ---------------------------------------------------------------------------

def test_outlier_rule_recovers_seeded_channels():
    for lay in (synth.config1_tiny()[0],
                synth.make_layer(4, 64, 1024, seed=77, outlier_gain=30.0, n_cal=256)):
        f = len(lay.outlier_idx)
        assert np.array_equal(Cn.outlier_index_set(lay.X_cal, lay.W, f), lay.outlier_idx)


def test_outlier_rule_ties_go_to_lower_index():
    X = np.ones((2, 4), np.float16)
    W = np.ones((3, 4), np.float16)
    assert Cn.outlier_index_set(X, W, 2).tolist() == [0, 1]


def test_paper_smoothing_formula_by_hand():
    # abs-mean per channel: X-bar = [1, 8, 2, 4], W-bar = [1, 1, 1, 2]; product = [1, 8, 2, 8]
    X = np.array([[1, -8, 2, 4], [-1, 8, -2, -4]], np.float16)
    W = np.array([[1, 1, -1, 2], [-1, 1, 1, -2]], np.float16)
    m, idx = Cn.smoothing_vector_paper(X, W, f=2)
    assert idx.tolist() == [1, 3]
    assert m.tolist() == [1.0, 2.0, 1.0, 1.0]          # X-bar_min over I_f is 4
    m0, idx0 = Cn.smoothing_vector_paper(X, W, f=0)
    assert m0.tolist() == [1.0] * 4 and idx0.size == 0


def test_config_smoothing_formula_by_hand():
    X = np.array([[1, -16, 2, 4], [-1, 8, -2, -9]], np.float16)
    W = np.array([[1, 1, -1, 0.25], [-1, 4, 1, -0.125]], np.float16)
    s = Cn.smoothing_vector_config(X, W, np.array([1, 3]))
    assert s.tolist() == [1.0, 2.0, 1.0, 6.0]          # sqrt(16/4), sqrt(9/0.25)
    assert s.dtype == np.float32


def test_smoothing_shrinks_activation_range():
    lay, _ = synth.config1_tiny()
    s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
    assert np.all(s[lay.outlier_idx] > 4) and np.count_nonzero(s != 1) == 4
    raw = np.abs(lay.X.astype(np.float32)).max()
    smooth = np.abs(F.smooth_act(lay.X, s)).max()
    assert smooth < raw / 3


def test_outlier_split_variant(small_layer):
    """W M = W_s + W_o (Eq. 12): the outlier columns are not quantized and move into the
    SVD target, which then equals W diag(s) - Q(W_s)."""
    lay, s = small_layer
    idx = lay.outlier_idx
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=8, split_outliers=idx)
    assert not L.q[:, idx].any()
    assert np.array_equal(L.E[:, idx], L.ws[:, idx].astype(np.float64))
    keep = np.setdiff1d(np.arange(48), idx)
    deq = L.q.astype(np.float64) * L.w_scale.astype(np.float64)[:, None]
    assert np.array_equal(L.E[:, keep], L.ws[:, keep].astype(np.float64) - deq[:, keep])
    # with full rank the split layer reproduces the smoothed weight too
    Lf = Cn.construct_layer(lay.W, lay.X_cal, s, r=40, split_outliers=idx)
    deqf = Lf.q.astype(np.float64) * Lf.w_scale.astype(np.float64)[:, None]
    assert np.allclose(deqf + Lf.L_B64 @ Lf.L_A64, Lf.ws.astype(np.float64), atol=1e-10)


# ---------------------------------------------------------------------------
# rank rule and overhead model
# ---------------------------------------------------------------------------

def test_rank_from_alpha_by_hand():
    sig = np.array([4.0, 3.0, 2.0, 1.0])       # shares 0.4, 0.7, 0.9, 1.0
    assert Cn.rank_from_alpha(sig, 0.5) == 1
    assert Cn.rank_from_alpha(sig, 0.4) == 0   # strict inequality
    assert Cn.rank_from_alpha(sig, 0.71) == 2
    assert Cn.rank_from_alpha(sig, 0.95) == 3
    assert Cn.rank_from_alpha(sig, 0.05) == 0


def test_overhead_model_reproduces_table4():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "table4_rank_overhead.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 5
    for _alpha, rbar, pct in rows:
        got = 100.0 * Cn.extra_flops_fraction(float(rbar), 4096)
        assert round(got, 2) == pytest.approx(float(pct), abs=0.0051)


def test_construct_with_alpha_uses_rank_rule(small_layer):
    lay, s = small_layer
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=None, alpha=0.3)
    share = np.cumsum(L.sigma) / L.sigma.sum()
    r = L.L_A.shape[0]
    assert (r == 0 or share[r - 1] < 0.3) and share[r] >= 0.3


def test_compensation_reduces_output_error_config1():
    """End to end on the tiny configuration: rank-16 factors from 128 calibration tokens
    reduce the output error of plain W4A8 on fresh tokens."""
    lay, r = synth.config1_tiny()
    s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
    L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
    ref = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    plain = F.forward(lay.X, s, L.Wq, L.w_scale)
    comp = F.forward(lay.X, s, L.Wq, L.w_scale, L.L_A, L.L_B)
    assert np.linalg.norm(comp.y - ref) < np.linalg.norm(plain.y - ref)
