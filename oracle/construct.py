"""Oracle construction of an ASER-quantized layer (test infrastructure, NumPy fp64).

Follows the per-layer body of Algorithm 1 of the paper: smoothing vector
(Sec. 4.2, Eq. 11), int4 round-to-nearest of the smoothed weight, whitening by
Cholesky (Sec. 4.1, Eq. 5), SVD of the whitened error and truncation (Eq. 6),
factor split (text below Eq. 8), rank threshold (Eq. 9 of Sec. 4.1).

Operand names follow the library, not the paper: L_B = U_r Sigma_r is the UP
projection [N,r] (paper: L_A) and L_A = V_r^T S^-1 the DOWN projection [r,K]
(paper: L_B).  Storage is token-major (X is [tokens, K]), so the paper's
X X^T is X^T X here.

Readings where the paper is silent (all recorded in the design notes):
  * the Gram matrix is damped, G + lambda I with lambda = damping * trace(G)/K,
    because the benchmark configurations calibrate with fewer tokens than
    channels and an undamped Cholesky would not exist;
  * the Cholesky factor is the lower one, the Gram matrix is not normalised;
  * the SVD target with the outlier split is W diag(s) - Q(W_s), i.e.
    E_q + W_o with E_q = W_s - Q(W_s) (Eq. 12), not the double-counted
    expression printed inside Algorithm 1.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import scipy.linalg

from . import forward as F


# ---------------------------------------------------------------------------
# Activation smoothing (Sec. 4.2)
# ---------------------------------------------------------------------------

def channel_abs_mean(A: np.ndarray) -> np.ndarray:
    """Absolute mean per channel (column) in fp64: the paper's X-bar / W-bar."""
    return np.abs(A.astype(np.float64)).mean(axis=0)


def outlier_index_set(X_cal: np.ndarray, W: np.ndarray, f: int) -> np.ndarray:
    """I_f: the f channels with the largest X-bar * W-bar; ties go to the lower index."""
    score = channel_abs_mean(X_cal) * channel_abs_mean(W)
    order = np.lexsort((np.arange(score.size), -score))  # by -score, then index
    return np.sort(order[:f]).astype(np.int64)


def smoothing_vector_paper(X_cal: np.ndarray, W: np.ndarray, f: int):
    """Eq. 11: m_i = X-bar_i / min_{I_f} X-bar on the outlier set, 1 elsewhere."""
    idx = outlier_index_set(X_cal, W, f)
    xbar = channel_abs_mean(X_cal)
    m = np.ones(X_cal.shape[1], dtype=np.float64)
    if f > 0:
        m[idx] = xbar[idx] / xbar[idx].min()
    return m.astype(np.float32), idx


def smoothing_vector_config(X_cal: np.ndarray, W: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """The benchmark configurations' rule: s_c = sqrt(max|X_c| / max|W_c|) on the
    outlier channels (maxima over calibration tokens / over all output rows), 1 elsewhere."""
    xmax = np.abs(X_cal[:, idx].astype(np.float32)).max(axis=0)
    wmax = np.abs(W[:, idx].astype(np.float32)).max(axis=0)
    s = np.ones(X_cal.shape[1], dtype=np.float32)
    s[idx] = np.sqrt(xmax / wmax).astype(np.float32)
    return s


# ---------------------------------------------------------------------------
# Whitening SVD (Sec. 4.1)
# ---------------------------------------------------------------------------

def gram(Xs_cal: np.ndarray) -> np.ndarray:
    """X X^T of the paper (channels x channels), token-major input, fp64, unnormalised."""
    A = Xs_cal.astype(np.float64)
    return A.T @ A


def whitening_factor(G: np.ndarray, damping: float = 0.01) -> tuple[np.ndarray, float]:
    """Lower Cholesky factor S with S S^T = G + lambda I (Eq. 5 with damping)."""
    K = G.shape[0]
    lam = float(damping) * float(np.trace(G)) / K
    S = np.linalg.cholesky(G + lam * np.eye(K))
    return S, lam


def whitened_svd(E: np.ndarray, S: np.ndarray):
    """Thin SVD of E S (Alg. 1, 'SVD decomposition')."""
    U, sig, Vt = np.linalg.svd(E @ S, full_matrices=False)
    return U, sig, Vt


def factors_from_svd(U, sig, Vt, S, r: int) -> tuple[np.ndarray, np.ndarray]:
    """L_B = U_r Sigma_r  [N,r];  L_A = V_r^T S^-1  [r,K]  (triangular solve), fp64."""
    L_B = U[:, :r] * sig[:r]
    if r == 0:
        return np.zeros((0, S.shape[0])), L_B
    # L_A S = V_r^T  <=>  S^T L_A^T = V_r
    L_A = scipy.linalg.solve_triangular(S, Vt[:r].T, trans="T", lower=True).T
    return L_A, L_B


def rank_from_alpha(sig: np.ndarray, alpha: float) -> int:
    """Largest r whose leading singular values hold a share < alpha of the total
    (Sec. 4.1, the max_r ... < alpha rule); 0 when even sigma_1 exceeds the share."""
    share = np.cumsum(sig) / np.sum(sig)
    return int(np.searchsorted(share, alpha, side="left"))


def extra_flops_fraction(r: float, d: int) -> float:
    """Overhead model of the paper's complexity table: (s d^2 + 2 s r d) / (s d^2) - 1 = 2r/d."""
    return 2.0 * r / d


# ---------------------------------------------------------------------------
# One layer, end to end (body of Algorithm 1)
# ---------------------------------------------------------------------------

@dataclass
class Layer:
    s: np.ndarray          # [K] fp32 smoothing vector
    q: np.ndarray          # [N,K] int8 container of int4 codes
    Wq: np.ndarray         # [N,K/2] canonical packed nibbles
    w_scale: np.ndarray    # [N] fp32
    L_A: np.ndarray        # [r,K] fp16 (rounded)
    L_B: np.ndarray        # [N,r] fp16 (rounded)
    L_A64: np.ndarray      # unrounded
    L_B64: np.ndarray
    E: np.ndarray          # [N,K] fp64 SVD target (E_q, plus W_o with the split)
    S: np.ndarray          # [K,K] fp64 Cholesky factor
    sigma: np.ndarray      # singular values of E S
    lam: float
    ws: np.ndarray         # [N,K] fp32 smoothed weight W diag(s)


def construct_layer(W: np.ndarray, X_cal: np.ndarray, s: np.ndarray | None, r: int | None,
                    *, alpha: float | None = None, damping: float = 0.01,
                    split_outliers: np.ndarray | None = None) -> Layer:
    """Quantize W diag(s) to int4 and build rank-r factors from calibration tokens.

    `split_outliers`: index set I_f whose columns of W diag(s) are kept out of
    the quantizer (W_o, Eq. 12) and carried by the low-rank term only.
    Exactly one of `r`, `alpha` selects the rank.
    """
    N, K = W.shape
    s32 = np.ones(K, np.float32) if s is None else np.ascontiguousarray(s, dtype=np.float32)
    if split_outliers is None:
        q, w_scale, ws = F.quant_w4(W, s32, want_ws=True)
    else:
        _, _, ws = F.quant_w4(W, s32, want_ws=True)
        W_s = W.copy()
        W_s[:, split_outliers] = 0
        q, w_scale = F.quant_w4(W_s, s32)
    deq = q.astype(np.float64) * w_scale.astype(np.float64)[:, None]
    E = ws.astype(np.float64) - deq            # = E_q (+ W_o on the split columns)
    Xs_cal = F.smooth_act(X_cal, s32)
    S, lam = whitening_factor(gram(Xs_cal), damping)
    U, sig, Vt = whitened_svd(E, S)
    if r is None:
        r = rank_from_alpha(sig, alpha)
    L_A64, L_B64 = factors_from_svd(U, sig, Vt, S, r)
    return Layer(s=s32, q=q, Wq=F.pack_w4(q), w_scale=w_scale,
                 L_A=L_A64.astype(np.float16), L_B=L_B64.astype(np.float16),
                 L_A64=L_A64, L_B64=L_B64, E=E, S=S, sigma=sig, lam=lam, ws=ws)
