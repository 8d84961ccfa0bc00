"""Shared helpers of the GPU parity tests: build a layer with the oracle, run the CUDA
library on the same arrays, compare stage by stage."""
from __future__ import annotations

import numpy as np
import torch

import aser_synth as synth
from oracle import construct as Cn
from oracle import forward as F

Y_RTOL_ROW = 2e-3   # |y - y_ref| <= 2e-3 * max_n |y_ref[m, :]| per token row


def to_dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def oracle_layer(lay: synth.LayerInputs, r: int, construct: bool):
    """Smoothing vector, packed weights and factors.  With `construct` the oracle's
    whitening SVD builds the factors; otherwise stand-in factors (forward parity does not
    depend on how the factors were made: both sides consume the same fp16 arrays)."""
    N, K = lay.W.shape
    s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
    if construct:
        L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
        return s, L.Wq, L.w_scale, L.L_A, L.L_B
    q, w_scale = F.quant_w4(lay.W, s)
    L_A, L_B = synth.standin_factors(N, K, r, seed=lay.meta["seed"], scale_a=0.01, scale_b=0.01)
    return s, F.pack_w4(q), w_scale, L_A, L_B


def assert_rows_close(Y, y_ref, rows=None, tol=Y_RTOL_ROW):
    Y = Y.astype(np.float64)
    if rows is not None:
        Y = Y[rows]
    bound = tol * np.abs(y_ref).max(axis=1, keepdims=True)
    err = np.abs(Y - y_ref)
    worst = (err / np.maximum(bound, 1e-30)).max()
    assert np.all(err <= bound), f"worst error / bound = {worst:.3f}"


def assert_T_close(T_gpu, T_ref, xs, L_A):
    """T = x~ L_A^T is accumulated in fp32 and stored in bf16.  What may separate it from the
    fp64 oracle, entry by entry:
      * the bf16 store: 8 significant bits, so half a unit in the last place is at most 2^-8 |T|;
      * the tensor-core kernels round x~ to fp16 first: each product is off by at most
        2^-11 of itself, independently and with either sign, so the sum is off by about
        2^-11.8 * rms with rms = sqrt(sum_k (L_A[j,k] x~[m,k])^2); six standard deviations
        of that are 2^-9.2 * rms;
      * fp32 accumulation: 2^-20 of sum_k |L_A[j,k] x~[m,k]| covers every order of summation.
    """
    T_gpu = T_gpu.astype(np.float64)
    xs64 = xs.astype(np.float64)
    la64 = L_A.astype(np.float64)
    rms = np.sqrt((xs64 ** 2) @ (la64 ** 2).T)
    l1 = np.abs(xs64) @ np.abs(la64).T
    tol = 2.0 ** -8 * (1 + 1e-3) * np.abs(T_ref) + 2.0 ** -9.2 * rms + 2.0 ** -20 * l1 + 1e-30
    err = np.abs(T_gpu - T_ref)
    assert np.all(err <= tol), f"worst error / bound = {(err / tol).max():.3f}"
