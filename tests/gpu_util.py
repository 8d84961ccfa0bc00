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


def assert_T_close(T_gpu, T_ref):
    """T is stored in bf16 (8 significant bits) after an fp32 (or fp16-input) accumulation."""
    T_gpu = T_gpu.astype(np.float64)
    scale = np.abs(T_ref).max() + 1e-30
    err = np.abs(T_gpu - T_ref)
    assert np.all(err <= 2.0 ** -8 * np.abs(T_ref) + 2e-3 * scale), (err.max(), scale)
