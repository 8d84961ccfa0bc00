"""GPU construction of the factors (aser_construct: Gram, Cholesky, top-r singular triplets of the
whitened error, on the device) against the CPU oracle's construction, by what is unique:
the packed weights and scales (bit-exact), the whitening factor S (the Cholesky factor is unique),
the singular values, the product L_B L_A, and the truncation loss of Eq. 8.  The factors
themselves are determined only up to sign and are not compared element by element."""
import numpy as np
import pytest
import torch

import aser_synth as synth
from oracle import construct as Cn
from oracle import forward as F
from gpu_util import to_dev, assert_rows_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def aser(cuda_device):
    import paper_2411_07762_b200 as aser
    return aser


def _check(aser, lay, r, iterations=0, split=False):
    if split:       # the paper's own smoothing rule (Eq. 11) and outlier split (Eq. 12)
        s, idx = Cn.smoothing_vector_paper(lay.X_cal, lay.W, f=len(lay.outlier_idx))
        L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r, split_outliers=idx)
        split_idx = to_dev(idx.astype(np.int32))
    else:
        s = Cn.smoothing_vector_config(lay.X_cal, lay.W, lay.outlier_idx)
        L = Cn.construct_layer(lay.W, lay.X_cal, s, r=r)
        split_idx = None
    out = aser.construct(to_dev(lay.W), to_dev(s), to_dev(lay.X_cal), r, damping=0.01,
                         iterations=iterations, want_S=True, split_idx=split_idx)
    torch.cuda.synchronize()
    # quantizer: bit-exact
    assert np.array_equal(out["Wq"].cpu().numpy(), L.Wq)
    assert np.array_equal(out["w_scale"].cpu().numpy().view(np.uint32), L.w_scale.view(np.uint32))
    # whitening factor (Eq. 5): unique, compared entry by entry, and S S^T against the damped Gram
    S = out["S"].cpu().numpy()
    assert np.allclose(S, L.S, rtol=1e-9, atol=1e-9 * np.abs(L.S).max())
    Xs = F.smooth_act(lay.X_cal, s).astype(np.float64)
    G = Xs.T @ Xs
    G += L.lam * np.eye(G.shape[0])
    assert np.allclose(S @ S.T, G, rtol=1e-10, atol=1e-10 * np.abs(G).max())
    # singular values of E S (Eq. 6)
    sig = out["sigma"].cpu().numpy()
    assert np.allclose(sig, L.sigma[:r], rtol=1e-6)
    # product and truncation loss (Eq. 8): the fp16-rounded factors of both sides
    LA = out["L_A"].cpu().numpy().astype(np.float64)
    LB = out["L_B"].cpu().numpy().astype(np.float64)
    prod_gpu = LB @ LA
    prod_ref = L.L_B.astype(np.float64) @ L.L_A.astype(np.float64)
    rel = np.linalg.norm(prod_gpu - prod_ref) / np.linalg.norm(prod_ref)
    assert rel < 2e-3, rel                       # two fp16 roundings of each side: about 3e-4 each
    tail = float((L.sigma[r:] ** 2).sum())
    loss_gpu = np.linalg.norm((L.E - prod_gpu) @ L.S) ** 2
    loss_ref = np.linalg.norm((L.E - prod_ref) @ L.S) ** 2
    assert loss_gpu <= loss_ref * (1 + 1e-3) and loss_gpu >= tail * (1 - 1e-9)
    return s, L, out


def test_construct_config1_tiny_and_forward_with_its_factors(aser):
    """Configuration 1 end to end on the device: construction, then the forward pass with the
    device-built factors against the oracle's forward pass on the same factors."""
    lay, r = synth.config1_tiny()
    s, L, out = _check(aser, lay, r)
    LA, LB = out["L_A"].cpu().numpy(), out["L_B"].cpu().numpy()
    layer = aser.AserLinear(to_dev(lay.W), to_dev(s), out["L_A"].contiguous(), out["L_B"], lay.X.shape[0])
    Y = layer(to_dev(lay.X)).cpu().numpy()
    ref = F.forward(lay.X, s, L.Wq, L.w_scale, LA, LB)
    assert_rows_close(Y, ref.y)
    # and the compensated output beats plain W4A8 against the fp product
    plain = layer(to_dev(lay.X), lowrank=False).cpu().numpy().astype(np.float64)
    exact = lay.X.astype(np.float64) @ lay.W.astype(np.float64).T
    assert np.linalg.norm(Y.astype(np.float64) - exact) < np.linalg.norm(plain - exact)


@pytest.mark.parametrize("N,K,r,n_cal", [(384, 512, 32, 256), (1024, 1024, 64, 512), (520, 768, 48, 100)])
def test_construct_matches_oracle_invariants(aser, N, K, r, n_cal):
    lay = synth.make_layer(4, N, K, seed=synth.seed_for(2, N + K + r), n_cal=n_cal)
    _check(aser, lay, r)


def test_construct_with_outlier_split(aser):
    """The split variant: the outlier columns are zero in Wq and the factors carry them."""
    lay = synth.make_layer(4, 512, 512, seed=synth.seed_for(1, 9), n_out=4, outlier_gain=40.0, n_cal=128)
    s, L, out = _check(aser, lay, 32, split=True)
    q = F.unpack_w4(out["Wq"].cpu().numpy())
    assert not q[:, lay.outlier_idx].any()


def test_construct_rank_zero_only_packs_and_bad_arguments(aser):
    lay = synth.make_layer(4, 256, 256, seed=31, n_cal=64)
    out = aser.construct(to_dev(lay.W), None, to_dev(lay.X_cal), 0)
    q, w_scale = F.quant_w4(lay.W, None)
    assert np.array_equal(out["Wq"].cpu().numpy(), F.pack_w4(q))
    with pytest.raises(aser.AserError) as err:
        aser.construct(to_dev(lay.W), None, to_dev(lay.X_cal), 16, damping=0.0)
    assert err.value.code == -3


def test_construct_config2_full_size(aser):
    """The 4096 x 4096 attention projection with 512 calibration tokens, rank 64 (configuration 2)."""
    lay, r = synth.config2_decode(8)
    _check(aser, lay, r)
