"""Pins for the oracle's mismatch diagnostics (Eq. channel-score, Eq. linear-mismatch)."""
import numpy as np
import torch

from oracle import diagnostics as D
from oracle import moe as M
from oracle import nvfp4 as Q
from oracle import rac as R
from paper_2607_15810_b200 import synth


def _dense(T=24, K=64, N=8, seed=3):
    x, w = synth.dense_inputs(seed=seed, T=T, K=K, N=N, outlier_channels=(3, 41))
    return x.to(torch.float32).numpy(), w.to(torch.float32).numpy()


def test_channel_scores_are_the_column_sums_of_the_squared_residual():
    x, _ = _dense()
    s = D.channel_scores_of(x)
    site = R.rac(x, 7)
    assert np.array_equal(s, site["scores"])                     # what RAC ranks on
    r = (Q.dequantize_f32(site["codes"], site["sf"], site["gs"]) - x).astype(np.float64)
    brute = np.array([sum(float(v) ** 2 for v in r[:, j]) for j in range(x.shape[1])])
    assert np.allclose(s, brute, rtol=1e-13)
    assert list(site["sel"]) == sorted(np.argsort(-brute, kind="stable")[:7])
    # the blocks that hold the outlier channels carry the large residuals ("vertical bands")
    top = set(int(j) // 16 for j in np.argsort(-s)[:8])
    assert top <= {3 // 16, 41 // 16}
    # a tensor NVFP4 represents exactly has no residual at all
    mags = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6, 6], dtype=np.float32)
    xe = np.tile(mags * np.float32(448 * 2.0 ** -5), (4, 2))
    assert not D.channel_scores_of(xe).any()
    # a supplied (saturating) scale changes the residual, and the scores follow the definition
    g = np.float32(0.25) * Q.tensor_global_scale(x)
    c, sf, _ = Q.quantize(x, g)
    r2 = (Q.dequantize_f32(c, sf, g) - x).astype(np.float64)
    assert np.allclose(D.channel_scores_of(x, g), (r2 * r2).sum(axis=0), rtol=1e-13)
    assert D.channel_scores_of(x, g).sum() > s.sum()


def test_mismatch_norms_closed_forms():
    rng = np.random.default_rng(1)
    b = rng.normal(size=(5, 7))
    n = D.mismatch_norms(b, b)
    assert n[0] == 0 and n[1] == n[2] == np.sum(b * b)
    n = D.mismatch_norms(2 * b, b)
    assert np.isclose(n[0], np.sum(b * b)) and np.isclose(n[1], 4 * np.sum(b * b))
    a = np.zeros((2, 2)); a[0, 1] = 3.0
    c = np.zeros((2, 2)); c[1, 0] = 4.0
    assert list(D.mismatch_norms(a, c)) == [25.0, 9.0, 16.0]


def test_linear_mismatch_decomposition_holds():
    """Eq. linear-mismatch with eta = 0: Y_infer - Y_train = W dX + dW X + dW dX, and the pieces are
    what the one-sided modes isolate: W16A4 - W16A16 = W dX, W4A16 - W16A16 = dW X."""
    x, w = _dense(T=12, K=64, N=6, seed=5)
    t = D.linear_mismatch_terms(x, w)
    lhs = t["y_infer"] - t["y_train"]
    assert np.allclose(lhs, t["act"] + t["wgt"] + t["second"], rtol=1e-9, atol=1e-12)
    wq = Q.quantize(w)
    y_w4a16 = M.dense_w4a16(x, *wq)["y64"]
    y_w16a4 = M.dense_w16a4(x, w)["y64"]
    assert np.allclose(y_w16a4 - t["y_train"], t["act"], rtol=1e-9, atol=1e-12)
    assert np.allclose(y_w4a16 - t["y_train"], t["wgt"], rtol=1e-9, atol=1e-12)
    # the second-order term is the product of two small errors
    assert np.linalg.norm(t["second"]) < 0.25 * min(np.linalg.norm(t["act"]), np.linalg.norm(t["wgt"]))
    # the norms helper on these matrices
    n = D.mismatch_norms(t["y_infer"], t["y_train"])
    assert np.isclose(np.sqrt(n[0]), np.linalg.norm(lhs))
