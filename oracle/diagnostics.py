"""Mismatch diagnostics of the paper's analysis, as plain definitions.

TEST INFRASTRUCTURE ONLY (see oracle/formats.py).

  channel_scores_of(x)   s_j^2 = sum_t (Q_A(X) - X)[t, j]^2, the squared channel score of Eq.
                         "channel-score": the per-channel residual map behind Fig.
                         "residual-distribution" (its heavy channels are the "vertical bands").
  mismatch_norms(a, b)   ||A - B||_F^2, ||A||_F^2, ||B||_F^2: with A = Y_infer and B = Y_train the
                         square root of the first is the layer-wise forward mismatch of Eq.
                         "linear-mismatch".
  linear_mismatch_terms  the three terms of Eq. "linear-mismatch" for one projection with no
                         engine mismatch (eta = 0): W dX (activation error), dW X (weight error),
                         dW dX (second order), with dX = Q_A(X) - X and dW = Q_W(W) - W taken on the
                         bf16-decoded operands.

Pinned: the identity Y_infer - Y_train = W dX + dW X + dW dX (exact in float64 up to rounding),
zero scores for tensors NVFP4 represents exactly, closed forms of the norms.
"""
import numpy as np

from . import nvfp4 as Q
from . import rac as R

F32 = np.float32


def channel_scores_of(x, gs=None):
    """x float32 (bf16-valued) [T, H] -> float64 [H]."""
    x = np.asarray(x, dtype=F32)
    codes, sf8, gs = Q.quantize(x, gs)
    return R.channel_scores(R.residual_f32(x, codes, sf8, gs))


def mismatch_norms(a, b):
    a64, b64 = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    d = a64 - b64
    return np.array([np.sum(d * d), np.sum(a64 * a64), np.sum(b64 * b64)])


def linear_mismatch_terms(x, w):
    """x [T, K], w [N, K] float32 (bf16-valued).  Returns dict of float64 [T, N] matrices:
    y_train = W X, y_infer = W^ X^, act = W dX, wgt = dW X, second = dW dX (bf16-decoded W^, X^)."""
    x64, w64 = np.asarray(x, dtype=np.float64), np.asarray(w, dtype=np.float64)
    xh = Q.dequantize_bf16(*Q.quantize(np.asarray(x, dtype=F32))).astype(np.float64)
    wh = Q.dequantize_bf16(*Q.quantize(np.asarray(w, dtype=F32))).astype(np.float64)
    dx, dw = xh - x64, wh - w64
    return dict(y_train=x64 @ w64.T, y_infer=xh @ wh.T, act=dx @ w64.T, wgt=x64 @ dw.T, second=dx @ dw.T)
