"""Residual Activation Compensation (Section "Activation Error Compensation
for Rollout-side").

TEST INFRASTRUCTURE ONLY (see oracle/formats.py).

  residual        dX_q = Q_A(X) - X                         (Eq. residual-def)
  channel score   s_j  = || dX_q[:, j] ||_2 over the batch  (Eq. channel-score)
  selection       S    = the n_sel channels with largest s  (Eq. channel-select)
  reconstruction  X~   = Q_A(X) - M_S (.) Q_A(dX_q)         (Eq. residual-recon)

Readings where the paper is silent:
  * the residual is kept in float32 (it is not rounded to bf16 first);
  * scores are ranked on the sum of squares (the square root is monotone),
    accumulated in float64; ties go to the lower channel index; the percentage
    k% of the paper is given as an integer count n_sel;
  * Q_A applied to the residual is the same operator as for X: the same
    16-blocks along the hidden dimension and, by default, the SAME per-tensor
    scale as X (`r_gs=None`), so that one accumulator can hold both GEMM terms.
    Passing `r_gs="own"` gives the residual its own amax-derived per-tensor
    scale instead; the shrink inequality (Eq. residual-shrink) holds for both
    and is pinned for both;
  * Q_A is applied to the full residual tensor and the mask then clears the
    codes of unselected channels; block scales are left as computed.
"parity unpinned" for these choices; pinned: sign convention and shrink
inequality, monotone error in n_sel, n_sel=0 / n_sel=K special cases, brute
force selection on tiny inputs.
"""
import numpy as np

from . import nvfp4 as Q

F32 = np.float32


def residual_f32(x, codes, sf8, gs):
    """dX_q = Q_A(X) - X in float32 (Eq. residual-def)."""
    return (Q.dequantize_f32(codes, sf8, gs) - np.asarray(x, dtype=F32)).astype(F32)


def channel_scores(r):
    """Sum over the token batch of the squared residual per channel, float64
    (the square of s_j in Eq. channel-score)."""
    r64 = np.asarray(r, dtype=np.float64)
    return np.sum(r64 * r64, axis=0)


def select_channels(scores, n_sel):
    """Indices (ascending) of the n_sel largest scores; ties to the lower index."""
    scores = np.asarray(scores, dtype=np.float64)
    order = np.lexsort((np.arange(scores.size), -scores))   # by -score, then index
    return np.sort(order[:n_sel]).astype(np.int32)


def rac(x, n_sel, gs=None, r_gs=None):
    """Full RAC at one activation site.  x: float32 (bf16-valued) [rows, K].
    Returns a dict with the quantized activation (codes, sf, gs), the selected
    channels, and the masked quantized residual (r_codes, r_sf, r_gs)."""
    x = np.asarray(x, dtype=F32)
    codes, sf8, gs = Q.quantize(x, gs)
    r = residual_f32(x, codes, sf8, gs)
    scores = channel_scores(r)
    sel = select_channels(scores, n_sel)
    if r_gs is None:
        r_gs_val = gs
    elif isinstance(r_gs, str) and r_gs == "own":
        r_gs_val = Q.tensor_global_scale(r)
    else:
        r_gs_val = F32(r_gs)
    r_codes, r_sf8, r_gs_val = Q.quantize(r, r_gs_val)
    mask = np.zeros(x.shape[1], dtype=bool)
    mask[sel] = True
    r_codes = np.where(mask[None, :], r_codes, np.uint8(0)).astype(np.uint8)
    return dict(codes=codes, sf=sf8, gs=gs, residual=r, scores=scores, sel=sel,
                r_codes=r_codes, r_sf=r_sf8, r_gs=r_gs_val)


def reconstruct_real(site):
    """X~ of Eq. residual-recon as real numbers (float64)."""
    return (Q.dequantize_real(site["codes"], site["sf"], site["gs"])
            - Q.dequantize_real(site["r_codes"], site["r_sf"], site["r_gs"]))
