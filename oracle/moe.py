"""MoE expert layer forward with native W4A4 operands and RAC at both
activation sites, and the single dense W4A4+RAC projection.

TEST INFRASTRUCTURE ONLY (see oracle/formats.py).

The paper names the projection pair only ("linear or MoE projection", the
"W13" site, Section "Activation Error Compensation for Rollout-side") and never
defines the expert MLP or the router.  The reading here, "parity unpinned"
where marked:
  * routing: the top-k experts by router logit, ties to the lower expert id,
    listed by descending logit; weights are the softmax over ALL experts
    restricted to the chosen ones, optionally renormalised to sum to one;
  * dispatch order: assignments (token, slot) sorted by (expert, token, slot);
  * expert MLP: h = silu(W1 x) * (W3 x) with W13 = [W1 (gate) rows; W3 (up)
    rows], silu(z) = z / (1 + exp(-z)); h is rounded to bf16 before it is
    quantized for the down projection W2;
  * the GEMMs contract the exact real values of the quantized operands
    (value * block scale * tensor scale) in float64: this is the plain
    definition the tensor-core path reaches up to accumulation rounding.  The
    main GEMM stays W4A4 (Section "Activation Error Compensation ...", last
    sentence of "Targeted residual compensation"): by linearity
    W X~ = W Q_A(X) - W (M_S (.) Q_A(dX_q)), both terms W4A4 products.
Pinned: brute-force routing/sort on tiny inputs, float64 triple loop on tiny
shapes, the exact-integer special case, linearity, E=1/top-1 reducing to the
dense projection; the `h_override` and forced-selection branches (used by the
staged comparison of an implementation) against explicit loops and a
brute-force re-mask.
"""
import numpy as np

from . import formats as F
from . import nvfp4 as Q
from . import rac as R

F32 = np.float32


def route(logits, topk, renormalize=True):
    """logits float32 [T, E] -> ids int32 [T, topk], weights float32 [T, topk]."""
    logits = np.asarray(logits, dtype=F32)
    T, E = logits.shape
    # stable sort on -logit keeps the lower expert id first among equal logits
    order = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")
    ids = order[:, :topk].astype(np.int32)
    z = logits.astype(np.float64)
    z = z - z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p = p / p.sum(axis=1, keepdims=True)
    w = np.take_along_axis(p, ids.astype(np.int64), axis=1)
    if renormalize:
        w = w / w.sum(axis=1, keepdims=True)
    return ids, w.astype(F32)


def dispatch(ids, E):
    """ids int32 [T, topk] -> counts [E], offsets [E+1] (exclusive scan),
    perm [A]: flat assignment indices t*topk+slot sorted by (expert, t, slot)."""
    T, topk = ids.shape
    flat = ids.reshape(-1).astype(np.int64)
    counts = np.bincount(flat, minlength=E).astype(np.int32)
    offsets = np.zeros(E + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    perm = np.argsort(flat, kind="stable").astype(np.int32)   # flat index order = (t, slot)
    return counts, offsets, perm


def silu(z):
    z = np.asarray(z, dtype=np.float64)
    return z / (1.0 + np.exp(-z))


def dense_w4a4_rac(x, w_codes, w_sf, w_gs, n_sel, a_gs=None, r_gs=None):
    """One projection Y = W X~ (config "single dense W4A4+RAC GEMM").
    x float32 (bf16-valued) [T, K]; weight codes [N, K], sf [N, K/16], gs.
    Returns dict(site=..., y64 float64 [T,N], y bf16-as-float32, absdot float64)."""
    site = R.rac(x, n_sel, a_gs, r_gs)
    xt = R.reconstruct_real(site)
    w = Q.dequantize_real(w_codes, w_sf, w_gs)
    y64 = xt @ w.T
    absdot = _absdot(site, np.abs(w))
    return dict(site=site, y64=y64, y=F.bf16_round(y64), absdot=absdot)


def dense_w4a16(x, w_codes, w_sf, w_gs):
    """One-sided mode "W4A16" (Table "qdq-alignment"; also the learner's forward of Eq.
    w4a16-qat-forward): Y = W^ X with W^ = QDQ_W(W) as the bf16 tensor the trainer multiplies
    by, activations left in bf16.  x float32 (bf16-valued) [T, K].  The contraction is the
    plain definition in float64.  Returns dict(y64, y, absdot)."""
    w = Q.dequantize_bf16(w_codes, w_sf, w_gs).astype(np.float64)
    x64 = np.asarray(x, dtype=np.float64)
    y64 = x64 @ w.T
    return dict(y64=y64, y=F.bf16_round(y64), absdot=np.abs(x64) @ np.abs(w).T)


def dense_w16a4(x, w_bf16, a_gs=None):
    """One-sided mode "W16A4": Y = W QDQ_A(X), activations quantized as the rollout does (Eq.
    act-error-def) and decoded to bf16, weights left in bf16 ([N, K] float32, bf16-valued).
    Returns dict(codes, sf, gs of the activation, y64, y, absdot)."""
    x = np.asarray(x, dtype=F32)
    codes, sf8, gs = Q.quantize(x, a_gs)
    xh = Q.dequantize_bf16(codes, sf8, gs).astype(np.float64)
    w64 = np.asarray(w_bf16, dtype=np.float64)
    y64 = xh @ w64.T
    return dict(codes=codes, sf=sf8, gs=gs, y64=y64, y=F.bf16_round(y64), absdot=np.abs(xh) @ np.abs(w64).T)


def _absdot(site, w_abs):
    """sum_k |a_k * b_k| over every product the tensor cores form: the main
    term and the residual term (the tolerance of the GEMM comparison scales
    with it)."""
    xa = np.abs(Q.dequantize_real(site["codes"], site["sf"], site["gs"]))
    ra = np.abs(Q.dequantize_real(site["r_codes"], site["r_sf"], site["r_gs"]))
    return (xa + ra) @ w_abs.T


def moe_forward(x, logits, w13, w2, topk, n_sel13, n_sel2, a2_gs,
                a13_gs=None, renormalize=True, forced_sel13=None, forced_sel2=None, h_override=None,
                expert_range=None):
    """MoE layer forward.
      x       float32 (bf16-valued) [T, H]
      logits  float32 [T, E]
      w13     dict(codes [E,2I,H], sf [E,2I,H/16], gs [E]) gate rows first, then up
      w2      dict(codes [E,H,I],  sf [E,H,I/16],  gs [E])
      a2_gs   per-tensor scale of the SwiGLU output h (caller supplied; the
              paper is silent; a fused requantize needs it before h exists)
      h_override  bf16 values [A, I] to use in place of the computed h for the
              second half of the layer.  h feeds a quantizer, so two correct
              first halves that differ by one bf16 ulp give different (both
              valid) codes; the staged comparison checks the second half of
              an implementation on that implementation's own h.
      expert_range  (lo, hi): expert-sharded execution.  Only the contributions of experts lo..hi-1 are
              computed (w13 / w2 still hold all experts here): routing and site 13 are those of the whole
              layer, h / site 2 cover the shard's dispatched rows offsets[lo]..offsets[hi] only (its own
              "current token batch" for the site-2 scores), out64 is the shard's partial sum.  The
              partial sums of disjoint shards that cover all experts add up to the layer output when
              site 2 is not compensated; with site-2 RAC every shard selects on its own rows.
    Returns a dict of every intermediate the CUDA path can export."""
    x = np.asarray(x, dtype=F32)
    T, H = x.shape
    E = logits.shape[1]
    I = w2["codes"].shape[2]
    ids, wts = route(logits, topk, renormalize)
    counts, offsets, perm = dispatch(ids, E)
    A = T * topk

    # ---- site 13: the T un-permuted token rows are the "current token batch"
    site13 = R.rac(x, n_sel13, a13_gs, None)
    if forced_sel13 is not None:
        site13 = _force_selection(x, site13, forced_sel13)
    xt = R.reconstruct_real(site13)                       # [T, H] float64
    xa = (np.abs(Q.dequantize_real(site13["codes"], site13["sf"], site13["gs"]))
          + np.abs(Q.dequantize_real(site13["r_codes"], site13["r_sf"], site13["r_gs"])))

    tok_of = perm // topk                                  # token of each dispatched row
    e_lo, e_hi = (0, E) if expert_range is None else expert_range
    row_lo, row_hi = int(offsets[e_lo]), int(offsets[e_hi])
    h64 = np.zeros((A, I), dtype=np.float64)
    g64 = np.zeros((A, 2 * I), dtype=np.float64)
    g_absdot = np.zeros((A, 2 * I), dtype=np.float64)
    for e in range(e_lo, e_hi):
        lo, hi = offsets[e], offsets[e + 1]
        if lo == hi:
            continue
        w = Q.dequantize_real(w13["codes"][e], w13["sf"][e], w13["gs"][e])   # [2I, H]
        rows = tok_of[lo:hi]
        g = xt[rows] @ w.T
        g64[lo:hi] = g
        g_absdot[lo:hi] = xa[rows] @ np.abs(w).T
        h64[lo:hi] = silu(g[:, :I]) * g[:, I:]
    h = F.bf16_round(h64)[row_lo:row_hi]                   # the shard's rows of [A, I], dispatch order
    g64, g_absdot, h64 = g64[row_lo:row_hi], g_absdot[row_lo:row_hi], h64[row_lo:row_hi]
    h_own = h
    if h_override is not None:
        h = np.asarray(h_override, dtype=F32)
        assert h.shape == h_own.shape

    # ---- site 2: all A dispatched rows together are the batch
    site2 = R.rac(h, n_sel2, a2_gs, None)
    if forced_sel2 is not None:
        site2 = _force_selection(h, site2, forced_sel2)
    ht = R.reconstruct_real(site2)
    ha = (np.abs(Q.dequantize_real(site2["codes"], site2["sf"], site2["gs"]))
          + np.abs(Q.dequantize_real(site2["r_codes"], site2["r_sf"], site2["r_gs"])))

    out64 = np.zeros((T, H), dtype=np.float64)
    out_absdot = np.zeros((T, H), dtype=np.float64)
    w_flat = wts.reshape(-1).astype(np.float64)
    for e in range(e_lo, e_hi):
        lo, hi = offsets[e], offsets[e + 1]
        if lo == hi:
            continue
        w = Q.dequantize_real(w2["codes"][e], w2["sf"][e], w2["gs"][e])      # [H, I]
        y = ht[lo - row_lo:hi - row_lo] @ w.T
        ya = ha[lo - row_lo:hi - row_lo] @ np.abs(w).T
        gw = w_flat[perm[lo:hi]][:, None]
        rows = tok_of[lo:hi]                 # distinct: a token picks an expert at most once
        assert np.unique(rows).size == rows.size
        out64[rows] += gw * y
        out_absdot[rows] += gw * ya
    return dict(ids=ids, weights=wts, counts=counts, offsets=offsets, perm=perm,
                site13=site13, g64=g64, g_absdot=g_absdot, h64=h64, h=h_own,
                site2=site2, out64=out64, out=F.bf16_round(out64), out_absdot=out_absdot)


def _force_selection(x, site, sel):
    """Re-mask the quantized residual with a given channel set (used when a
    near-tie at the selection boundary is being examined)."""
    r_codes, r_sf8, r_gs = Q.quantize(site["residual"], site["r_gs"])
    mask = np.zeros(x.shape[1], dtype=bool)
    mask[np.asarray(sel, dtype=np.int64)] = True
    out = dict(site)
    out["sel"] = np.sort(np.asarray(sel, dtype=np.int32))
    out["r_codes"] = np.where(mask[None, :], r_codes, np.uint8(0)).astype(np.uint8)
    return out
