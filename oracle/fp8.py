"""FP8 W8A8 with fine-grained block scaling: the comparison format of the paper (Section
"Low-Precision Inference", paragraph FP8; the "FP8 W8A8" arm of Section "Rollout Throughput
Comparison").

TEST INFRASTRUCTURE ONLY (see oracle/formats.py).

The paper fixes only the element format (E4M3: 4 exponent bits, 3 mantissa bits, maximum 448) and that
"each tile of values carries its own" scale.  The reading used here ("parity unpinned": the tile
shapes, the power-of-two scale and its rounding are this repository's choice, the common one for
Blackwell's block-scaled FP8 tensor-core path):

  activations  one scale per (row, 128 consecutive channels)
  weights      one scale per (128 rows x 128 channels) tile
  scale        2^e, e = ceil(log2(amax / 448)) computed exactly from the float32 bits
               (an 8-bit exponent-only "UE8M0" code e + 127); amax = 0 gives e = -127
  element      E4M3 round-to-nearest-even, saturating, of x * 2^-e (exact scaling)

The GEMM is the plain definition in float64 over the decoded operands (element * 2^e), exact
products; expert MLP, routing and dispatch as in oracle/moe.py; h is rounded to bf16 and requantized
per (row, 128 features) before the down projection.

Pinned: the scale is the smallest power of two that avoids saturation, decoded tiles never exceed
448 * 2^e, exact round trip of representable tensors, float64 triple loop on tiny shapes, torch's
float8_e4m3fn conversion for the element rounding (formats.e4m3_encode is pinned there).
"""
import numpy as np

from . import formats as F
from . import moe as M

F32 = np.float32
TILE = 128


def scale_exponent(amax):
    """Smallest integer e with amax <= 448 * 2^e (float32 amax >= 0, array); -127 for amax == 0."""
    amax = np.asarray(amax, dtype=np.float64)
    with np.errstate(divide="ignore"):
        m, ex = np.frexp(amax / F.E4M3_MAX)               # amax/448 = m * 2^ex, 0.5 <= m < 1 (division by 448 = 7 * 64)
    # amax/448 is not exact in float64 only if it needs > 53 bits: amax has 24 bits and 1/448 = 1/(7*64),
    # so decide the boundary case exactly with integers: e is ex when amax > 448 * 2^(ex-1), and m == 0.5
    # means amax == 448 * 2^(ex-1) exactly when that product equals amax
    e = ex.astype(np.int64)
    exact_pow2 = (F.E4M3_MAX * np.ldexp(1.0, (e - 1).astype(np.int64)) >= amax)
    e = np.where(exact_pow2, e - 1, e)
    e = np.where(amax == 0, -127, e)
    return np.clip(e, -127, 127).astype(np.int32)


def quantize_act(x):
    """x float32 (bf16-valued) [rows, K], K % 128 == 0 -> (codes u8 [rows, K], exps int32 [rows, K/128])."""
    x = np.asarray(x, dtype=F32)
    rows, K = x.shape
    assert K % TILE == 0
    t = x.reshape(rows, K // TILE, TILE)
    e = scale_exponent(np.max(np.abs(t), axis=2) if rows else np.zeros((0, K // TILE)))
    v = np.ldexp(t.astype(np.float64), -e[:, :, None]).astype(F32)       # exact: a power-of-two scaling
    return F.e4m3_encode(v).reshape(rows, K), e


def quantize_weight(w):
    """w float32 (bf16-valued) [N, K], N % 128 == 0, K % 128 == 0 -> (codes u8 [N, K], exps [N/128, K/128])."""
    w = np.asarray(w, dtype=F32)
    N, K = w.shape
    assert N % TILE == 0 and K % TILE == 0
    t = w.reshape(N // TILE, TILE, K // TILE, TILE)
    e = scale_exponent(np.max(np.abs(t), axis=(1, 3)))
    v = np.ldexp(t.astype(np.float64), -e[:, None, :, None]).astype(F32)
    return F.e4m3_encode(v).reshape(N, K), e


def dequantize_act(codes, exps):
    rows, K = codes.shape
    v = F.e4m3_decode(codes).reshape(rows, K // TILE, TILE)
    return np.ldexp(v, exps[:, :, None]).reshape(rows, K)


def dequantize_weight(codes, exps):
    N, K = codes.shape
    v = F.e4m3_decode(codes).reshape(N // TILE, TILE, K // TILE, TILE)
    return np.ldexp(v, exps[:, None, :, None]).reshape(N, K)


def moe_forward(x, logits, w13, w2, topk, renormalize=True, h_override=None):
    """FP8 W8A8 MoE layer.  w13: dict(codes [E, 2I, H], exps [E, 2I/128, H/128]) gate rows first;
    w2: dict(codes [E, H, I], exps [E, H/128, I/128]).  Returns the intermediates the CUDA path exports
    (h in dispatch order) and out64 / out_absdot / g64 / g_absdot for the tolerance."""
    x = np.asarray(x, dtype=F32)
    T, H = x.shape
    E = logits.shape[1]
    I = w2["codes"].shape[2]
    ids, wts = M.route(logits, topk, renormalize)
    counts, offsets, perm = M.dispatch(ids, E)
    A = T * topk
    xc, xe = quantize_act(x)
    xd = dequantize_act(xc, xe)
    tok_of = perm // topk
    g64 = np.empty((A, 2 * I))
    g_absdot = np.empty((A, 2 * I))
    for e in range(E):
        lo, hi = offsets[e], offsets[e + 1]
        if lo == hi:
            continue
        w = dequantize_weight(w13["codes"][e], w13["exps"][e])
        g64[lo:hi] = xd[tok_of[lo:hi]] @ w.T
        g_absdot[lo:hi] = np.abs(xd[tok_of[lo:hi]]) @ np.abs(w).T
    h64 = M.silu(g64[:, :I]) * g64[:, I:]
    h_own = F.bf16_round(h64)
    h = h_own if h_override is None else np.asarray(h_override, dtype=F32)
    hc, he = quantize_act(h)
    hd = dequantize_act(hc, he)
    out64 = np.zeros((T, H))
    out_absdot = np.zeros((T, H))
    w_flat = wts.reshape(-1).astype(np.float64)
    for e in range(E):
        lo, hi = offsets[e], offsets[e + 1]
        if lo == hi:
            continue
        w = dequantize_weight(w2["codes"][e], w2["exps"][e])
        gw = w_flat[perm[lo:hi]][:, None]
        out64[tok_of[lo:hi]] += gw * (hd[lo:hi] @ w.T)
        out_absdot[tok_of[lo:hi]] += gw * (np.abs(hd[lo:hi]) @ np.abs(w).T)
    return dict(ids=ids, weights=wts, offsets=offsets, perm=perm, x_codes=xc, x_exps=xe, g64=g64, g_absdot=g_absdot,
                h64=h64, h=h_own, h_codes=hc, h_exps=he, out64=out64, out=F.bf16_round(out64), out_absdot=out_absdot)
