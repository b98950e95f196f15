"""NVFP4 quantize / dequantize / fake-quantize, the operators Q_A, Q_W and QDQ_W.

TEST INFRASTRUCTURE ONLY (see oracle/formats.py).

Format (Section "Low-Precision Inference", paragraph FP4): E2M1 elements,
sixteen consecutive elements along the contraction dimension share one E4M3
block scale, and one FP32 per-tensor scale sits on top.  Q_A / Q_W are the
"quantize then dequantize" operators of Eqs. "act-error-def" and
"weight-error-def"; QDQ_W of Eq. "w4a16-qat-forward" is the same operator with
a bf16 result, and Eq. "weight-qdq-align" asks that trainer and rollout agree.

The paper does not say how the scales are derived.  The reading used here (all
steps are single IEEE-754 float32 operations, in this order):

  s_g  = amax(tensor) / (6 * 448)             (1 if the tensor is all zero)
  u    = amax(block) / (6 * s_g)
  sf   = E4M3(u)                              round-to-nearest-even, saturating
  d    = sf * s_g                             the decoded block scale
  code = E2M1(x * (1 / d))                    all-zero codes when sf == 0
  x^   = value(code) * d                      one float32 multiply

"parity unpinned": the order of these float32 operations and the layout of the
output bytes are this repository's reading; the invariants the format itself
fixes (idempotence, exact round trip of representable tensors, the error bound,
scale invariance under powers of two, trainer == rollout) are pinned in tests.
"""
import numpy as np

from . import formats as F

BLOCK = 16
F32 = np.float32
SIX = F32(6.0)
GLOBAL_DIV = F32(6.0 * 448.0)        # 2688


def global_scale_from_amax(amax):
    amax = F32(amax)
    return F32(amax / GLOBAL_DIV) if amax > 0 else F32(1.0)


def tensor_global_scale(t):
    return global_scale_from_amax(np.max(np.abs(np.asarray(t, dtype=F32))) if np.size(t) else 0.0)


def quantize(t, gs=None):
    """t: float32 [rows, K], K a multiple of 16.  Returns (codes u8 [rows,K]
    one nibble per element, sf u8 [rows,K/16], gs float32)."""
    t = np.asarray(t, dtype=F32)
    rows, K = t.shape
    assert K % BLOCK == 0
    gs = tensor_global_scale(t) if gs is None else F32(gs)
    blocks = t.reshape(rows, K // BLOCK, BLOCK)
    a_b = np.max(np.abs(blocks), axis=2).astype(F32) if rows else np.zeros((0, K // BLOCK), F32)
    d6 = F32(SIX * gs)
    with np.errstate(divide="ignore", invalid="ignore", over="ignore"):
        u = (a_b / d6).astype(F32)
        sf8 = F.e4m3_encode(u)
        sf = F.e4m3_decode(sf8).astype(F32)
        d = (sf * gs).astype(F32)
        inv = np.where(sf == 0, F32(0), (F32(1.0) / d).astype(F32)).astype(F32)
        v = (blocks * inv[:, :, None]).astype(F32)
    codes = F.e2m1_encode(v).reshape(rows, K)
    return codes, sf8, gs


def block_scales_f32(sf8, gs):
    """Decoded block scale d = sf * s_g as float32 [rows, K/16]."""
    return (F.e4m3_decode(sf8).astype(F32) * F32(gs)).astype(F32)


def dequantize_f32(codes, sf8, gs):
    """x^ = value(code) * d with one float32 multiply; float32 [rows, K]."""
    rows, K = codes.shape
    d = block_scales_f32(sf8, gs)
    val = F.e2m1_decode(codes).astype(F32).reshape(rows, K // BLOCK, BLOCK)
    return (val * d[:, :, None]).astype(F32).reshape(rows, K)


def dequantize_real(codes, sf8, gs):
    """The real number value * sf * s_g in float64 (exact: at most 3+4+24
    significant bits).  This is the operand the FP4 tensor-core GEMM sees."""
    rows, K = codes.shape
    d = F.e4m3_decode(sf8) * np.float64(F32(gs))
    val = F.e2m1_decode(codes).reshape(rows, K // BLOCK, BLOCK)
    return (val * d[:, :, None]).reshape(rows, K)


def dequantize_bf16(codes, sf8, gs):
    """bf16 (as float32) of the float32 dequantized value: what the trainer's
    QDQ_W produces and what the rollout side gets by dequantizing the packed
    bytes (Eq. weight-qdq-align compares the two)."""
    return F.bf16_round(dequantize_f32(codes, sf8, gs))


def fake_quant_activations(x, gs=None):
    """x: float32 (bf16-valued) [rows, K].  The activation QDQ node of the
    learner-side ablations (Table "qdq-alignment"): quantize as the rollout
    does (Eq. act-error-def), decode, round to bf16.  Returns (x_fq
    bf16-as-float32, gs float32)."""
    c, s, g = quantize(np.asarray(x, dtype=F32), gs)
    return dequantize_bf16(c, s, g), g


def fake_quant_weights(w):
    """w: float32 (bf16-valued) [n_tensors, N, K].  Each [N, K] slice is one
    tensor with its own amax-derived per-tensor scale (Eq. w4a16-qat-forward).
    Returns (w_fq bf16-as-float32, packed u8 [n,N,K/2], sf u8 [n,N,K/16],
    gs float32 [n])."""
    w = np.asarray(w, dtype=F32)
    n, N, K = w.shape
    w_fq = np.empty_like(w)
    q = np.empty((n, N, K // 2), np.uint8)
    sf = np.empty((n, N, K // BLOCK), np.uint8)
    gs = np.empty((n,), F32)
    for i in range(n):
        c, s, g = quantize(w[i])
        w_fq[i] = dequantize_bf16(c, s, g)
        q[i] = F.pack_nibbles(c)
        sf[i] = s
        gs[i] = g
    return w_fq, q, sf, gs
