"""Pins for the oracle's NVFP4 quantizer and weight fake-quant: invariants the
format fixes whatever the order of operations (round trip of representable
tensors, idempotence, error bound, power-of-two scale invariance, the largest
block hitting scale 448) and the trainer == rollout equality of
Eq. weight-qdq-align."""
import numpy as np
import torch

from oracle import formats as F
from oracle import nvfp4 as Q
from paper_2607_15810_b200 import synth


def _rand_bf16(shape, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16).to(torch.float32).numpy()


def test_exact_roundtrip_of_representable_tensor():
    rng = np.random.default_rng(0)
    rows, K = 7, 128
    for p in (-3, 0, 5):
        gs = np.float32(2.0 ** p)
        codes = rng.integers(0, 16, (rows, K)).astype(np.uint8)
        codes[:, ::16] = 7                                  # every block's max is code 6.0
        sf8 = rng.integers(0x08, 0x7F, (rows, K // 16)).astype(np.uint8)   # normal scales
        t = Q.dequantize_f32(codes, sf8, gs)
        assert np.array_equal(t.astype(np.float64), Q.dequantize_real(codes, sf8, gs))  # exact here
        c2, s2, g2 = Q.quantize(t, gs)
        assert np.array_equal(s2, sf8)
        # -0 and +0 differ in the sign nibble only; compare decoded values and non-zero codes
        assert np.array_equal(F.e2m1_decode(c2), F.e2m1_decode(codes))
        assert np.array_equal(Q.dequantize_f32(c2, s2, g2), t)


def test_idempotent_on_its_own_output():
    x = _rand_bf16((33, 256), 1)
    x[:, 5] *= 30
    c, s, g = Q.quantize(x)
    xh = Q.dequantize_f32(c, s, g)
    c2, s2, _ = Q.quantize(xh, g)
    assert np.array_equal(s2, s) and np.array_equal(c2, c)


def test_error_bound_half_grid_step():
    x = _rand_bf16((64, 512), 2)
    x[:, 100] *= 50
    c, s, g = Q.quantize(x)
    d = Q.block_scales_f32(s, g).astype(np.float64).repeat(16, axis=1)
    xh = Q.dequantize_real(c, s, g)
    v = np.abs(x.astype(np.float64)) / d
    step = np.where(v < 2, 0.5, np.where(v < 4, 1.0, 2.0))
    inside = v <= 6
    slack = 1e-6
    assert np.all(np.abs(xh - x)[inside] <= (0.5 * step * d)[inside] * (1 + slack))
    # saturated elements (scale rounded down) still land on 6*d
    assert np.allclose(np.abs(xh)[~inside], (6 * d)[~inside], rtol=1e-6, atol=0)
    # the scale is within E4M3 rounding (2^-4 relative) of amax/6, so saturation is mild
    assert np.all(v[~inside] <= 6 * (1 + 2.0 ** -4) * (1 + slack))


def test_block_holding_tensor_amax_gets_scale_448():
    x = _rand_bf16((16, 64), 3)
    x[3, 17] = 123.0
    c, s, g = Q.quantize(x)
    assert g == np.float32(np.float32(123.0) / np.float32(2688.0))
    assert s[3, 1] == 0x7E
    assert abs(F.e2m1_decode(c[3, 17])) == 6.0


def test_zero_tensor_and_zero_block():
    c, s, g = Q.quantize(np.zeros((4, 32), np.float32))
    assert g == 1.0 and not s.any() and not (c & 7).any()
    x = _rand_bf16((4, 64), 4)
    x[:, 16:32] = 0
    c, s, g = Q.quantize(x)
    assert not s[:, 1].any() and not (c[:, 16:32] & 7).any()
    assert np.all(Q.dequantize_f32(c, s, g)[:, 16:32] == 0)


def test_power_of_two_scaling_changes_only_the_tensor_scale():
    x = _rand_bf16((20, 128), 5)
    c, s, g = Q.quantize(x)
    for p in (-7, 3, 12):
        c2, s2, g2 = Q.quantize((x * np.float32(2.0 ** p)).astype(np.float32))
        assert np.array_equal(c2, c) and np.array_equal(s2, s)
        assert g2 == np.float32(g * np.float32(2.0 ** p))


def test_supplied_scale_saturates():
    x = _rand_bf16((8, 64), 6)
    c, s, g = Q.quantize(x, np.float32(1e-6))             # far too small a tensor scale
    assert np.all(s == 0x7E)
    assert np.all(np.abs(F.e2m1_decode(c)) <= 6)


def test_trainer_fake_quant_equals_rollout_dequant_bitwise():
    w = synth.to_bf16(torch.randn(3, 48, 256, generator=torch.Generator().manual_seed(7)) * 0.02)
    w = w.to(torch.float32).numpy()
    w_fq, q, sf, gs = Q.fake_quant_weights(w)
    for i in range(3):
        rollout = Q.dequantize_bf16(F.unpack_nibbles(q[i]), sf[i], gs[i])
        assert np.array_equal(F.bf16_bits(rollout), F.bf16_bits(w_fq[i]))
        # w_fq is a bf16 value
        assert not (w_fq[i].view(np.uint32) & 0xFFFF).any()
    # slices are independent tensors: permuting them permutes the outputs
    w_fq2, q2, sf2, gs2 = Q.fake_quant_weights(w[[2, 0, 1]])
    assert np.array_equal(q2, q[[2, 0, 1]]) and np.array_equal(gs2, gs[[2, 0, 1]])
    assert np.array_equal(sf2, sf[[2, 0, 1]]) and np.array_equal(w_fq2, w_fq[[2, 0, 1]])


def test_fake_quant_error_is_small_relative_to_block_amax():
    w = _rand_bf16((1, 64, 512), 8, 0.015)
    w_fq, q, sf, gs = Q.fake_quant_weights(w)
    blk = np.abs(w[0]).reshape(64, 32, 16).max(axis=2).repeat(16, axis=1)
    # half of the coarsest step (2/6 of amax), E4M3 scale rounding, bf16 rounding
    assert np.all(np.abs(w_fq[0] - w[0]) <= blk * (1 / 6 + 2.0 ** -4 + 2.0 ** -8) + 1e-12)


def test_activation_fake_quant_is_the_decode_of_the_rollout_operand():
    """The learner-side activation QDQ (Table "qdq-alignment") must return what
    the rollout's quantized operand decodes to, leave a representable tensor
    unchanged, stay within half a grid step of the block's own scale, and be a
    projection (applying it twice changes nothing when the scale is kept)."""
    x = _rand_bf16((19, 192), 4, 1.5)
    x[:, 3] *= 25
    xf, g = Q.fake_quant_activations(x)
    c, s, g2 = Q.quantize(x)
    assert g == g2 and np.array_equal(xf, F.bf16_round(Q.dequantize_f32(c, s, g)))
    # error bound: at most half a step of the coarsest E2M1 interval (2 units) times the block scale, + bf16 rounding
    d = Q.block_scales_f32(s, g).astype(np.float64)
    err = np.abs(xf.astype(np.float64) - x.astype(np.float64)).reshape(19, -1, 16)
    assert np.all(err <= d[:, :, None] * 1.0 * (1 + 2.0 ** -7))
    # projection with the scale held fixed
    xf2, _ = Q.fake_quant_activations(Q.dequantize_f32(c, s, g), g)
    assert np.array_equal(xf2, xf)
    # a tensor that is already on the grid (bf16-representable products) comes back bit for bit
    rng = np.random.default_rng(2)
    codes = rng.integers(0, 16, (5, 64)).astype(np.uint8)
    codes[:, ::16] = 7
    sf8 = np.full((5, 4), 0x38, np.uint8)                   # block scale 1.0
    t = Q.dequantize_f32(codes, sf8, np.float32(0.25))
    tf, _ = Q.fake_quant_activations(t, np.float32(0.25))
    assert np.array_equal(tf, t)
