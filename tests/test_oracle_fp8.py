"""Pins for the oracle's FP8 W8A8 comparison path (fine-grained block scaling)."""
import numpy as np
import torch

from oracle import formats as F
from oracle import fp8 as P
from oracle import moe as M
from paper_2607_15810_b200 import synth


def test_scale_is_the_smallest_power_of_two_without_saturation():
    amax = np.array([0.0, 448.0, 448.0001, 447.9, 224.0, 224.1, 1.0, 3.5e-3, 7 * 2.0 ** -20, 1e30], dtype=np.float32)
    e = P.scale_exponent(amax)
    assert e[0] == -127
    for a, ee in zip(amax[1:], e[1:]):
        assert float(a) <= 448.0 * 2.0 ** int(ee)                      # no saturation
        assert float(a) > 448.0 * 2.0 ** (int(ee) - 1)                 # and no smaller exponent would do
    assert list(e[1:6]) == [0, 1, 0, -1, 0]
    # brute force over every bf16 magnitude in a range that crosses many binades
    bits = np.arange(0x3000, 0x4800, dtype=np.uint32) << 16
    a = bits.view(np.float32)
    ee = P.scale_exponent(a)
    want = np.array([min(k for k in range(-40, 40) if float(v) <= 448.0 * 2.0 ** k) for v in a])
    assert np.array_equal(ee, want)


def test_fp8_round_trip_bound_and_torch_elements():
    x, w = synth.dense_inputs(seed=6, T=9, K=256, N=128)
    x, w = x.to(torch.float32).numpy(), w.to(torch.float32).numpy()
    c, e = P.quantize_act(x)
    assert c.shape == (9, 256) and e.shape == (9, 2)
    xd = P.dequantize_act(c, e)
    step = np.repeat(np.ldexp(1.0, e), 128, axis=1)                    # 2^e per element
    # E4M3 relative spacing is 2^-3: error <= half a step of the element's binade, and <= 16 * 2^e overall
    assert np.all(np.abs(xd - x) <= np.maximum(np.abs(x) * 2.0 ** -4, 2.0 ** -10 * step) + 1e-30)
    assert np.all(np.abs(xd) <= 448.0 * step)
    # the element rounding is torch's float8_e4m3fn on the scaled values
    scaled = torch.from_numpy((x.astype(np.float64) / step).astype(np.float32))
    tcodes = scaled.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(c, tcodes)
    # representable tensors survive exactly, whatever tile they sit in
    mags = F.E4M3_MAGNITUDES[8:120:7]
    xe = (np.tile(mags, (3, 16)) * np.array([[2.0 ** -5], [1.0], [2.0 ** 9]])).astype(np.float32)
    xe[:, 0] = 448.0 * np.array([2.0 ** -5, 1.0, 2.0 ** 9])           # pins each row's exponent
    xe[:, 128] = xe[:, 0]
    cc, ee = P.quantize_act(xe)
    assert np.array_equal(P.dequantize_act(cc, ee), xe.astype(np.float64)) and list(ee[:, 0]) == [-5, 0, 9]
    cw, ew = P.quantize_weight(w)
    assert ew.shape == (1, 2)
    wd = P.dequantize_weight(cw, ew)
    assert np.all(np.abs(wd - w) <= np.maximum(np.abs(w) * 2.0 ** -4, 2.0 ** -10 * np.ldexp(1.0, ew).max()))
    # a weight tile's scale follows its own amax only
    w2 = w.copy()
    w2[:, 128:] *= 64
    _, ew2 = P.quantize_weight(w2)
    assert ew2[0, 0] == ew[0, 0] and ew2[0, 1] == ew[0, 1] + 6


def test_fp8_moe_against_explicit_loops():
    shape = synth.MoEShape("t", 24, 7, 128, 3, 2, 128, 0.05, 1, 3.0, 10.0)
    x, _ = synth.activations(shape)
    x = x.to(torch.float32).numpy()
    logits = synth.router_logits(shape).numpy()
    w13 = synth.expert_weights(shape, "w13").to(torch.float32).numpy()
    w2 = synth.expert_weights(shape, "w2").to(torch.float32).numpy()
    q13 = [P.quantize_weight(w13[e]) for e in range(3)]
    q2 = [P.quantize_weight(w2[e]) for e in range(3)]
    W13 = dict(codes=np.stack([q[0] for q in q13]), exps=np.stack([q[1] for q in q13]))
    W2 = dict(codes=np.stack([q[0] for q in q2]), exps=np.stack([q[1] for q in q2]))
    out = P.moe_forward(x, logits, W13, W2, 2)
    ids, wts = M.route(logits, 2, True)
    assert np.array_equal(out["ids"], ids)
    xd = P.dequantize_act(*P.quantize_act(x))
    inv = np.empty(14, int)
    inv[out["perm"]] = np.arange(14)
    want = np.zeros((7, 128))
    for t in range(7):
        for s in range(2):
            e = int(ids[t, s])
            row = inv[t * 2 + s]
            wd = P.dequantize_weight(W13["codes"][e], W13["exps"][e])
            g = np.array([sum(float(a) * float(b) for a, b in zip(xd[t], wr)) for wr in wd])
            assert np.allclose(out["g64"][row], g, rtol=1e-12, atol=1e-15)
            h = np.array([(gi / (1 + np.exp(-gi))) * ui for gi, ui in zip(g[:128], g[128:])])
            assert np.allclose(out["h64"][row], h, rtol=1e-12)
            hb = F.bf16_round(h)[None]
            hd = P.dequantize_act(*P.quantize_act(hb))[0]
            w2d = P.dequantize_weight(W2["codes"][e], W2["exps"][e])
            want[t] += float(wts[t, s]) * np.array([sum(float(a) * float(b) for a, b in zip(hd, wr)) for wr in w2d])
    assert np.allclose(out["out64"], want, rtol=1e-11, atol=1e-14)
    # an overriding h replaces the second half, as in the NVFP4 oracle
    hp = out["h"].copy()
    hp[3, 5] *= 2
    o2 = P.moe_forward(x, logits, W13, W2, 2, h_override=hp)
    assert np.array_equal(o2["h_codes"], P.quantize_act(hp)[0]) and not np.array_equal(o2["out64"], out["out64"])
