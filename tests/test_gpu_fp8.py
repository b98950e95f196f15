"""FP8 W8A8 comparison path against its oracle through the C ABI: quantizers bit for bit, the grouped
block-scaled FP8 GEMMs within the GEMM tolerance (staged like the NVFP4 layer: the requantization of h
is checked on the implementation's own h)."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import fp8 as P
from paper_2607_15810_b200 import synth

pytestmark = pytest.mark.gpu
GEMM_RTOL, BF16_ULP = 2e-3, 2.0 ** -7


@pytest.fixture(scope="module")
def B():
    from paper_2607_15810_b200 import binding
    return binding


def _f32(t):
    return t.to(torch.float32).cpu().numpy()


def _oracle_weights(w):
    qs = [P.quantize_weight(_f32(w[e])) for e in range(w.shape[0])]
    return dict(codes=np.stack([q[0] for q in qs]), exps=np.stack([q[1] for q in qs]))


@pytest.mark.parametrize("n,N,K,scale", [(1, 128, 128, 1.0), (3, 256, 384, 0.02), (2, 1536, 2048, 0.02)])
def test_fp8_weight_quantizer_bit_exact(B, n, N, K, scale):
    w = (torch.randn(n, N, K, generator=torch.Generator().manual_seed(n + N)) * scale).to(torch.bfloat16)
    w[0, :64, :64] *= 300.0                                   # tiles with very different scales
    w[0, 64:128, 64:128] = 0
    r = B.fp8_quantize_weights(w.cuda())
    o = _oracle_weights(w)
    assert np.array_equal(r["exps"].cpu().numpy().astype(np.int32) - 127, o["exps"])
    assert np.array_equal(r["q"].cpu().numpy(), o["codes"])
    at = r["atoms"].cpu().numpy()
    assert np.array_equal(at, np.broadcast_to(r["exps"].cpu().numpy()[..., None], at.shape))


def _layer(B, sh, full=True):
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    g13, g2 = B.fp8_quantize_weights(w13.cuda()), B.fp8_quantize_weights(w2.cuda())
    res = B.moe_fp8_w8a8(x.cuda(), lg.cuda(), g13, g2, sh.topk, export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    o13, o2 = _oracle_weights(w13), _oracle_weights(w2)
    assert np.array_equal(g13["q"].cpu().numpy(), o13["codes"]) and np.array_equal(g2["q"].cpu().numpy(), o2["codes"])
    orc = P.moe_forward(_f32(x), lg.numpy(), o13, o2, sh.topk)
    I = sh.I
    assert np.array_equal(res["ids"].cpu().numpy(), orc["ids"]) and np.array_equal(res["perm"].cpu().numpy(), orc["perm"])
    assert np.array_equal(res["xq"].cpu().numpy(), orc["x_codes"])
    assert np.array_equal(res["xexp"].cpu().numpy().astype(np.int32) - 127, orc["x_exps"])
    # h within the propagated GEMM tolerance
    h_gpu = _f32(res["h"])
    g, gad = orc["g64"], orc["g_absdot"]
    gate, up = g[:, :I], g[:, I:]
    sig = 1.0 / (1.0 + np.exp(-gate))
    dsilu = sig * (1.0 + gate * (1.0 - sig))
    dg, du = GEMM_RTOL * gad[:, :I], GEMM_RTOL * gad[:, I:]
    tol_h = np.abs(dsilu * up) * dg + np.abs(gate * sig) * du + 2 * dg * du + (BF16_ULP + 1e-5) * np.abs(orc["h64"]) + 1e-30
    rh = float((np.abs(h_gpu - orc["h64"]) / tol_h).max())
    assert rh <= 1.0, rh
    # requantization of the implementation's own h, bit for bit
    orc2 = P.moe_forward(_f32(x), lg.numpy(), o13, o2, sh.topk, h_override=h_gpu)
    assert np.array_equal(res["hq"].cpu().numpy(), orc2["h_codes"])
    assert np.array_equal(res["hexp"].cpu().numpy().astype(np.int32) - 127, orc2["h_exps"])
    out = _f32(res["out"]).astype(np.float64)
    tol_o = (GEMM_RTOL + 4e-5) * orc2["out_absdot"] + BF16_ULP * np.abs(orc2["out64"]) + 1e-30
    ro = float((np.abs(out - orc2["out64"]) / tol_o).max())
    assert ro <= 1.0, ro
    rel = np.linalg.norm(out - orc["out64"]) / (np.linalg.norm(orc["out64"]) + 1e-30)
    assert rel <= 1e-2
    # the export-free call gives the same bits
    res2 = B.moe_fp8_w8a8(x.cuda(), lg.cuda(), g13, g2, sh.topk)
    assert torch.equal(res2["out"], res["out"])
    return rh, ro


FP8_SHAPES = [synth.MOE_SHAPES["tiny"], synth.MOE_SHAPES["small"],
              synth.MoEShape("one_token", 31, 1, 128, 256, 1, 128, 0.05, 1, 3.0, 10.0),
              synth.MoEShape("k_tail", 34, 70, 384, 4, 2, 128, 0.05, 2, 3.0, 10.0),
              synth.MoEShape("many_tiles", 35, 2100, 256, 4, 2, 384, 0.05, 1, 3.0, 10.0)]


@pytest.mark.parametrize("shape", FP8_SHAPES, ids=[s.name for s in FP8_SHAPES])
def test_fp8_layer_against_the_oracle(B, shape):
    rh, ro = _layer(B, shape)
    print(shape.name, "h err/tol %.3f out err/tol %.3f" % (rh, ro))


def test_fp8_decode_layer_in_full(B):
    _layer(B, synth.MOE_SHAPES["decode"])
