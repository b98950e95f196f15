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


def test_fp8_prefill_layer_at_full_size_sampled(B):
    """The FP8 arm at the size the benchmark times it (prefill, T = 8192, skewed routing): integer stages
    in full, the two GEMMs on sampled outputs (every expert hit, >= 512 dispatched rows), the oracle
    quantizing each expert's sampled weight rows once (a weight tile's scale needs the whole 128 x 128
    tile, so whole 128-row groups are quantized and the sampled rows taken from them)."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    import moe_check as MC
    from oracle import moe as M
    sh = synth.MOE_SHAPES["prefill"]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    parts13, parts2 = [], []
    for e0 in range(0, sh.E, 16):
        ex = range(e0, e0 + 16)
        parts13.append(B.fp8_quantize_weights(synth.expert_weights(sh, "w13", ex).cuda()))
        parts2.append(B.fp8_quantize_weights(synth.expert_weights(sh, "w2", ex).cuda()))
    g13 = {k: torch.cat([p[k] for p in parts13]) for k in ("q", "exps", "atoms")}
    g2 = {k: torch.cat([p[k] for p in parts2]) for k in ("q", "exps", "atoms")}
    res = B.moe_fp8_w8a8(x.cuda(), lg.cuda(), g13, g2, sh.topk, export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    T, H, I, topk, E = sh.T, sh.H, sh.I, sh.topk, sh.E
    xf, lgn = _f32(x), lg.numpy()
    ids, wts = M.route(lgn, topk, True)
    counts, offsets, perm = M.dispatch(ids, E)
    assert np.array_equal(res["ids"].cpu().numpy(), ids) and np.array_equal(res["perm"].cpu().numpy(), perm)
    xc, xe = P.quantize_act(xf)
    assert np.array_equal(res["xq"].cpu().numpy(), xc)
    assert np.array_equal(res["xexp"].cpu().numpy().astype(np.int32) - 127, xe)
    h_gpu = _f32(res["h"])
    hc, he = P.quantize_act(h_gpu)                               # requantization of the implementation's own h, in full
    assert np.array_equal(res["hq"].cpu().numpy(), hc)
    assert np.array_equal(res["hexp"].cpu().numpy().astype(np.int32) - 127, he)
    xd, hd = P.dequantize_act(xc, xe), P.dequantize_act(hc, he)
    tokens, extra = MC.sample_plan(ids, offsets, topk, sh.hot_experts, 64, 8, 7)
    inv = np.empty(T * topk, dtype=np.int64)
    inv[perm] = np.arange(T * topk)
    tok_rows = {int(inv[t * topk + s]): (t, s) for t in tokens for s in range(topk)}
    rows = sorted(set(extra) | set(tok_rows))
    assert len(rows) >= 512
    row_expert = np.searchsorted(offsets, np.asarray(rows), side="right") - 1
    tok_of = perm // topk
    rng = np.random.default_rng(11)
    ftile = rng.integers(0, I // 128, size=E)                    # one 128-feature tile of h per expert ...
    ctile = rng.integers(0, H // 128, size=E)                    # ... and one 128-column tile of out
    out_gpu = _f32(res["out"]).astype(np.float64)
    worst_h = 0.0
    o64 = {t: {} for t in tokens}
    for e in sorted(set(int(v) for v in row_expert)):
        mine = np.asarray([r for r, re_ in zip(rows, row_expert) if re_ == e])
        w13 = _f32(synth.expert_weights(sh, "w13", [e])[0])
        f0 = int(ftile[e]) * 128
        wg = P.dequantize_weight(*P.quantize_weight(w13[f0:f0 + 128]))
        wu = P.dequantize_weight(*P.quantize_weight(w13[I + f0:I + f0 + 128]))
        xs = xd[tok_of[mine]]
        gate, up = xs @ wg.T, xs @ wu.T
        gad_g, gad_u = np.abs(xs) @ np.abs(wg).T, np.abs(xs) @ np.abs(wu).T
        sig = 1.0 / (1.0 + np.exp(-gate))
        h64 = gate * sig * up
        dsilu = sig * (1.0 + gate * (1.0 - sig))
        dg, du = GEMM_RTOL * gad_g, GEMM_RTOL * gad_u
        tol_h = np.abs(dsilu * up) * dg + np.abs(gate * sig) * du + 2 * dg * du + (BF16_ULP + 1e-5) * np.abs(h64) + 1e-30
        worst_h = max(worst_h, float((np.abs(h_gpu[mine][:, f0:f0 + 128] - h64) / tol_h).max()))
        mine_tok = [int(r) for r in mine if int(r) in tok_rows]
        if mine_tok:
            w2 = _f32(synth.expert_weights(sh, "w2", [e])[0])
            for c0 in sorted({int(ctile[int(ids[tok_rows[r][0], s])]) * 128 for r in mine_tok for s in range(topk)}):
                w2d = P.dequantize_weight(*P.quantize_weight(w2[c0:c0 + 128]))
                y = hd[np.asarray(mine_tok)] @ w2d.T
                ya = np.abs(hd[np.asarray(mine_tok)]) @ np.abs(w2d).T
                for k, r in enumerate(mine_tok):
                    t, s_ = tok_rows[r]
                    acc = o64[t].setdefault(c0, [np.zeros(128), np.zeros(128), 0])
                    acc[0] += float(wts[t, s_]) * y[k]
                    acc[1] += float(wts[t, s_]) * ya[k]
                    acc[2] += 1
    worst_o, n_out = 0.0, 0
    for t in tokens:
        for c0, (v, va, n) in o64[t].items():
            if n != topk:
                continue                                          # column tile not accumulated over all of the token's experts
            tol = (GEMM_RTOL + 4e-5) * va + BF16_ULP * np.abs(v) + 1e-30
            worst_o = max(worst_o, float((np.abs(out_gpu[t, c0:c0 + 128] - v) / tol).max()))
            n_out += 128
    print("fp8 prefill: rows %d, h err/tol %.3f, out values %d err/tol %.3f" % (len(rows), worst_h, n_out, worst_o))
    assert worst_h <= 1.0 and worst_o <= 1.0 and n_out >= 64 * 128
