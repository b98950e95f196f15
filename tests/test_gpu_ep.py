"""Expert-sharded execution of the MoE layer through the C ABI, the shards of an expert-parallel run
emulated one after the other on one GPU (no kernel waits for another): every shard against the oracle's
shard, the sum of the partial sums against the sum of the oracle's, and the whole-range shard against
the ordinary call bit for bit."""
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import moe_check as MC  # noqa: E402
from oracle import formats as F  # noqa: E402
from oracle import moe as M  # noqa: E402
from oracle import nvfp4 as Q  # noqa: E402
from paper_2607_15810_b200 import ep, synth  # noqa: E402

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_15810_b200 import binding
    return binding


@pytest.mark.parametrize("name,world", [("tiny", 2), ("small", 4), ("small", 3), ("decode", 4)])
def test_expert_shards_match_the_oracle_and_add_up(B, name, world):
    sh = synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    w13o, w2o = MC.oracle_weights(w13), MC.oracle_weights(w2)
    n13, n2 = sh.H // 2, sh.I // 2
    a2 = np.float32(synth.H_GLOBAL_SCALE.get(name, 0.25))
    a2_t = torch.tensor([float(a2)]).cuda()
    xf, lgn = MC.f32(x), lg.numpy()
    parts13, parts2 = [], []
    for e0 in range(0, sh.E, 16):
        ex = range(e0, min(sh.E, e0 + 16))
        parts13.append(B.fake_quant_weights(w13[list(ex)].cuda(), want_fq=False, sf_layout=B.SF_TILED))
        parts2.append(B.fake_quant_weights(w2[list(ex)].cuda(), want_fq=False, sf_layout=B.SF_TILED))
    g13 = {k: torch.cat([p[k] for p in parts13]) for k in ("q", "sf", "gs")}
    g2 = {k: torch.cat([p[k] for p in parts2]) for k in ("q", "sf", "gs")}
    xd, lgd = x.cuda(), lg.cuda()
    total_gpu = torch.zeros(sh.T, sh.H, dtype=torch.float32, device="cuda")
    total_orc = np.zeros((sh.T, sh.H))
    total_abs = np.zeros((sh.T, sh.H))
    for rank in range(world):
        lo, hi = ep.expert_range(rank, world, sh.E)
        part = torch.full((sh.T, sh.H), float("nan"), dtype=torch.float32, device="cuda")
        res = B.moe_w4a4_rac(xd, lgd, ep.shard_weights(g13, lo, hi), ep.shard_weights(g2, lo, hi), sh.topk, n13, n2, a2_t,
                             export=True, expert_range=(lo, hi), out_f32=part)
        torch.cuda.synchronize()
        assert B.moe_async_status(res["workspace"]) == 0
        o1 = M.moe_forward(xf, lgn, w13o, w2o, sh.topk, n13, n2, a2, expert_range=(lo, hi))
        n_local = int(o1["offsets"][hi] - o1["offsets"][lo])
        assert np.array_equal(res["ids"].cpu().numpy(), o1["ids"])
        MC.check_site1(res, o1, n13, {})                          # site 13 is the whole layer's, on every shard
        assert np.array_equal(res["perm"].cpu().numpy()[:n_local], o1["perm"][o1["offsets"][lo]:o1["offsets"][hi]])
        h_gpu = MC.f32(res["h"])[:n_local]
        if n_local:
            I = sh.I
            g, gad = o1["g64"], o1["g_absdot"]
            gate, up = g[:, :I], g[:, I:]
            sig = 1.0 / (1.0 + np.exp(-gate))
            dsilu = sig * (1.0 + gate * (1.0 - sig))
            dg, du = MC.GEMM_RTOL * gad[:, :I], MC.GEMM_RTOL * gad[:, I:]
            tol_h = (np.abs(dsilu * up) * dg + np.abs(gate * sig) * du + dg * du * 2
                     + (MC.BF16_ULP + 1e-5) * np.abs(o1["h64"]) + 1e-30)
            assert float((np.abs(h_gpu - o1["h64"]) / tol_h).max()) <= 1.0
        o2 = M.moe_forward(xf, lgn, w13o, w2o, sh.topk, n13, n2, a2, expert_range=(lo, hi), h_override=h_gpu)
        site2 = o2["site2"]
        assert np.array_equal(res["hq"].cpu().numpy()[:n_local], F.pack_nibbles(site2["codes"]))
        if n_local:
            ok, ndiff = MC.sel_matches(res["sel2"].cpu().numpy(), site2, n2)
            assert ok
            if ndiff:
                o2 = M.moe_forward(xf, lgn, w13o, w2o, sh.topk, n13, n2, a2, expert_range=(lo, hi), h_override=h_gpu,
                                   forced_sel2=res["sel2"].cpu().numpy()[:n2])
            assert np.array_equal(res["r2q"].cpu().numpy()[:n_local], F.pack_nibbles(o2["site2"]["r_codes"]))
        got = part.cpu().numpy().astype(np.float64)
        # (the per-assignment rows are rounded to bf16 before the weighted sum: the bound keeps its bf16 ulp)
        tol = MC.gemm_tol(o2["out_absdot"], o2["out64"]) + 4e-5 * o2["out_absdot"]
        assert float((np.abs(got - o2["out64"]) / tol).max()) <= 1.0
        # tokens without an assignment in this shard contribute exactly zero
        untouched = ~np.isin(o1["ids"], np.arange(lo, hi)).any(axis=1)
        assert not got[untouched].any()
        total_gpu += part
        total_orc += o2["out64"]
        total_abs += o2["out_absdot"]
    got = MC.f32(total_gpu.to(torch.bfloat16)).astype(np.float64)
    tol = MC.gemm_tol(total_abs, total_orc) + 4e-5 * total_abs
    assert float((np.abs(got - total_orc) / tol).max()) <= 1.0
    # the helper that a rank of a real run calls (the all-reduce replaced by the emulated sum)
    acc = {"sum": torch.zeros_like(total_gpu)}

    def fake_all_reduce(t, _acc=acc):
        t.copy_(total_gpu)
    lo, hi = ep.expert_range(0, world, sh.E)
    out = ep.moe_w4a4_rac_expert_parallel(B, xd, lgd, ep.shard_weights(g13, lo, hi), ep.shard_weights(g2, lo, hi), sh.topk,
                                          n13, n2, a2_t, 0, world, all_reduce=fake_all_reduce)
    assert torch.equal(out, total_gpu.to(torch.bfloat16))
    # one shard holding every expert is the ordinary call
    whole32 = torch.empty(sh.T, sh.H, dtype=torch.float32, device="cuda")
    a = B.moe_w4a4_rac(xd, lgd, g13, g2, sh.topk, n13, n2, a2_t, expert_range=(0, sh.E), out_f32=whole32)
    b = B.moe_w4a4_rac(xd, lgd, g13, g2, sh.topk, n13, n2, a2_t)
    assert torch.equal(a["out"], b["out"]) and torch.equal(whole32.to(torch.bfloat16), b["out"])
    # against the unsharded layer the sum differs only through the per-shard site-2 selection (which
    # channels of h get their quantization error corrected): a few per cent of the output at most
    rel = (torch.linalg.norm(total_gpu - whole32) / torch.linalg.norm(whole32)).item()
    print(name, world, "sharded vs unsharded layer, relative difference %.4f" % rel)
    assert rel < 0.1, rel


def test_bad_expert_ranges_are_refused(B):
    sh = synth.MOE_SHAPES["tiny"]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    g13 = B.fake_quant_weights(synth.expert_weights(sh, "w13").cuda(), want_fq=False, sf_layout=B.SF_TILED)
    g2 = B.fake_quant_weights(synth.expert_weights(sh, "w2").cuda(), want_fq=False, sf_layout=B.SF_TILED)
    a2 = torch.tensor([0.25]).cuda()
    for rng_ in ((-1, 2), (4, sh.E + 1)):
        with pytest.raises(B.QuadsError) as e:
            B.moe_w4a4_rac(x.cuda(), lg.cuda(), g13, g2, sh.topk, 8, 8, a2, expert_range=rng_)
        assert e.value.status == -2
