"""CUDA W4A4+RAC projections against the oracle through the C ABI: the dense
config, small MoE layers compared in full, and the decode / prefill / large
configs at full size."""
import os
import random
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import moe_check as MC  # noqa: E402
from oracle import formats as F  # noqa: E402
from oracle import moe as M  # noqa: E402
from oracle import nvfp4 as Q  # noqa: E402
from paper_2607_15810_b200 import synth  # noqa: E402

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_15810_b200 import binding
    return binding


def _dense_case(B, x, w, nsel):
    wq = B.fake_quant_weights(w.unsqueeze(0).cuda(), want_fq=False, sf_layout=B.SF_TILED)
    res = B.dense_w4a4_rac(x.cuda(), wq, nsel, export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    wo = MC.oracle_weights(w[None])
    o = M.dense_w4a4_rac(MC.f32(x), wo["codes"][0], wo["sf"][0], wo["gs"][0], nsel)
    MC.check_site1(res, dict(site13=o["site"]), nsel, {})
    got = MC.f32(res["out"]).astype(np.float64)
    ratio = float((np.abs(got - o["y64"]) / MC.gemm_tol(o["absdot"], o["y64"])).max())
    assert ratio <= 1.0, ratio
    return ratio


@pytest.mark.parametrize("nsel", [0, 16, 64, 128, 256, 384, 512])
def test_dense_config_all_ratios(B, nsel):
    """Config "single dense W4A4+RAC GEMM" (n_sel = 16) and the paper's channel
    ratios 12.5 .. 100 % of K = 512."""
    x, w = synth.dense_inputs(seed=0)
    _dense_case(B, x, w, nsel)


@pytest.mark.parametrize("T,K,N,nsel,seed", [(1, 128, 128, 8, 1), (200, 640, 384, 64, 5), (300, 2048, 512, 1024, 6),
                                             (129, 384, 128, 96, 7),
                                             # the widest layer the library takes (K = 16384: 64 pipeline stages
                                             # per tile, 128 KB of score keys in the selection kernel)
                                             (64, 16384, 128, 4096, 8)])
def test_dense_ragged_shapes(B, T, K, N, nsel, seed):
    x, w = synth.dense_inputs(seed, T=T, K=K, N=N)
    _dense_case(B, x, w, nsel)


def test_dense_exact_integer_case(B):
    """Integer-valued operands with unit scales: the tensor-core result must be
    the exact small-integer product."""
    rng = np.random.default_rng(3)
    ints = np.array([0, 1, 2, 3, 4, 6, -1, -2, -3, -4, -6], dtype=np.float32)
    a = rng.choice(ints, (128, 256)).astype(np.float32)
    b = rng.choice(ints, (128, 256)).astype(np.float32)
    a[:, ::16] = 6
    b[:, ::16] = 6
    gs = torch.tensor([1.0]).cuda()
    x = torch.from_numpy(a).to(torch.bfloat16)
    b = b * 7.0   # weight amax 42 -> tensor scale 42/2688 = 2^-6 and block scales 448: every factor is exact
    w = torch.from_numpy(b).to(torch.bfloat16)
    wq = B.fake_quant_weights(w.unsqueeze(0).cuda(), want_fq=False, sf_layout=B.SF_TILED)
    res = B.dense_w4a4_rac(x.cuda(), wq, 0, a_gs=gs)
    want = a.astype(np.float64) @ b.astype(np.float64).T
    got = MC.f32(res["out"]).astype(np.float64)
    assert np.array_equal(got, MC.f32(torch.from_numpy(want).to(torch.bfloat16)).astype(np.float64))


def test_dense_at_the_size_where_cta_pairs_are_chosen(B):
    """From 1024 rows per weight matrix the call takes the CTA-pair kernel (256 x 256 tiles,
    cta_group::2) on its own; compared element by element with the oracle, ragged last pair."""
    x, w = synth.dense_inputs(seed=9, T=2300, K=1024, N=640)
    ratio = _dense_case(B, x, w, 512)
    print("cta-pair dense 2300x1024x640: worst err / tol = %.3f" % ratio)


def _sweep_operands():
    """Operands in which every finite non-negative E4M3 scale code and every E2M1 nibble occurs on
    both sides of the tensor-core product, laid out so that a single wrong decode shows: weight row
    n is non-zero in block n only, hence out[t, n] is the 16-term product of activation block
    (t, n) and weight block n, all terms of one sign.  Values are exactly representable (<= 6
    significant bits), so the quantizers reproduce the chosen codes."""
    mags = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6], dtype=np.float64)
    sf = F.E4M3_MAGNITUDES[:127].astype(np.float64)             # codes 0x00 .. 0x7E
    T, NB = 128, 128
    K = NB * 16
    a_gs, w_gs = 2.0 ** -6, 2.0 ** -10
    i = np.arange(16)
    sgn = np.where(i < 8, 1.0, -1.0)
    x = np.zeros((T, K))
    w = np.zeros((NB, K))
    for n in range(NB):
        w[n, 16 * n:16 * n + 16] = sgn * mags[(i + n) % 8] * sf[n % 127] * w_gs
        for t in range(T):
            x[t, 16 * n:16 * n + 16] = sgn * mags[(i + t) % 8] * sf[(t + n) % 127] * a_gs
    xb, wb = torch.from_numpy(x).to(torch.bfloat16), torch.from_numpy(w).to(torch.bfloat16)
    assert np.array_equal(xb.to(torch.float64).numpy(), x) and np.array_equal(wb.to(torch.float64).numpy(), w)
    return xb, wb, np.float32(a_gs), np.float32(w_gs)


def test_tensor_cores_decode_every_scale_code_and_every_nibble(B):
    xb, wb, a_gs, w_gs = _sweep_operands()
    wo = MC.oracle_weights(wb[None])
    assert wo["gs"][0] == w_gs                                  # amax = 6 * 448 * w_gs
    o = M.dense_w4a4_rac(MC.f32(xb), wo["codes"][0], wo["sf"][0], wo["gs"][0], 0, a_gs=a_gs)
    # the sweep really covers the code space on both sides
    assert set(o["site"]["sf"].reshape(-1).tolist()) == set(range(127))
    assert set(np.diag(wo["sf"][0][:, :128]).tolist()) == set(range(127))
    w_blocks = np.stack([wo["codes"][0][n, 16 * n:16 * n + 16] for n in range(128)])
    for side in (o["site"]["codes"], w_blocks):
        assert set(side.reshape(-1).tolist()) >= set(range(1, 8)) | set(range(9, 16))
    wq = B.fake_quant_weights(wb.unsqueeze(0).cuda(), want_fq=False, sf_layout=B.SF_TILED)
    assert np.array_equal(wq["q"].cpu().numpy(), wo["q"])
    res = B.dense_w4a4_rac(xb.cuda(), wq, 0, a_gs=torch.tensor([float(a_gs)]).cuda(), export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    MC.check_site1(res, dict(site13=o["site"]), 0, {})
    got = MC.f32(res["out"]).astype(np.float64)
    # all products of an output have one sign: sum|a b| = |y|, so the bound is 2e-3 |y| + one bf16 ulp,
    # while a mis-decoded scale byte or nibble changes y by at least 1/16 of itself
    assert np.allclose(o["absdot"], np.abs(o["y64"]), rtol=1e-12)
    ratio = float((np.abs(got - o["y64"]) / MC.gemm_tol(o["absdot"], o["y64"])).max())
    assert ratio <= 1.0, ratio
    exact = float((got == MC.f32(torch.from_numpy(o["y64"]).to(torch.bfloat16))).mean())
    print("scale/nibble sweep: worst err / tol = %.3f, outputs equal to the rounded exact value: %.4f" % (ratio, exact))
    # with every channel compensated nothing changes: the residual of exactly representable values is zero
    res_k = B.dense_w4a4_rac(xb.cuda(), wq, xb.shape[1], a_gs=torch.tensor([float(a_gs)]).cuda())
    assert torch.equal(res_k["out"], res["out"])


def _moe_small(B, name, f13, f2, renorm, shape=None):
    sh = shape if shape is not None else synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    w13o, w2o = MC.oracle_weights(w13), MC.oracle_weights(w2)
    nsel13, nsel2 = int(sh.H * f13), int(sh.I * f2)
    pilot = M.moe_forward(MC.f32(x), lg.numpy(), w13o, w2o, sh.topk, nsel13, 0, np.float32(1.0), renormalize=renorm)
    a2 = Q.tensor_global_scale(pilot["h"])
    gw13 = B.fake_quant_weights(w13.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(w2.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    assert np.array_equal(gw13["q"].cpu().numpy(), w13o["q"]) and np.array_equal(gw2["q"].cpu().numpy(), w2o["q"])
    res = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, nsel13, nsel2, torch.tensor([a2]).cuda(),
                         renormalize=renorm, export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    rep = MC.check_moe(res, x, lg, w13o, w2o, sh.topk, nsel13, nsel2, a2, renormalize=renorm)
    # the export-free call gives the same output bits (every reduction runs in a fixed order)
    res2 = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, nsel13, nsel2, torch.tensor([a2]).cuda(),
                          renormalize=renorm)
    assert torch.equal(res2["out"], res["out"])
    return rep


@pytest.mark.parametrize("name,f13,f2,renorm", [("tiny", 0.5, 0.5, True), ("tiny", 0.0, 0.0, True),
                                                ("tiny", 1.0, 1.0, False), ("small", 0.5, 0.5, True),
                                                ("small", 0.25, 0.0, False), ("small", 0.0, 0.5, True)])
def test_moe_small_layers_in_full(B, name, f13, f2, renorm):
    _moe_small(B, name, f13, f2, renorm)


EDGE_SHAPES = [
    # one token, one choice out of many experts: 255 empty experts, a tile with a single valid row
    synth.MoEShape("one_token", 31, 1, 128, 256, 1, 128, 0.05, 1, 3.0, 10.0),
    # fewer tokens than experts, the widest top-k the library takes
    synth.MoEShape("top16", 32, 9, 256, 32, 16, 128, 0.05, 2, 3.0, 10.0),
    # a single expert owning several full tiles plus a ragged one (all rows in one segment)
    synth.MoEShape("one_expert", 33, 300, 128, 1, 1, 256, 0.05, 1, 3.0, 10.0),
    # K tails: H and I that are not multiples of the 256-element pipeline stage
    synth.MoEShape("k_tail", 34, 70, 384, 4, 2, 128, 0.05, 2, 3.0, 10.0),
    # more than 256 routing chunks (second pass of the per-expert chunk scan), dozens of tiles per expert
    synth.MoEShape("many_chunks", 35, 8300, 128, 4, 2, 128, 0.05, 1, 3.0, 10.0),
    # few rows per expert on average (operand-swapped GEMMs) but one hot expert whose slot uses
    # both 64-row halves and a second slot
    synth.MoEShape("hot_expert_few_rows", 36, 200, 256, 16, 2, 128, 0.05, 2, 3.0, 10.0, 1, 0.45),
]


@pytest.mark.parametrize("shape", EDGE_SHAPES, ids=[s.name for s in EDGE_SHAPES])
def test_moe_edge_shapes(B, shape):
    _moe_small(B, None, 0.5, 0.5, True, shape=shape)


def _random_shape(seed):
    rng = random.Random(seed)
    E = rng.choice([1, 2, 3, 5, 8, 16, 24, 32, 64])
    topk = rng.randint(1, min(E, 8))
    T = rng.choice([1, 2, 7, 31, 64, 129, 200, 257, 400, 777])
    H = 128 * rng.choice([1, 2, 3, 4, 5, 8])
    I = 128 * rng.choice([1, 2, 3, 4])
    hot = min(rng.choice([0, 0, 1, 2]), E)
    sh = synth.MoEShape("random%d" % seed, 1000 + seed, T, H, E, topk, I, 0.05, rng.randint(0, 4), 3.0, 10.0,
                        hot, 0.5 if hot else 0.0)
    return sh, rng.choice([0.0, 0.25, 0.5, 1.0]), rng.choice([0.0, 0.5, 1.0]), rng.random() < 0.5


@pytest.mark.parametrize("seed", range(16))
def test_moe_random_shapes(B, seed):
    """Seeded random layer shapes, expert counts, top-k, hot experts, compensation ratios: the whole layer
    against the oracle as in the named cases above."""
    sh, f13, f2, renorm = _random_shape(seed)
    _moe_small(B, None, f13, f2, renorm, shape=sh)


def test_zero_tokens_is_a_no_op(B):
    sh = synth.MOE_SHAPES["tiny"]
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    gw13 = B.fake_quant_weights(w13.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(w2.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    x = torch.empty(0, sh.H, dtype=torch.bfloat16).cuda()
    lg = torch.empty(0, sh.E, dtype=torch.float32).cuda()
    res = B.moe_w4a4_rac(x, lg, gw13, gw2, sh.topk, 8, 8, torch.tensor([0.1]).cuda())
    assert res["out"].shape == (0, sh.H)


def test_bad_arguments_are_refused(B):
    sh = synth.MOE_SHAPES["tiny"]
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    gw13 = B.fake_quant_weights(w13.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(w2.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    a2 = torch.tensor([0.1]).cuda()
    with pytest.raises(B.QuadsError) as e:                      # more compensated channels than channels
        B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, sh.H + 1, 0, a2)
    assert e.value.status == -2
    with pytest.raises(B.QuadsError) as e:                      # workspace too small
        B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, 8, 8, a2,
                       workspace=torch.empty(1024, dtype=torch.uint8).cuda())
    assert e.value.status == -3
    with pytest.raises(B.QuadsError) as e:                      # top-k larger than the expert count
        B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.E + 1, 8, 8, a2)
    assert e.value.status == -2


_W = {}


def _gpu_weights(B, sh):
    key = (sh.weight_seed if sh.weight_seed >= 0 else sh.seed, sh.H, sh.I, sh.E)
    if key not in _W:
        out = {}
        for which in ("w13", "w2"):
            parts = []
            for e0 in range(0, sh.E, 16):
                w = synth.expert_weights(sh, which, range(e0, min(sh.E, e0 + 16)))
                parts.append(B.fake_quant_weights(w.cuda(), want_fq=False, sf_layout=B.SF_TILED))
            out[which] = {k: torch.cat([p[k] for p in parts]) for k in ("q", "sf", "gs")}
        _W.clear()
        _W[key] = out
    return _W[key]["w13"], _W[key]["w2"]


@pytest.mark.parametrize("name,variant", [("decode", "both"), ("prefill", "both"), ("prefill", "w13"),
                                          ("prefill", "plain"), ("large", "both")])
def test_moe_full_size_sampled(B, name, variant):
    """The benchmark configurations at full size, in the launch configuration
    the benchmark times; GEMM outputs are compared on sampled tokens."""
    sh = synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    gw13, gw2 = _gpu_weights(B, sh)
    nsel13 = 0 if variant == "plain" else sh.H // 2
    nsel2 = sh.I // 2 if variant == "both" else 0
    a2 = np.float32(synth.H_GLOBAL_SCALE[name])
    res = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, nsel13, nsel2, torch.tensor([a2]).cuda(),
                         export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    if sh.hot_experts:
        ids = res["ids"].cpu().numpy()
        share = float((ids < sh.hot_experts).mean())
        assert abs(share - sh.hot_share) <= 0.005
    # >= 512 dispatched rows over every expert, the first and last tile of every hot expert and the last
    # wave of tiles; the variants other than the benchmarked one take a lighter plan (they share the kernels)
    heavy = variant == "both"
    rep = MC.check_moe_sampled(res, x, lg, sh,
                               lambda e: synth.expert_weights(sh, "w13", [e])[0],
                               lambda e: synth.expert_weights(sh, "w2", [e])[0],
                               nsel13, nsel2, a2, n_tokens=64 if heavy else 16, n_features=96 if heavy else 48,
                               n_columns=128 if heavy else 64, tail_experts=8 if heavy else 2)
    assert rep["h_max_err_over_tol"] <= 1 and rep["out_max_err_over_tol"] <= 1
    assert rep["sampled_experts"] == sh.E
    if heavy:
        assert rep["sampled_rows"] >= 512 and rep["sampled_tokens"] >= 64
    print(name, variant, rep)
    for k in ("xq", "rq", "h", "hq", "r2q"):
        res.pop(k)


def test_decode_layer_in_full(B):
    """Config "MoE layer decode" compared element by element in full."""
    sh = synth.MOE_SHAPES["decode"]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    w13o, w2o = MC.oracle_weights(w13), MC.oracle_weights(w2)
    gw13, gw2 = _gpu_weights(B, sh)
    assert np.array_equal(gw13["q"].cpu().numpy(), w13o["q"]) and np.array_equal(gw13["gs"].cpu().numpy(), w13o["gs"])
    assert np.array_equal(gw2["q"].cpu().numpy(), w2o["q"]) and np.array_equal(gw2["gs"].cpu().numpy(), w2o["gs"])
    a2 = np.float32(synth.H_GLOBAL_SCALE["decode"])
    nsel13, nsel2 = sh.H // 2, sh.I // 2
    res = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, nsel13, nsel2, torch.tensor([a2]).cuda(),
                         export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    MC.check_moe(res, x, lg, w13o, w2o, sh.topk, nsel13, nsel2, a2)


def test_cta_pair_gemm_variant_in_a_subprocess():
    """The optional CTA-pair GEMM (cta_group::2, selected by an environment
    variable read once per process) passes the same dense and small-layer
    parity cases."""
    import subprocess
    env = dict(os.environ, QUADS_GEMM_CTA_GROUP="2")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-m", "pytest", os.path.join(root, "tests", "test_gpu_moe.py"), "-x", "-q", "-m",
                        "gpu", "-k", "dense_config_all_ratios or dense_ragged or small_layers or edge_shapes"],
                       cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0, r.stdout[-3000:]


def test_moe_call_is_capturable_in_a_cuda_graph(B):
    """The layer call allocates nothing and never synchronises, so (after one
    eager call has set the kernels' attributes) it can be captured into a CUDA
    graph; replays on new inputs reproduce the eager results bit for bit."""
    sh = synth.MOE_SHAPES["tiny"]
    w13 = synth.expert_weights(sh, "w13")
    w2 = synth.expert_weights(sh, "w2")
    gw13 = B.fake_quant_weights(w13.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(w2.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    x0, _ = synth.activations(sh)
    lg0 = synth.router_logits(sh)
    a2 = torch.tensor([0.25], device="cuda")
    nsel13, nsel2 = sh.H // 2, sh.I // 2
    ws = torch.empty(B.moe_workspace_bytes(sh.T, sh.H, sh.I, sh.E, sh.topk), dtype=torch.uint8, device="cuda")
    x_s, lg_s = x0.cuda().clone(), lg0.cuda().clone()
    out_s = torch.empty(sh.T, sh.H, dtype=torch.bfloat16, device="cuda")

    def call(x, lg, out):
        B.moe_w4a4_rac(x, lg, gw13, gw2, sh.topk, nsel13, nsel2, a2, workspace=ws, out=out)

    inputs = []
    g = torch.Generator().manual_seed(77)
    for i in range(3):
        x = (x0.float() * (1.0 + 0.1 * i) + 0.01 * torch.randn(x0.shape, generator=g)).to(torch.bfloat16)
        lg = lg0 + 0.5 * torch.randn(lg0.shape, generator=g)
        inputs.append((x.cuda(), lg.cuda()))
    eager = []
    for x, lg in inputs:
        o = torch.empty_like(out_s)
        call(x, lg, o)
        torch.cuda.synchronize()
        eager.append(o.clone())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call(x_s, lg_s, out_s)
    for (x, lg), want in zip(inputs, eager):
        x_s.copy_(x)
        lg_s.copy_(lg)
        graph.replay()
        torch.cuda.synchronize()
        assert B.moe_async_status(ws) == 0
        assert torch.equal(out_s, want)


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_moe_with_a_static_activation_scale(B, name):
    """Caller-supplied per-tensor scale for x (no amax pass), chosen at half of
    the amax-derived one so that the largest activations saturate."""
    sh = synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    w13o, w2o = MC.oracle_weights(w13), MC.oracle_weights(w2)
    nsel13, nsel2 = sh.H // 2, sh.I // 4
    a13 = np.float32(0.5) * Q.tensor_global_scale(MC.f32(x))
    pilot = M.moe_forward(MC.f32(x), lg.numpy(), w13o, w2o, sh.topk, nsel13, 0, np.float32(1.0), a13_gs=a13)
    a2 = Q.tensor_global_scale(pilot["h"])
    gw13 = B.fake_quant_weights(w13.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(w2.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    res = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, nsel13, nsel2, torch.tensor([a2]).cuda(),
                         a13_gs=torch.tensor([a13]).cuda(), export=True)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    MC.check_moe(res, x, lg, w13o, w2o, sh.topk, nsel13, nsel2, a2, a13_gs=a13)


@pytest.mark.parametrize("name", ["tiny", "small"])
def test_workspace_content_does_not_matter(B, name):
    """The caller-owned workspace may hold anything on entry: a call on a
    workspace filled with 0xFF bytes gives the bits of a call on a zeroed one
    (both GEMM families: few rows per expert and the row-major tiles)."""
    sh = synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    gw13 = B.fake_quant_weights(synth.expert_weights(sh, "w13").cuda(), want_fq=False, sf_layout=B.SF_TILED)
    gw2 = B.fake_quant_weights(synth.expert_weights(sh, "w2").cuda(), want_fq=False, sf_layout=B.SF_TILED)
    a2 = torch.tensor([0.25]).cuda()
    n = B.moe_workspace_bytes(sh.T, sh.H, sh.I, sh.E, sh.topk)
    outs = []
    for fill in (0, 255, 0x5A):
        ws = torch.full((n + 4096,), fill, dtype=torch.uint8, device="cuda")
        res = B.moe_w4a4_rac(x.cuda(), lg.cuda(), gw13, gw2, sh.topk, sh.H // 2, sh.I // 2, a2, workspace=ws, export=True)
        torch.cuda.synchronize()
        assert B.moe_async_status(ws) == 0
        outs.append({k: v.clone() for k, v in res.items() if isinstance(v, torch.Tensor) and k != "workspace"})
    for other in outs[1:]:
        for k, v in outs[0].items():
            assert torch.equal(v, other[k]), k


@pytest.mark.parametrize("name", ["small", "decode"])
def test_results_are_reproducible_bit_for_bit(B, name):
    """No floating-point atomics anywhere on the path: every reduction runs in a
    fixed order, so repeated calls on the same inputs give identical bits (row-major
    GEMMs for `small`, operand-swapped GEMMs for `decode`)."""
    sh = synth.MOE_SHAPES[name]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    parts13, parts2 = [], []
    for e0 in range(0, sh.E, 16):
        ex = range(e0, min(sh.E, e0 + 16))
        parts13.append(B.fake_quant_weights(synth.expert_weights(sh, "w13", ex).cuda(), want_fq=False, sf_layout=B.SF_TILED))
        parts2.append(B.fake_quant_weights(synth.expert_weights(sh, "w2", ex).cuda(), want_fq=False, sf_layout=B.SF_TILED))
    gw13 = {k: torch.cat([p[k] for p in parts13]) for k in ("q", "sf", "gs")}
    gw2 = {k: torch.cat([p[k] for p in parts2]) for k in ("q", "sf", "gs")}
    a2 = torch.tensor([synth.H_GLOBAL_SCALE.get(name, 0.25)]).cuda()
    xd, lgd = x.cuda(), lg.cuda()
    ws = torch.empty(B.moe_workspace_bytes(sh.T, sh.H, sh.I, sh.E, sh.topk), dtype=torch.uint8, device="cuda")
    first = None
    for i in range(6):
        res = B.moe_w4a4_rac(xd, lgd, gw13, gw2, sh.topk, sh.H // 2, sh.I // 2, a2, workspace=ws)
        torch.cuda.synchronize()
        assert B.moe_async_status(ws) == 0
        if first is None:
            first = res["out"].clone()
        else:
            assert torch.equal(res["out"], first), "call %d differs" % i


def test_compensating_more_channels_shrinks_the_mismatch_against_the_learner(B):
    """Property at a size the oracle does not reach: against the learner's
    QDQ_W(W) x in float32 (a library GEMM, independent of this code), the
    W4A4 + RAC projection gets closer as the share of compensated channels
    grows, full compensation removes most of the activation error, and no
    compensation equals plain W4A4 (Table "channel-ratio" states the trend)."""
    T, K, N = 1024, 2048, 1024
    g = torch.Generator().manual_seed(5)
    x = torch.randn(T, K, generator=g)
    x[:, torch.randperm(K, generator=g)[: K // 50]] *= 25.0
    x = x.to(torch.bfloat16).cuda()
    w = B.fake_quant_weights((torch.randn(1, N, K, generator=g) * 0.02).to(torch.bfloat16).cuda(),
                             want_fq=True, sf_layout=B.SF_TILED)
    tf32 = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    y_ref = x.to(torch.float32) @ w["w_fq"][0].to(torch.float32).t()
    torch.backends.cuda.matmul.allow_tf32 = tf32
    errs = []
    for nsel in (0, K // 8, K // 4, K // 2, K):
        y = B.dense_w4a4_rac(x, w, nsel)["out"].to(torch.float32)
        errs.append((torch.linalg.norm(y - y_ref) / torch.linalg.norm(y_ref)).item())
    assert all(a > b for a, b in zip(errs, errs[1:])), errs
    assert errs[-1] < 0.25 * errs[0], errs
    assert 0.01 < errs[0] < 0.3, errs            # plain W4A4: a few per cent, as NVFP4 activations give


@pytest.mark.parametrize("T,K,N,seed", [(128, 512, 256, 0), (300, 2048, 384, 6), (1, 128, 128, 1), (2300, 1024, 640, 9)])
def test_one_sided_modes_of_the_dense_projection(B, T, K, N, seed):
    """W4A16 (NVFP4 weights decoded to bf16, activations untouched) and W16A4 (activations through Q_A and
    back, bf16 weights): the ablation modes of Table "qdq-alignment", bf16 tensor-core products, against
    the float64 oracle; the quantized side's bytes are the ones the W4A4 path uses."""
    x, w = synth.dense_inputs(seed, T=T, K=K, N=N)
    wo = MC.oracle_weights(w[None])
    wq = B.fake_quant_weights(w.unsqueeze(0).cuda(), want_fq=False, sf_layout=B.SF_TILED)
    # ---- W4A16
    res = B.dense_one_sided(x.cuda(), B.W4A16, w=wq)
    torch.cuda.synchronize()
    assert B.moe_async_status(res["workspace"]) == 0
    o = M.dense_w4a16(MC.f32(x), wo["codes"][0], wo["sf"][0], wo["gs"][0])
    got = MC.f32(res["out"]).astype(np.float64)
    r1 = float((np.abs(got - o["y64"]) / MC.gemm_tol(o["absdot"], o["y64"])).max())
    assert r1 <= 1.0, r1
    # ---- W16A4, amax-derived and supplied activation scale
    for a_gs in (None, np.float32(0.5) * Q.tensor_global_scale(MC.f32(x))):
        gs_t = None if a_gs is None else torch.tensor([float(a_gs)]).cuda()
        res = B.dense_one_sided(x.cuda(), B.W16A4, w_bf16=w.cuda(), a_gs=gs_t, export=True)
        torch.cuda.synchronize()
        assert B.moe_async_status(res["workspace"]) == 0
        o = M.dense_w16a4(MC.f32(x), MC.f32(w), a_gs)
        assert np.float32(res["a13_gs"].item()) == o["gs"]
        assert np.array_equal(res["xq"].cpu().numpy(), F.pack_nibbles(o["codes"]))
        assert np.array_equal(res["xsf"].cpu().numpy(), o["sf"])
        got = MC.f32(res["out"]).astype(np.float64)
        r2 = float((np.abs(got - o["y64"]) / MC.gemm_tol(o["absdot"], o["y64"])).max())
        assert r2 <= 1.0, r2
    # RAC is not part of these modes
    with pytest.raises(B.QuadsError) as e:
        a = B.MoEArgs()
        a.T, a.H, a.I, a.E, a.topk, a.N = T, K, 0, 1, 1, N
        a.operand_mode, a.rac_nsel_13 = B.W4A16, 16
        B.check(B.lib.quads_moe_w4a4_rac(B.C.byref(a), None))
    assert e.value.status == -2
