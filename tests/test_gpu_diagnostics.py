"""Device-side mismatch diagnostics against the oracle: per-channel squared residual scores (Eq.
channel-score) and the Frobenius norms of Eq. linear-mismatch, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import diagnostics as D
from oracle import moe as M
from oracle import nvfp4 as Q
from paper_2607_15810_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_15810_b200 import binding
    return binding


def _f32(t):
    return t.to(torch.float32).cpu().numpy()


@pytest.mark.parametrize("name,rows", [("tiny", None), ("small", None), ("decode", None), ("large", 1500)])
def test_channel_scores_match_the_oracle(B, name, rows):
    sh = synth.MOE_SHAPES[name]
    x, heavy = synth.activations(sh)
    if rows:
        x = x[:rows].contiguous()
    s = B.rac_channel_scores(x.cuda())
    want = D.channel_scores_of(_f32(x))
    got = s.cpu().numpy()
    # per-CTA float32 partial sums over at most 14 rows, float64 from there on
    assert np.allclose(got, want, rtol=2e-6, atol=0), float(np.abs(got / want - 1).max())
    # the ranking RAC takes from them is the oracle's, up to exact near-ties
    k = sh.H // 2
    a, b = set(np.argsort(-got, kind="stable")[:k].tolist()), set(np.argsort(-want, kind="stable")[:k].tolist())
    edge = np.sort(want)[::-1][k - 1]
    assert all(abs(want[j] - edge) <= 1e-5 * edge for j in a ^ b)
    # the heavy-tailed channels' blocks hold the largest residuals (the "vertical bands")
    top_blocks = {int(j) // 16 for j in np.argsort(-got)[:8]}
    assert top_blocks <= {int(c) // 16 for c in heavy}
    # a supplied scale
    g = np.float32(0.5) * Q.tensor_global_scale(_f32(x))
    s2 = B.rac_channel_scores(x.cuda(), gs=torch.tensor([float(g)]).cuda())
    assert np.allclose(s2.cpu().numpy(), D.channel_scores_of(_f32(x), g), rtol=2e-6, atol=0)


def test_mismatch_norms_and_the_terms_of_the_linear_mismatch(B):
    """Eq. linear-mismatch on the device: the norms kernel against numpy, then the decomposition of
    one projection's mismatch with the library's own W16A16 / W4A16 / W16A4 / W4A4(+RAC) outputs."""
    g = torch.Generator().manual_seed(8)
    a = torch.randn(1000, 333, generator=g).to(torch.bfloat16)
    b = (a.float() + 0.05 * torch.randn(1000, 333, generator=g)).to(torch.bfloat16)
    for aa, bb in ((a, b), (a[:7, :5].contiguous(), b[:7, :5].contiguous()), (a, a)):
        got = B.mismatch_norms(aa.cuda(), bb.cuda()).cpu().numpy()
        assert np.allclose(got, D.mismatch_norms(_f32(aa), _f32(bb)), rtol=1e-12, atol=0)
    again = B.mismatch_norms(a.cuda(), b.cuda()).cpu().numpy()
    assert np.array_equal(again, B.mismatch_norms(a.cuda(), b.cuda()).cpu().numpy())     # fixed order
    x, w = synth.dense_inputs(seed=2, T=512, K=1024, N=512)
    wq = B.fake_quant_weights(w.unsqueeze(0).cuda(), want_fq=False, sf_layout=B.SF_TILED)
    xc, wc = x.cuda(), w.cuda()
    y_train = B.dense_one_sided(xc, B.W16A16, w_bf16=wc)["out"]
    y = {"W4A16": B.dense_one_sided(xc, B.W4A16, w=wq)["out"], "W16A4": B.dense_one_sided(xc, B.W16A4, w_bf16=wc)["out"],
         "W4A4": B.dense_w4a4_rac(xc, wq, 0)["out"], "W4A4+RAC50": B.dense_w4a4_rac(xc, wq, 512)["out"],
         "W4A4+RAC100": B.dense_w4a4_rac(xc, wq, 1024)["out"]}
    rel = {k: float(np.sqrt(B.mismatch_norms(v, y_train).cpu().numpy()[0] / B.mismatch_norms(v, y_train).cpu().numpy()[2]))
           for k, v in y.items()}
    t = D.linear_mismatch_terms(_f32(x), _f32(w))
    nt = np.linalg.norm(t["y_train"])
    # the one-sided modes isolate the two first-order terms (outputs are rounded to bf16: 2^-9 relative)
    assert abs(rel["W16A4"] - np.linalg.norm(t["act"]) / nt) < 3e-3
    assert abs(rel["W4A16"] - np.linalg.norm(t["wgt"]) / nt) < 3e-3
    assert abs(rel["W4A4"] - np.linalg.norm(t["y_infer"] - t["y_train"]) / nt) < 3e-3
    # RAC removes activation error: the mismatch falls towards the weight-only level as channels are added
    assert rel["W4A4"] > rel["W4A4+RAC50"] > rel["W4A4+RAC100"] > 0.9 * rel["W4A16"]
    # against the asymmetric-QAT learner (forward = W4A16) the weight term is gone altogether
    learner = y["W4A16"]
    gap = {k: float(np.sqrt(B.mismatch_norms(y[k], learner).cpu().numpy()[0])) for k in ("W4A4", "W4A4+RAC50", "W4A4+RAC100")}
    assert gap["W4A4"] > gap["W4A4+RAC50"] > gap["W4A4+RAC100"]
    assert gap["W4A4+RAC100"] < 0.35 * gap["W4A4"]
    print("relative mismatch vs W16A16:", rel, "| vs W4A16 learner:", gap)
