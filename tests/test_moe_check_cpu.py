"""The staged / sampled comparison helpers that the GPU tests use, exercised on
the CPU: fed with the oracle's own layer they must pass, and fed with a layer
in which one sampled value is wrong (beyond tolerance) they must fail."""
import os
import sys

import numpy as np
import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import moe_check as MC  # noqa: E402
from oracle import formats as F  # noqa: E402
from oracle import moe as M  # noqa: E402
from paper_2607_15810_b200 import synth  # noqa: E402


def _oracle_as_result():
    sh = synth.MOE_SHAPES["small"]
    x, _ = synth.activations(sh)
    lg = synth.router_logits(sh)
    w13, w2 = synth.expert_weights(sh, "w13"), synth.expert_weights(sh, "w2")
    w13o, w2o = MC.oracle_weights(w13), MC.oracle_weights(w2)
    n13, n2, a2 = sh.H // 2, sh.I // 2, np.float32(0.05)
    o = M.moe_forward(MC.f32(x), lg.numpy(), w13o, w2o, sh.topk, n13, n2, a2)
    t = torch.from_numpy
    res = dict(ids=t(o["ids"]), weights=t(o["weights"]), offsets=t(o["offsets"]), perm=t(o["perm"]),
               xq=t(F.pack_nibbles(o["site13"]["codes"])), xsf=t(o["site13"]["sf"]),
               a13_gs=torch.tensor([float(o["site13"]["gs"])]), sel13=t(o["site13"]["sel"]),
               rq=t(F.pack_nibbles(o["site13"]["r_codes"])), rsf=t(o["site13"]["r_sf"]),
               h=t(o["h"].copy()), hq=t(F.pack_nibbles(o["site2"]["codes"])), hsf=t(o["site2"]["sf"]),
               sel2=t(o["site2"]["sel"]), r2q=t(F.pack_nibbles(o["site2"]["r_codes"])), r2sf=t(o["site2"]["r_sf"]),
               out=t(o["out"].copy()))
    return sh, x, lg, w13, w2, w13o, w2o, n13, n2, a2, o, res


def test_sampled_and_full_checkers_accept_the_oracle_and_reject_a_wrong_value():
    sh, x, lg, w13, w2, w13o, w2o, n13, n2, a2, o, res = _oracle_as_result()
    kw = dict(n_tokens=16, n_features=32, n_columns=32, tail_experts=3)
    rep = MC.check_moe_sampled(res, x, lg, sh, lambda e: w13[e], lambda e: w2[e], n13, n2, a2, **kw)
    assert rep["sampled_experts"] == sh.E and rep["h_max_err_over_tol"] < 1 and rep["out_max_err_over_tol"] < 1
    full = MC.check_moe(res, x, lg, w13o, w2o, sh.topk, n13, n2, a2)
    assert full["h_bitwise_equal_fraction"] == 1.0
    # the plan: every expert with rows is covered by a sampled token, its first and last row are sampled,
    # and so is every tile of the last experts
    ids, offsets = o["ids"], o["offsets"]
    tokens, rows = MC.sample_plan(ids, offsets, sh.topk, sh.hot_experts, 16, 3, 99)
    assert {int(e) for t in tokens for e in ids[t]} == {e for e in range(sh.E) if offsets[e + 1] > offsets[e]}
    for e in range(sh.E):
        if offsets[e + 1] > offsets[e]:
            assert int(offsets[e]) in rows and int(offsets[e + 1]) - 1 in rows
    for e in range(sh.E - 3, sh.E):
        tiles = {(r - int(offsets[e])) // 128 for r in rows if offsets[e] <= r < offsets[e + 1]}
        assert tiles == set(range((int(offsets[e + 1] - offsets[e]) + 127) // 128))
    # a wrong `out` value in a sampled (token, column): the first column is always sampled
    bad = dict(res)
    bad["out"] = res["out"].clone()
    bad["out"][tokens[0], 0] += 0.25 * res["out"].abs().max()
    with pytest.raises(AssertionError):
        MC.check_moe_sampled(bad, x, lg, sh, lambda e: w13[e], lambda e: w2[e], n13, n2, a2, **kw)
    # a wrong h value in a sampled row (first row of expert 0, first feature) changes Q_A(h) too:
    # the bit-exact stage or the tolerance stage must object
    bad = dict(res)
    bad["h"] = res["h"].clone()
    bad["h"][int(offsets[0]), 0] += 1.0
    with pytest.raises(AssertionError):
        MC.check_moe_sampled(bad, x, lg, sh, lambda e: w13[e], lambda e: w2[e], n13, n2, a2, **kw)
