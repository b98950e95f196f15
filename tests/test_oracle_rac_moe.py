"""Pins for the oracle's Residual Activation Compensation, routing and MoE
forward: the paper's shrink inequality and sign convention, monotone error over
the paper's channel ratios, the two degenerate ratios, brute force on tiny
inputs, a float64 triple loop written independently of numpy's matmul, the
exact-integer special case, linearity and the dense special case."""
import os

import numpy as np
import torch

from oracle import formats as F
from oracle import moe as M
from oracle import nvfp4 as Q
from oracle import rac as R
from paper_2607_15810_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _ratios():
    with open(os.path.join(GOLD, "rac_ratios.txt")) as fh:
        line = [ln for ln in fh if not ln.startswith("#") and ln.strip()][0]
    return [float(v) for v in line.split()]


def _dense():
    x, w = synth.dense_inputs(seed=0)
    return x.to(torch.float32).numpy(), w.to(torch.float32).numpy()


def test_shrink_inequality_and_sign_for_both_residual_scale_readings():
    x, _ = _dense()
    for r_gs in (None, "own"):
        plain = R.rac(x, 0, None, r_gs)
        e0 = np.linalg.norm(R.reconstruct_real(plain) - x)
        assert e0 == np.linalg.norm(Q.dequantize_real(plain["codes"], plain["sf"], plain["gs"]) - x)
        prev = e0
        for pct in _ratios():
            n_sel = int(round(x.shape[1] * pct / 100))
            site = R.rac(x, n_sel, None, r_gs)
            e = np.linalg.norm(R.reconstruct_real(site) - x)
            assert e < prev, (r_gs, pct, e, prev)           # strictly shrinking, Eq. residual-shrink
            prev = e
            # the opposite sign would grow the error
            wrong = (Q.dequantize_real(site["codes"], site["sf"], site["gs"])
                     + Q.dequantize_real(site["r_codes"], site["r_sf"], site["r_gs"]))
            assert np.linalg.norm(wrong - x) > e0


def test_degenerate_ratios():
    x, _ = _dense()
    K = x.shape[1]
    s0 = R.rac(x, 0)
    assert s0["sel"].size == 0 and not s0["r_codes"].any()
    sK = R.rac(x, K)
    assert np.array_equal(sK["sel"], np.arange(K))
    full_c, full_s, _ = Q.quantize(sK["residual"], sK["r_gs"])
    assert np.array_equal(sK["r_codes"], full_c) and np.array_equal(sK["r_sf"], full_s)
    # masking never touches the scales
    s16 = R.rac(x, 16)
    assert np.array_equal(s16["r_sf"], full_s)
    keep = np.zeros(K, bool)
    keep[s16["sel"]] = True
    assert np.array_equal(s16["r_codes"][:, keep], full_c[:, keep])
    assert not s16["r_codes"][:, ~keep].any()


def test_selection_is_brute_force_topk_with_low_index_ties():
    scores = np.array([3.0, 7.0, 7.0, 1.0, 9.0, 7.0, 0.0, 3.0])
    for n in range(9):
        # brute force: repeatedly take the largest remaining score, lowest index first
        rest, chosen = list(range(8)), []
        for _ in range(n):
            best = max(rest, key=lambda j: (scores[j], -j))
            chosen.append(best)
            rest.remove(best)
        assert list(R.select_channels(scores, n)) == sorted(chosen)
    x, _ = _dense()
    site = R.rac(x[:9, :32], 5)
    r = site["residual"].astype(np.float64)
    brute = sorted(sorted(range(32), key=lambda j: (-float((r[:, j] ** 2).sum()), j))[:5])
    assert list(site["sel"]) == brute
    assert np.allclose(site["scores"], [(r[:, j] ** 2).sum() for j in range(32)], rtol=1e-12)


def test_dense_config_selects_inside_the_outlier_blocks():
    """The x20 outlier channels inflate their 16-block's scale, so every channel
    of those four blocks carries a large residual: the paper's "vertical bands"
    (Section "Activation Error Compensation for Rollout-side")."""
    x, _ = _dense()
    site = R.rac(x, 16)
    blocks = {c // 16 for c in synth.DENSE_OUTLIER_CHANNELS}
    assert {int(j) // 16 for j in site["sel"]} <= blocks
    # the residual really is Q_A(X) - X (Eq. residual-def), not X - Q_A(X)
    xh = Q.dequantize_f32(site["codes"], site["sf"], site["gs"])
    assert np.array_equal(site["residual"], xh - x)


def test_routing_against_brute_force():
    rng = np.random.default_rng(5)
    logits = rng.normal(size=(13, 6)).astype(np.float32)
    logits[2, 1] = logits[2, 4] = logits[2].max() + 1       # a tie at the top
    ids, w = M.route(logits, 3, renormalize=True)
    for t in range(13):
        order = sorted(range(6), key=lambda e: (-float(logits[t, e]), e))[:3]
        assert list(ids[t]) == order
        p = np.exp(logits[t].astype(np.float64))
        p /= p.sum()
        want = p[order] / p[order].sum()
        assert np.allclose(w[t], want, rtol=1e-6)
    ids2, w2 = M.route(logits, 3, renormalize=False)
    assert np.array_equal(ids, ids2)
    assert np.all(w2.sum(axis=1) < 1)
    counts, offsets, perm = M.dispatch(ids, 6)
    assert counts.sum() == 13 * 3 and offsets[0] == 0 and offsets[-1] == 39
    assert np.all(np.diff(offsets) == counts)
    assert sorted(perm) == list(range(39))
    keys = [(int(ids.reshape(-1)[p]), int(p)) for p in perm]
    assert keys == sorted(keys)                              # (expert, token, slot) order


def _tiny_weights(n, N, K, seed, std=0.05):
    w = (torch.randn(n, N, K, generator=torch.Generator().manual_seed(seed)) * std)
    w = w.to(torch.bfloat16).to(torch.float32).numpy()
    _, q, sf, gs = Q.fake_quant_weights(w)
    return dict(codes=F.unpack_nibbles(q), sf=sf, gs=gs)


def _triple_loop(a, b):
    """a [M,K], b [N,K] -> a b^T with python floats (IEEE double), no numpy matmul."""
    out = [[0.0] * len(b) for _ in a]
    for i, ar in enumerate(a):
        for j, br in enumerate(b):
            s = 0.0
            for u, v in zip(ar, br):
                s += u * v
            out[i][j] = s
    return np.array(out)


def _scalar_dequant(codes, sf8, gs):
    """Element-by-element dequantization written from the format definition."""
    e2 = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    out = np.zeros(codes.shape)
    for i in range(codes.shape[0]):
        for k in range(codes.shape[1]):
            c = int(codes[i, k])
            s = int(sf8[i, k // 16])
            ef, m = s >> 3, s & 7
            sc = (m / 8.0) * 2.0 ** -6 if ef == 0 else (1 + m / 8.0) * 2.0 ** (ef - 7)
            out[i, k] = (-1.0 if c & 8 else 1.0) * e2[c & 7] * sc * float(gs)
    return out


def test_dense_gemm_against_triple_loop_and_linearity():
    x, w = synth.dense_inputs(seed=3, T=5, K=32, N=4, outlier_channels=(3,))
    x = x.to(torch.float32).numpy()
    wq = _tiny_weights(1, 4, 32, 9)
    res = M.dense_w4a4_rac(x, wq["codes"][0], wq["sf"][0], wq["gs"][0], n_sel=8)
    site = res["site"]
    xa = _scalar_dequant(site["codes"], site["sf"], site["gs"])
    ra = _scalar_dequant(site["r_codes"], site["r_sf"], site["r_gs"])
    wa = _scalar_dequant(wq["codes"][0], wq["sf"][0], wq["gs"][0])
    want = _triple_loop((xa - ra).tolist(), wa.tolist())
    assert np.allclose(res["y64"], want, rtol=1e-12, atol=1e-15)
    # linearity: W X~ = W Q(X) - W (M (.) Q(dX))
    lin = _triple_loop(xa.tolist(), wa.tolist()) - _triple_loop(ra.tolist(), wa.tolist())
    assert np.allclose(res["y64"], lin, rtol=1e-10, atol=1e-14)
    # n_sel = 0 is the plain W4A4 product
    plain = M.dense_w4a4_rac(x, wq["codes"][0], wq["sf"][0], wq["gs"][0], n_sel=0)
    assert np.allclose(plain["y64"], _triple_loop(xa.tolist(), wa.tolist()), rtol=1e-12, atol=1e-15)
    absd = _triple_loop((np.abs(xa) + np.abs(ra)).tolist(), np.abs(wa).tolist())
    assert np.allclose(res["absdot"], absd, rtol=1e-12)


def test_exact_integer_special_case():
    """Scales of one and integer-valued codes: the contraction is a small-integer
    matrix product (textbook check, exact)."""
    rng = np.random.default_rng(11)
    ints = np.array([0, 1, 2, 3, 4, 6, -1, -2, -3, -4, -6])
    a = rng.choice(ints, (6, 32)).astype(np.float32)
    a[:, 0] = 6
    a[:, 16] = -6
    b = rng.choice(ints, (3, 32)).astype(np.float32)
    b[:, 0] = 6
    b[:, 16] = 6
    ca, sa, ga = Q.quantize(a, np.float32(1.0))
    cb, sb, gb = Q.quantize(b, np.float32(1.0))
    assert np.all(sa == 0x38) and np.all(sb == 0x38)        # E4M3 code of 1.0
    res = M.dense_w4a4_rac(a, cb, sb, gb, n_sel=0, a_gs=np.float32(1.0))
    assert np.array_equal(res["y64"], (a.astype(np.int64) @ b.astype(np.int64).T).astype(np.float64))


def test_moe_single_expert_reduces_to_dense_and_matches_loops():
    shape = synth.MoEShape("t", 21, 6, 32, 1, 1, 16, 0.05, 1, 3.0, 10.0)
    x, _ = synth.activations(shape)
    x = x.to(torch.float32).numpy()
    logits = np.zeros((6, 1), np.float32)
    w13 = _tiny_weights(1, 32, 32, 31)
    w2 = _tiny_weights(1, 32, 16, 32)
    a2_gs = np.float32(0.002)
    out = M.moe_forward(x, logits, w13, w2, 1, 8, 4, a2_gs)
    assert np.array_equal(out["perm"], np.arange(6)) and np.all(out["weights"] == 1.0)
    d = M.dense_w4a4_rac(x, w13["codes"][0], w13["sf"][0], w13["gs"][0], n_sel=8)
    assert np.array_equal(out["g64"], d["y64"])
    g = out["g64"]
    h = np.array([[(gi / (1 + np.exp(-gi))) * ui for gi, ui in zip(row[:16], row[16:])] for row in g])
    assert np.allclose(out["h64"], h, rtol=1e-13)
    d2 = M.dense_w4a4_rac(out["h"], w2["codes"][0], w2["sf"][0], w2["gs"][0], n_sel=4, a_gs=a2_gs)
    assert np.array_equal(out["out64"], d2["y64"])


def test_moe_two_experts_against_explicit_loops():
    shape = synth.MoEShape("t", 22, 9, 32, 3, 2, 16, 0.05, 1, 3.0, 10.0)
    x, _ = synth.activations(shape)
    x = x.to(torch.float32).numpy()
    logits = synth.router_logits(shape).numpy()
    w13 = _tiny_weights(3, 32, 32, 41)
    w2 = _tiny_weights(3, 32, 16, 42)
    a2_gs = np.float32(0.003)
    out = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2_gs, renormalize=True)
    # re-derive the output token by token from the exported intermediates
    xt = R.reconstruct_real(out["site13"])
    ht = R.reconstruct_real(out["site2"])
    inv = np.empty(18, int)
    inv[out["perm"]] = np.arange(18)
    want = np.zeros((9, 32))
    for t in range(9):
        for s in range(2):
            e = int(out["ids"][t, s])
            row = inv[t * 2 + s]
            assert out["offsets"][e] <= row < out["offsets"][e + 1]
            w13e = _scalar_dequant(w13["codes"][e], w13["sf"][e], w13["gs"][e])
            g = _triple_loop([xt[t].tolist()], w13e.tolist())[0]
            assert np.allclose(out["g64"][row], g, rtol=1e-12, atol=1e-15)
            w2e = _scalar_dequant(w2["codes"][e], w2["sf"][e], w2["gs"][e])
            y = _triple_loop([ht[row].tolist()], w2e.tolist())[0]
            want[t] += float(out["weights"][t, s]) * y
    assert np.allclose(out["out64"], want, rtol=1e-11, atol=1e-14)
    assert np.array_equal(out["out"], F.bf16_round(out["out64"]))
    # site-2 statistics run over all dispatched rows at once
    assert out["site2"]["codes"].shape == (18, 16) and out["site2"]["sel"].size == 8


def _two_expert_case():
    shape = synth.MoEShape("t", 23, 9, 32, 3, 2, 16, 0.05, 1, 3.0, 10.0)
    x, _ = synth.activations(shape)
    x = x.to(torch.float32).numpy()
    logits = synth.router_logits(shape).numpy()
    return x, logits, _tiny_weights(3, 32, 32, 51), _tiny_weights(3, 32, 16, 52), np.float32(0.003)


def _second_half_by_loops(out, ht, w2):
    """out[t] = sum over the token's slots of weight * W2_e h~[row], explicit loops."""
    T, topk = out["ids"].shape
    inv = np.empty(T * topk, int)
    inv[out["perm"]] = np.arange(T * topk)
    want = np.zeros((T, w2["codes"].shape[1]))
    for t in range(T):
        for s in range(topk):
            e = int(out["ids"][t, s])
            w2e = _scalar_dequant(w2["codes"][e], w2["sf"][e], w2["gs"][e])
            want[t] += float(out["weights"][t, s]) * _triple_loop([ht[inv[t * topk + s]].tolist()], w2e.tolist())[0]
    return want


def test_h_override_replays_and_replaces_the_second_half():
    """The staged comparison of an implementation runs the layer's second half
    on that implementation's own h.  Feeding the oracle its own h must change
    nothing; feeding it a perturbed h must give exactly what site-2 RAC and
    the down projection give for that h."""
    x, logits, w13, w2, a2 = _two_expert_case()
    base = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2)
    same = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, h_override=base["h"])
    for k in ("codes", "sf", "r_codes", "r_sf", "sel", "scores", "residual"):
        assert np.array_equal(same["site2"][k], base["site2"][k]), k
    assert same["site2"]["gs"] == base["site2"]["gs"] and same["site2"]["r_gs"] == base["site2"]["r_gs"]
    assert np.array_equal(same["out64"], base["out64"]) and np.array_equal(same["out_absdot"], base["out_absdot"])
    assert np.array_equal(same["out"], base["out"])
    # one bf16 ulp up on a few elements (and one sign flip): a different, equally valid h
    hp = base["h"].copy()
    bits = F.bf16_bits(hp).astype(np.uint32)
    for (i, j) in ((0, 0), (3, 7), (11, 15), (17, 2)):
        bits[i, j] += 1
    bits[5, 5] ^= 0x8000
    hp = (bits << 16).view(np.float32).reshape(hp.shape)
    assert np.all(F.bf16_round(hp) == hp) and (hp != base["h"]).sum() >= 4
    pert = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, h_override=hp)
    assert np.array_equal(pert["h"], base["h"])               # the oracle's own h is still reported
    want_site = R.rac(hp, 8, a2)
    for k in ("codes", "sf", "r_codes", "r_sf", "sel"):
        assert np.array_equal(pert["site2"][k], want_site[k]), k
    assert pert["site2"]["gs"] == a2 and pert["site2"]["r_gs"] == a2
    assert not np.array_equal(pert["site2"]["codes"], base["site2"]["codes"])   # the override is not ignored
    want = _second_half_by_loops(pert, R.reconstruct_real(want_site), w2)
    assert np.allclose(pert["out64"], want, rtol=1e-11, atol=1e-14)
    assert not np.allclose(pert["out64"], base["out64"], rtol=1e-6, atol=0)
    # the tolerance denominator follows the overriding operands too
    ha = (np.abs(_scalar_dequant(want_site["codes"], want_site["sf"], a2))
          + np.abs(_scalar_dequant(want_site["r_codes"], want_site["r_sf"], a2)))
    absd = np.zeros_like(want)
    inv = np.empty(18, int)
    inv[pert["perm"]] = np.arange(18)
    for t in range(9):
        for s in range(2):
            e = int(pert["ids"][t, s])
            w2e = np.abs(_scalar_dequant(w2["codes"][e], w2["sf"][e], w2["gs"][e]))
            absd[t] += float(pert["weights"][t, s]) * _triple_loop([ha[inv[t * 2 + s]].tolist()], w2e.tolist())[0]
    assert np.allclose(pert["out_absdot"], absd, rtol=1e-11)


def test_forced_selection_is_a_brute_force_remask():
    """_force_selection with the site's own set is the identity; with another
    set it equals clearing, by hand, the unselected channels of the quantized
    full residual (block scales untouched, everything else unchanged)."""
    x, _ = _dense()
    x = x[:24, :64]
    site = R.rac(x, 16)
    ident = M._force_selection(x, site, site["sel"])
    assert set(ident) == set(site)
    for k, v in site.items():
        assert np.array_equal(ident[k], v), k
    other = np.array([63, 0, 17, 5, 40], dtype=np.int32)        # unsorted on purpose
    forced = M._force_selection(x, site, other)
    full_c, full_s, full_g = Q.quantize(site["residual"], site["r_gs"])
    assert full_g == site["r_gs"] == site["gs"]                 # the residual shares its activation's scale
    want = np.zeros_like(full_c)
    for j in other:
        want[:, j] = full_c[:, j]
    assert np.array_equal(forced["r_codes"], want)
    assert np.array_equal(forced["sel"], np.sort(other))
    assert np.array_equal(forced["r_sf"], full_s) and np.array_equal(forced["r_sf"], site["r_sf"])
    for k in ("codes", "sf", "gs", "residual", "scores", "r_gs"):
        assert np.array_equal(forced[k], site[k]), k
    # a forced set that differs from the top-16 changes the reconstruction
    assert not np.array_equal(R.reconstruct_real(forced), R.reconstruct_real(site))


def test_forced_selections_flow_through_the_layer():
    """moe_forward(forced_sel13 / forced_sel2): with the sets the oracle picks
    itself nothing changes; with other sets the layer equals the explicit
    loops run on the re-masked operands."""
    x, logits, w13, w2, a2 = _two_expert_case()
    base = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2)
    same = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, forced_sel13=base["site13"]["sel"],
                         forced_sel2=base["site2"]["sel"])
    assert np.array_equal(same["g64"], base["g64"]) and np.array_equal(same["out64"], base["out64"])
    # swap one selected channel for an unselected one at each site
    def swapped(sel, C):
        rest = [j for j in range(C) if j not in set(int(v) for v in sel)]
        return np.array(sorted(list(sel[1:]) + [rest[0]]), dtype=np.int32)
    s13, s2 = swapped(base["site13"]["sel"], 32), swapped(base["site2"]["sel"], 16)
    f13 = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, forced_sel13=s13)
    want13 = M._force_selection(x, base["site13"], s13)
    assert np.array_equal(f13["site13"]["r_codes"], want13["r_codes"]) and np.array_equal(f13["site13"]["sel"], s13)
    xt = R.reconstruct_real(want13)
    for row in range(18):
        t = int(base["perm"][row]) // 2
        e = int(base["ids"].reshape(-1)[base["perm"][row]])
        w13e = _scalar_dequant(w13["codes"][e], w13["sf"][e], w13["gs"][e])
        assert np.allclose(f13["g64"][row], _triple_loop([xt[t].tolist()], w13e.tolist())[0], rtol=1e-12, atol=1e-15)
    assert not np.array_equal(f13["g64"], base["g64"])
    # site 2, on an overriding h as the staged comparison uses it
    f2 = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, h_override=base["h"], forced_sel2=s2)
    want2 = M._force_selection(base["h"], base["site2"], s2)
    assert np.array_equal(f2["site2"]["r_codes"], want2["r_codes"])
    assert np.allclose(f2["out64"], _second_half_by_loops(f2, R.reconstruct_real(want2), w2), rtol=1e-11, atol=1e-14)
    assert not np.array_equal(f2["out64"], base["out64"])


def test_residual_scale_readings_agree_on_the_benchmark_distributions():
    """The residual is quantized with its activation's per-tensor scale (the
    reading taken) or with its own amax-derived one (the other reading of Eq.
    residual-recon).  On activations drawn like the large MoE workload the two
    correct the same amount, and the shared scale leaves the residual's block
    scales in E4M3's normal range; only with an outlier beyond a few thousand
    times the typical block maximum do they start to fall into the subnormals."""
    sh = synth.MOE_SHAPES["large"]
    x, _ = synth.activations(sh)
    x = x[:96].to(torch.float32).numpy()
    K = x.shape[1]
    base = R.rac(x, 0)
    e0 = np.linalg.norm(Q.dequantize_real(base["codes"], base["sf"], base["gs"]) - x)
    for pct in (12.5, 50.0, 100.0):
        n = int(K * pct / 100)
        shared, own = R.rac(x, n), R.rac(x, n, None, "own")
        es = np.linalg.norm(R.reconstruct_real(shared) - x) / e0
        eo = np.linalg.norm(R.reconstruct_real(own) - x) / e0
        assert abs(es - eo) < 5e-3 * eo, (pct, es, eo)
        assert own["r_gs"] < shared["r_gs"] / 6                  # the residual is at least a grid step below
    full = R.rac(x, K)
    sub = ((full["r_sf"] > 0) & (full["r_sf"] < 8)).mean()      # E4M3 codes 1..7 are subnormal
    assert sub < 1e-3 and (full["r_sf"] == 0).mean() < 1e-3
    # one extreme outlier (3e4 against block maxima near 2.5) pushes the shared-scale residual scales into
    # the subnormal codes, where the own-scale reading keeps correcting
    y = x.copy()
    y[0, 0] = 30000.0
    fs, fo = R.rac(y, K), R.rac(y, K, None, "own")
    assert ((fs["r_sf"] > 0) & (fs["r_sf"] < 8)).mean() > 0.5
    assert ((fo["r_sf"] > 0) & (fo["r_sf"] < 8)).mean() < 0.05
    by = R.rac(y, 0)
    e0y = np.linalg.norm(Q.dequantize_real(by["codes"], by["sf"], by["gs"]) - y)
    assert np.linalg.norm(R.reconstruct_real(fo) - y) < np.linalg.norm(R.reconstruct_real(fs) - y) < e0y


def test_one_sided_modes_against_loops_and_their_special_cases():
    """W4A16 / W16A4 (Table "qdq-alignment"): explicit loops on the decoded bf16 operands; an operand
    that NVFP4 represents exactly makes its one-sided mode the plain bf16 product; and with both
    sides exactly representable (power-of-two tensor scales, <= 6 significant bits) all of W4A4,
    W4A16, W16A4 and the plain product coincide."""
    x, w = synth.dense_inputs(seed=4, T=5, K=32, N=4, outlier_channels=(3,))
    x, w = x.to(torch.float32).numpy(), w.to(torch.float32).numpy()
    wq = _tiny_weights(1, 4, 32, 9)
    a = M.dense_w4a16(x, wq["codes"][0], wq["sf"][0], wq["gs"][0])
    wd = Q.dequantize_bf16(wq["codes"][0], wq["sf"][0], wq["gs"][0])
    assert np.array_equal(F.bf16_round(wd), wd)
    assert np.allclose(a["y64"], _triple_loop(x.tolist(), wd.astype(np.float64).tolist()), rtol=1e-12, atol=1e-15)
    assert np.allclose(a["absdot"], _triple_loop(np.abs(x).tolist(), np.abs(wd).astype(np.float64).tolist()), rtol=1e-12)
    b = M.dense_w16a4(x, w)
    xq = Q.quantize(x)
    assert np.array_equal(b["codes"], xq[0]) and np.array_equal(b["sf"], xq[1]) and b["gs"] == xq[2]
    xd = Q.dequantize_bf16(*xq)
    assert np.allclose(b["y64"], _triple_loop(xd.astype(np.float64).tolist(), w.astype(np.float64).tolist()), rtol=1e-12, atol=1e-15)
    assert not np.allclose(b["y64"], x.astype(np.float64) @ w.astype(np.float64).T, rtol=1e-3)   # the activation error is there
    # exactly representable operands: values (code) * (E4M3 scale) * 2^-p
    mags = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6, 6])
    rng = np.random.default_rng(2)
    xe = np.stack([rng.permutation(mags) * 2.0 ** rng.integers(-3, 3) for _ in range(6 * 2)]).reshape(6, 32) * 2.0 ** -4
    we = np.stack([rng.permutation(mags) * 2.0 ** rng.integers(-3, 3) for _ in range(3 * 2)]).reshape(3, 32) * 2.0 ** -6
    xe[0, :16] = mags * 448 * 2.0 ** -4                         # a block at the top of the range: tensor scale 2^-4
    we[0, :16] = mags * 448 * 2.0 ** -6
    xe, we = xe.astype(np.float32), we.astype(np.float32)
    cw, sw, gw = Q.quantize(we)
    assert gw == np.float32(2.0 ** -6) and np.array_equal(Q.dequantize_f32(cw, sw, gw), we)
    plain = xe.astype(np.float64) @ we.astype(np.float64).T
    assert np.array_equal(M.dense_w4a16(xe, cw, sw, gw)["y64"], plain)
    assert np.array_equal(M.dense_w16a4(xe, we)["y64"], plain)
    assert np.array_equal(M.dense_w4a4_rac(xe, cw, sw, gw, 0)["y64"], plain)


def test_expert_sharded_oracle_adds_up_to_the_layer():
    """Expert-sharded execution: routing and site 13 are the layer's; a shard's rows are its experts'
    segment of the dispatch order; without site-2 compensation the shards' partial sums add up to the
    layer output, and with it every shard runs RAC on its own rows."""
    x, logits, w13, w2, a2 = _two_expert_case()                 # three experts, two slots
    full0 = M.moe_forward(x, logits, w13, w2, 2, 16, 0, a2)
    parts = [M.moe_forward(x, logits, w13, w2, 2, 16, 0, a2, expert_range=r) for r in ((0, 1), (1, 3))]
    assert np.allclose(parts[0]["out64"] + parts[1]["out64"], full0["out64"], rtol=1e-12, atol=1e-15)
    off = full0["offsets"]
    for p, (lo, hi) in zip(parts, ((0, 1), (1, 3))):
        assert np.array_equal(p["site13"]["r_codes"], full0["site13"]["r_codes"])
        assert np.array_equal(p["h"], full0["h"][off[lo]:off[hi]])
        assert np.array_equal(p["g64"], full0["g64"][off[lo]:off[hi]])
    # with site-2 RAC: the shard's site 2 is RAC on its own rows, and its partial output follows from it
    sh = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, expert_range=(1, 3))
    want = R.rac(full0["h"][off[1]:off[3]], 8, a2)
    for k in ("codes", "sf", "r_codes", "r_sf", "sel"):
        assert np.array_equal(sh["site2"][k], want[k]), k
    ht = R.reconstruct_real(want)
    inv = np.empty(18, int)
    inv[full0["perm"]] = np.arange(18)
    ref = np.zeros((9, 32))
    for t in range(9):
        for s in range(2):
            e = int(full0["ids"][t, s])
            if e in (1, 2):
                w2e = _scalar_dequant(w2["codes"][e], w2["sf"][e], w2["gs"][e])
                ref[t] += float(full0["weights"][t, s]) * _triple_loop([ht[inv[t * 2 + s] - off[1]].tolist()], w2e.tolist())[0]
    assert np.allclose(sh["out64"], ref, rtol=1e-11, atol=1e-14)
    # a whole-range shard is the layer itself
    whole = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2, expert_range=(0, 3))
    full = M.moe_forward(x, logits, w13, w2, 2, 16, 8, a2)
    assert np.array_equal(whole["out64"], full["out64"]) and np.array_equal(whole["site2"]["r_codes"], full["site2"]["r_codes"])
