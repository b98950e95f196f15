"""Staged comparison of the CUDA MoE layer against the CPU oracle.

Stage 1 (bit-exact): routing ids, expert offsets, dispatch permutation, Q_A(x)
codes / scales, selected channels, masked residual codes / scales.
Stage 2 (tolerance): h = silu(gate) * up against the oracle's float64 value,
|err| <= 2e-3 * sum|a_i b_i| propagated through SwiGLU to first order
+ 1 bf16 ulp.
Stage 3 (validity, bit-exact): the requantized h and its masked residual must be
what the oracle's quantizer gives for the SAME bf16 h the CUDA path produced (h
feeds a quantizer: a one-ulp difference in h legitimately flips codes, so the
codes are checked as a function of the implementation's own h).
Stage 4 (tolerance): out against the oracle's float64 contraction of those
operands, |err| <= 2e-3 * sum|a_i b_i| + 1 bf16 ulp.
Stage 5 (sanity): relative Frobenius error against the oracle run end to end on
its own.
"""
import numpy as np
import torch

from oracle import formats as F
from oracle import moe as M
from oracle import nvfp4 as Q
from oracle import rac as R

GEMM_RTOL = 2e-3          # x sum|a_i b_i|
BF16_ULP = 2.0 ** -7      # relative size of one bf16 ulp (upper bound)


def f32(t):
    return t.detach().to(torch.float32).cpu().numpy()


def oracle_weights(w_bf16):
    """bf16 torch [E, N, K] -> oracle dict(codes, sf, gs) and packed bytes."""
    _, q, sf, gs = Q.fake_quant_weights(f32(w_bf16))
    return dict(codes=F.unpack_nibbles(q), sf=sf, gs=gs, q=q)


def gemm_tol(absdot, ref):
    return GEMM_RTOL * absdot + BF16_ULP * np.abs(ref) + 1e-30


def sel_matches(gpu_sel, site, n_sel):
    """Equal sets, or differing only in channels whose score ties the boundary
    within 1e-6 relative."""
    want = set(int(v) for v in site["sel"])
    got = set(int(v) for v in gpu_sel[:n_sel])
    if want == got:
        return True, 0
    sc = site["scores"]
    order = np.sort(sc)[::-1]
    edge = order[n_sel - 1]
    diff = want ^ got
    ok = all(abs(sc[j] - edge) <= 1e-6 * edge for j in diff)
    return ok, len(diff)


def check_site1(res, orc, nsel13, report):
    site = orc["site13"]
    assert np.array_equal(res["xq"].cpu().numpy(), F.pack_nibbles(site["codes"])), "Q_A(x) codes differ"
    assert np.array_equal(res["xsf"].cpu().numpy(), site["sf"]), "Q_A(x) scales differ"
    assert np.float32(res["a13_gs"].item()) == site["gs"], "per-tensor scale differs"
    if nsel13 > 0:
        assert np.array_equal(res["sel13"].cpu().numpy()[:nsel13], site["sel"]), "site-13 selection differs"
        assert np.array_equal(res["rq"].cpu().numpy(), F.pack_nibbles(site["r_codes"])), "residual codes differ"
        assert np.array_equal(res["rsf"].cpu().numpy(), site["r_sf"]), "residual scales differ"
    report["site13_bit_exact"] = True


def check_moe(res, x, logits, w13o, w2o, topk, nsel13, nsel2, a2_gs, renormalize=True, row_sample=None, a13_gs=None):
    """res: dict from binding.moe_w4a4_rac(export=True); x, logits torch CPU
    tensors; w13o / w2o oracle weight dicts.  Returns a report dict; raises on
    any violation."""
    report = {}
    xf = f32(x)
    lg = logits.cpu().numpy()
    orc = M.moe_forward(xf, lg, w13o, w2o, topk, nsel13, nsel2, a2_gs, a13_gs=a13_gs, renormalize=renormalize)
    T, H = xf.shape
    I = w2o["codes"].shape[2]
    # ---- stage 1
    assert np.array_equal(res["ids"].cpu().numpy(), orc["ids"]), "top-k ids differ"
    assert np.allclose(res["weights"].cpu().numpy(), orc["weights"], rtol=2e-5, atol=1e-7), "routing weights differ"
    assert np.array_equal(res["offsets"].cpu().numpy(), orc["offsets"]), "expert offsets differ"
    assert np.array_equal(res["perm"].cpu().numpy(), orc["perm"]), "dispatch permutation differs"
    check_site1(res, orc, nsel13, report)
    # ---- stage 2: h
    h_gpu = f32(res["h"])
    g, gad = orc["g64"], orc["g_absdot"]
    gate, up = g[:, :I], g[:, I:]
    sig = 1.0 / (1.0 + np.exp(-gate))
    dsilu = sig * (1.0 + gate * (1.0 - sig))
    dg, du = GEMM_RTOL * gad[:, :I], GEMM_RTOL * gad[:, I:]
    tol_h = (np.abs(dsilu * up) * dg + np.abs(gate * sig) * du + dg * du * 2
             + (BF16_ULP + 1e-5) * np.abs(orc["h64"]) + 1e-30)
    err_h = np.abs(h_gpu - orc["h64"])
    report["h_max_err_over_tol"] = float((err_h / tol_h).max())
    assert report["h_max_err_over_tol"] <= 1.0, "h outside tolerance: %g" % report["h_max_err_over_tol"]
    report["h_bitwise_equal_fraction"] = float((F.bf16_bits(h_gpu) == F.bf16_bits(orc["h"])).mean())
    # ---- stage 3: requantize of the implementation's own h
    orc2 = M.moe_forward(xf, lg, w13o, w2o, topk, nsel13, nsel2, a2_gs, a13_gs=a13_gs, renormalize=renormalize,
                         h_override=h_gpu)
    site2 = orc2["site2"]
    assert np.array_equal(res["hq"].cpu().numpy(), F.pack_nibbles(site2["codes"])), "Q_A(h) codes differ"
    assert np.array_equal(res["hsf"].cpu().numpy(), site2["sf"]), "Q_A(h) scales differ"
    if nsel2 > 0:
        ok, ndiff = sel_matches(res["sel2"].cpu().numpy(), site2, nsel2)
        assert ok, "site-2 selection differs beyond ties (%d channels)" % ndiff
        report["sel2_tie_swaps"] = ndiff
        if ndiff:
            orc2 = M.moe_forward(xf, lg, w13o, w2o, topk, nsel13, nsel2, a2_gs, a13_gs=a13_gs, renormalize=renormalize,
                                 h_override=h_gpu, forced_sel2=res["sel2"].cpu().numpy()[:nsel2])
            site2 = orc2["site2"]
        assert np.array_equal(res["r2q"].cpu().numpy(), F.pack_nibbles(site2["r_codes"])), "residual-of-h codes differ"
        assert np.array_equal(res["r2sf"].cpu().numpy(), site2["r_sf"]), "residual-of-h scales differ"
    report["site2_bit_exact"] = True
    # ---- stage 4: out
    out_gpu = f32(res["out"]).astype(np.float64)
    tol_o = gemm_tol(orc2["out_absdot"], orc2["out64"])
    # the routing weights differ from the oracle's by float32 rounding of exp(): allow for it
    tol_o = tol_o + 4e-5 * orc2["out_absdot"]
    err_o = np.abs(out_gpu - orc2["out64"])
    report["out_max_err_over_tol"] = float((err_o / tol_o).max())
    assert report["out_max_err_over_tol"] <= 1.0, "out outside tolerance: %g" % report["out_max_err_over_tol"]
    # ---- stage 5: end to end against the oracle alone
    num = np.linalg.norm(out_gpu - orc["out64"])
    den = np.linalg.norm(orc["out64"]) + 1e-30
    report["out_rel_frobenius_vs_pure_oracle"] = float(num / den)
    assert num / den <= 1e-2
    return report


def sample_plan(ids, offsets, topk, hot_experts, n_tokens, tail_experts, seed):
    """Which outputs of a full-size layer the oracle recomputes one by one.
    Tokens: a seeded random order, taken greedily until every expert that has
    rows is hit by a sampled token, then topped up to n_tokens; all rows of a
    sampled token are checked (h) and so is its row of `out`.  Extra dispatched
    rows (h only): the first and the last row of every expert, three rows of
    the first tile and the first / last row of the last tile of every hot
    expert, and one row in every 128-row tile of the last `tail_experts`
    experts (the tiles the persistent kernels take in their last wave)."""
    T = ids.shape[0]
    E = offsets.size - 1
    rng = np.random.default_rng(seed)
    order = rng.permutation(T)
    need = {e for e in range(E) if offsets[e + 1] > offsets[e]}
    tokens = []
    for t in order:
        hit = need & {int(e) for e in ids[t]}
        if hit:
            tokens.append(int(t))
            need -= hit
        if not need:
            break
    for t in order:
        if len(tokens) >= n_tokens:
            break
        if int(t) not in tokens:
            tokens.append(int(t))
    rows = set()
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        rows.update((lo, hi - 1))
        if e < hot_experts:
            rows.update(r for r in (lo + 64, lo + 127) if r < hi)
            rows.add(lo + ((hi - lo - 1) // 128) * 128)
        if e >= E - tail_experts:
            rows.update(range(lo + int(rng.integers(0, 128)) % max(1, min(128, hi - lo)), hi, 128))
    return sorted(tokens), sorted(rows)


def check_moe_sampled(res, x, logits, shape, w13_bf16_of, w2_bf16_of, nsel13, nsel2, a2_gs,
                      n_tokens=64, n_features=96, n_columns=128, tail_experts=8, renormalize=True, seed=99):
    """Full-size variant: everything that is cheap on the CPU is compared in
    full and bit-exactly (routing, dispatch, Q_A(x), selection, residual, and the
    requantization of the implementation's own h); the two GEMMs are compared on
    sampled outputs the oracle computes one by one (see sample_plan): for every
    sampled dispatched row, `n_features` features of h (every 128-feature tile
    of the first projection is hit) against the float64 contraction; for every
    sampled token, `n_columns` columns of `out` (every 256-column tile hit)
    against the float64 contraction of the implementation's own quantized h.
    Each expert's weights are quantized by the oracle once: the per-tensor scale
    from the whole tensor, codes and block scales for the sampled rows only.
    w13_bf16_of / w2_bf16_of: callables expert -> bf16 torch weight [N, K]."""
    report = {}
    xf = f32(x)
    lg = logits.cpu().numpy()
    T, H = xf.shape
    topk, E, I = shape.topk, shape.E, shape.I
    ids, wts = M.route(lg, topk, renormalize)
    counts, offsets, perm = M.dispatch(ids, E)
    assert np.array_equal(res["ids"].cpu().numpy(), ids), "top-k ids differ"
    assert np.allclose(res["weights"].cpu().numpy(), wts, rtol=2e-5, atol=1e-7)
    assert np.array_equal(res["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(res["perm"].cpu().numpy(), perm)
    site13 = R.rac(xf, nsel13)
    check_site1(res, dict(site13=site13), nsel13, report)
    # ---- site 2 on the implementation's own h, in full
    h_gpu = f32(res["h"])
    site2 = R.rac(h_gpu, nsel2, a2_gs)
    assert np.array_equal(res["hq"].cpu().numpy(), F.pack_nibbles(site2["codes"])), "Q_A(h) codes differ"
    assert np.array_equal(res["hsf"].cpu().numpy(), site2["sf"]), "Q_A(h) scales differ"
    if nsel2 > 0:
        ok, ndiff = sel_matches(res["sel2"].cpu().numpy(), site2, nsel2)
        assert ok, "site-2 selection differs beyond ties (%d channels)" % ndiff
        report["sel2_tie_swaps"] = ndiff
        if ndiff:
            site2 = M._force_selection(h_gpu, site2, res["sel2"].cpu().numpy()[:nsel2])
        assert np.array_equal(res["r2q"].cpu().numpy(), F.pack_nibbles(site2["r_codes"])), "residual-of-h codes differ"
        assert np.array_equal(res["r2sf"].cpu().numpy(), site2["r_sf"]), "residual-of-h scales differ"
    report["site2_bit_exact"] = True
    # ---- sampled GEMM outputs
    tokens, extra_rows = sample_plan(ids, offsets, topk, shape.hot_experts, n_tokens, tail_experts, seed)
    inv = np.empty(T * topk, dtype=np.int64)
    inv[perm] = np.arange(T * topk)
    tok_rows = {int(inv[t * topk + s]): (t, s) for t in tokens for s in range(topk)}
    rows = sorted(set(extra_rows) | set(tok_rows))
    row_expert = np.searchsorted(offsets, np.asarray(rows), side="right") - 1
    tok_of = perm // topk
    rng = np.random.default_rng(seed + 1)

    def spread(n_total, tile, n_pick):
        """n_pick indices of range(n_total): the first, the last, and a seeded
        choice with every `tile`-sized tile represented."""
        per = max(1, n_pick // max(1, n_total // tile))
        pick = {0, n_total - 1}
        for t0 in range(0, n_total, tile):
            pick.update(int(v) for v in t0 + rng.choice(min(tile, n_total - t0), size=min(per, n_total - t0), replace=False))
        return np.array(sorted(pick), dtype=np.int64)

    cols = spread(H, 256, n_columns)
    xt_all = R.reconstruct_real(site13)
    xa_all = (np.abs(Q.dequantize_real(site13["codes"], site13["sf"], site13["gs"]))
              + np.abs(Q.dequantize_real(site13["r_codes"], site13["r_sf"], site13["r_gs"])))
    out_gpu = f32(res["out"]).astype(np.float64)
    o64 = {t: np.zeros(cols.size) for t in tokens}
    oad = {t: np.zeros(cols.size) for t in tokens}
    worst_h, n_h, experts_hit, tiles_hit = 0.0, 0, set(), set()
    for e in sorted(set(int(v) for v in row_expert)):
        mine = [r for r, re_ in zip(rows, row_expert) if re_ == e]
        experts_hit.add(e)
        w13 = f32(w13_bf16_of(e))                               # [2I, H] bf16 values
        feats = spread(I, 128, n_features)
        gs13 = Q.tensor_global_scale(w13)                      # per-tensor scale: from the WHOLE tensor
        sub = np.concatenate([w13[feats], w13[I + feats]])     # gate rows, then up rows of the sampled features
        c13, s13, _ = Q.quantize(sub, gs13)
        wd = Q.dequantize_real(c13, s13, gs13)
        toks = tok_of[np.asarray(mine)]
        g = xt_all[toks] @ wd.T
        gad = xa_all[toks] @ np.abs(wd).T
        nf = feats.size
        gate, up = g[:, :nf], g[:, nf:]
        sig = 1.0 / (1.0 + np.exp(-gate))
        h64 = gate * sig * up
        dsilu = sig * (1.0 + gate * (1.0 - sig))
        dg, du = GEMM_RTOL * gad[:, :nf], GEMM_RTOL * gad[:, nf:]
        tol_h = (np.abs(dsilu * up) * dg + np.abs(gate * sig) * du + dg * du * 2
                 + (BF16_ULP + 1e-5) * np.abs(h64) + 1e-30)
        got = h_gpu[np.asarray(mine)][:, feats]
        worst_h = max(worst_h, float((np.abs(got - h64) / tol_h).max()))
        n_h += got.size
        tiles_hit.update((e, (r - int(offsets[e])) // 128) for r in mine)
        # second projection on the implementation's own quantized h, for the rows of sampled tokens
        mine_tok = [r for r in mine if r in tok_rows]
        if mine_tok:
            w2 = f32(w2_bf16_of(e))                             # [H, I]
            gs2 = Q.tensor_global_scale(w2)
            c2, s2, _ = Q.quantize(w2[cols], gs2)
            w2d = Q.dequantize_real(c2, s2, gs2)
            idx = np.asarray(mine_tok)
            one = {k: (v[idx] if isinstance(v, np.ndarray) and v.ndim == 2 and v.shape[0] == h_gpu.shape[0] else v)
                   for k, v in site2.items()}
            ht = R.reconstruct_real(one)
            ha = (np.abs(Q.dequantize_real(one["codes"], one["sf"], one["gs"]))
                  + np.abs(Q.dequantize_real(one["r_codes"], one["r_sf"], one["r_gs"])))
            y, ya = ht @ w2d.T, ha @ np.abs(w2d).T
            for k, r in enumerate(mine_tok):
                t, s_ = tok_rows[r]
                o64[t] += float(wts[t, s_]) * y[k]
                oad[t] += float(wts[t, s_]) * ya[k]
    worst_o = 0.0
    for t in tokens:
        tol_o = gemm_tol(oad[t], o64[t]) + 4e-5 * oad[t]
        worst_o = max(worst_o, float((np.abs(out_gpu[t][cols] - o64[t]) / tol_o).max()))
    report["h_max_err_over_tol"] = worst_h
    report["out_max_err_over_tol"] = worst_o
    report["sampled_tokens"] = len(tokens)
    report["sampled_rows"] = len(rows)
    report["sampled_experts"] = len(experts_hit)
    report["sampled_row_tiles"] = len(tiles_hit)
    report["h_values_checked"] = n_h
    report["out_values_checked"] = len(tokens) * int(cols.size)
    assert worst_h <= 1.0, "h outside tolerance: %g" % worst_h
    assert worst_o <= 1.0, "out outside tolerance: %g" % worst_o
    return report
