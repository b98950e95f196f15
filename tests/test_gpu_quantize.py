"""CUDA quantize / fake-quant against the oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import formats as F
from oracle import nvfp4 as Q

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2607_15810_b200 import binding
    return binding


def _f32(t):
    return t.to(torch.float32).cpu().numpy()


def _bf16(shape, seed, scale=1.0):
    return (torch.randn(*shape, generator=torch.Generator().manual_seed(seed)) * scale).to(torch.bfloat16)


def _tiled_index(rows, K):
    KT = (K + 63) // 64
    r = np.arange(rows)[:, None]
    kb = np.arange(K // 16)[None, :]
    return ((r >> 7) * KT + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3)


@pytest.mark.parametrize("rows,K,seed", [(128, 512, 0), (1, 16, 1), (7, 64, 2), (333, 2048, 3), (129, 4096, 4),
                                         (8192, 2048, 5)])
def test_quantize_bit_exact(B, rows, K, seed):
    x = _bf16((rows, K), seed, 3.0)
    if K >= 64:
        x[:, 5] *= 20
    if rows > 3:
        x[2, :16] = 0
    q, sf, gs = B.quantize_nvfp4(x.cuda())
    c_o, s_o, g_o = Q.quantize(_f32(x))
    assert np.float32(gs.item()) == g_o
    assert np.array_equal(sf.cpu().numpy(), s_o)
    assert np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o))
    q2, sf2, _ = B.quantize_nvfp4(x.cuda(), sf_layout=B.SF_TILED)
    assert np.array_equal(q2.cpu().numpy(), F.pack_nibbles(c_o))
    assert np.array_equal(sf2.cpu().numpy()[_tiled_index(rows, K)], s_o)


def test_quantize_supplied_scale_strided_and_empty(B):
    big = _bf16((50, 256), 7)
    x = big[:, :128]                                    # row stride 256
    gs = torch.tensor([0.01], dtype=torch.float32)
    q, sf, g = B.quantize_nvfp4(x.cuda() if False else big.cuda()[:, :128], gs=gs.cuda())
    c_o, s_o, g_o = Q.quantize(_f32(x), np.float32(0.01))
    assert np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o)) and np.array_equal(sf.cpu().numpy(), s_o)
    assert g.item() == np.float32(0.01)
    # saturating scale
    q, sf, g = B.quantize_nvfp4(big.cuda(), gs=torch.tensor([1e-6]).cuda())
    c_o, s_o, _ = Q.quantize(_f32(big), np.float32(1e-6))
    assert np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o)) and np.array_equal(sf.cpu().numpy(), s_o)
    # all-zero tensor and zero rows
    z = torch.zeros(4, 64, dtype=torch.bfloat16).cuda()
    q, sf, g = B.quantize_nvfp4(z)
    assert g.item() == 1.0 and not sf.any() and not q.any()
    q, sf, g = B.quantize_nvfp4(torch.empty(0, 64, dtype=torch.bfloat16).cuda())
    assert g.item() == 1.0 and q.numel() == 0


def test_every_scale_code_and_every_tie(B):
    """Blocks whose amax sweeps every E4M3 code and every midpoint between two
    codes (with the float32 neighbours of the midpoints), and elements that
    sit on every E2M1 tie: the hardware conversions must agree with the
    oracle's tables everywhere."""
    mags = F.E4M3_MAGNITUDES
    mids = 0.5 * (mags[:-1] + mags[1:])
    u = np.concatenate([mags, mids]).astype(np.float32)
    gs = np.float32(1.0 / 64)                            # power of two: amax/(6 gs) exact
    amax = (u.astype(np.float64) * 6 * float(gs))
    amax_bf = torch.tensor(amax, dtype=torch.float32).to(torch.bfloat16)   # bf16-representable subset decides
    n = amax_bf.numel()
    x = torch.zeros(n, 16, dtype=torch.bfloat16)
    x[:, 0] = amax_bf
    frac = torch.tensor([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -0.75, -1.25, -1.75, -2.5, -3.5, -5.0, 0.0])
    x[:, 1:] = (amax_bf.to(torch.float32)[:, None] / 6.0 * frac[None, :]).to(torch.bfloat16)
    g = torch.tensor([float(gs)])
    q, sf, _ = B.quantize_nvfp4(x.cuda(), gs=g.cuda())
    c_o, s_o, _ = Q.quantize(_f32(x), gs)
    assert len(set(s_o.reshape(-1).tolist())) > 100      # the sweep really covers the code space
    assert np.array_equal(sf.cpu().numpy(), s_o)
    assert np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o))
    # every finite bf16 magnitude through the element rounding with unit scales
    bits = torch.arange(0, 0x7F80, dtype=torch.int32).to(torch.int16).view(torch.bfloat16)
    keep = bits.to(torch.float32) <= 8.0
    v = bits[keep]
    v = torch.cat([v, -v])
    pad = (-v.numel()) % 15
    v = torch.cat([v, torch.zeros(pad, dtype=torch.bfloat16)]).view(-1, 15)
    x = torch.cat([torch.full((v.shape[0], 1), 6.0, dtype=torch.bfloat16), v], dim=1)
    q, sf, _ = B.quantize_nvfp4(x.cuda(), gs=torch.tensor([1.0]).cuda())
    c_o, s_o, _ = Q.quantize(_f32(x), np.float32(1.0))
    assert np.array_equal(sf.cpu().numpy(), s_o) and np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o))


@pytest.mark.parametrize("n,N,K", [(3, 256, 512), (1, 3072, 4096), (5, 100, 80), (2, 4096, 1536)])
def test_fake_quant_bit_exact_and_trainer_equals_rollout(B, n, N, K):
    w = _bf16((n, N, K), 11 + n, 0.015)
    r = B.fake_quant_weights(w.cuda())
    wf_o, q_o, sf_o, gs_o = Q.fake_quant_weights(_f32(w))
    assert np.array_equal(r["gs"].cpu().numpy(), gs_o)
    assert np.array_equal(r["q"].cpu().numpy(), q_o)
    assert np.array_equal(r["sf"].cpu().numpy(), sf_o)
    assert np.array_equal(F.bf16_bits(_f32(r["w_fq"])), F.bf16_bits(wf_o))
    # rollout side: dequantize the packed bytes the GPU wrote (oracle arithmetic) == the GPU's bf16 fake-quant
    for i in range(n):
        roll = Q.dequantize_bf16(F.unpack_nibbles(r["q"][i].cpu().numpy()), r["sf"][i].cpu().numpy(),
                                 r["gs"][i].item())
        assert np.array_equal(F.bf16_bits(roll), F.bf16_bits(_f32(r["w_fq"][i])))
    # pack-only and fake-quant-only give the same bytes; tiled layout holds the same scales
    p = B.fake_quant_weights(w.cuda(), want_fq=False, sf_layout=B.SF_TILED)
    assert np.array_equal(p["q"].cpu().numpy(), q_o)
    idx = _tiled_index(N, K)
    assert np.array_equal(p["sf"].cpu().numpy()[:, idx], sf_o)
    f = B.fake_quant_weights(w.cuda(), want_pack=False)
    assert f["q"] is None and np.array_equal(F.bf16_bits(_f32(f["w_fq"])), F.bf16_bits(wf_o))


@pytest.mark.parametrize("n,N,K", [
    (40, 64, 128),       # more tensors than the kernel keeps in flight; 4 blocks per CTA, none for some CTAs
    (256, 256, 128),     # many tensors, 16 blocks per CTA, 20 CTAs without any: their arrivals must still count
    (2, 8, 16),          # two tensors of one block each
    (9, 1000, 2048),     # a share of 868 blocks: one full chunk and a ragged one, dealt to rotating groups
    (6, 1536, 2048),     # the 30B-A3B expert shape: 3 chunks per share over 4 groups
    (3, 3072, 4096),     # the 235B-A22B expert shape: 12 chunks per share
])
def test_fake_quant_batch_kernel_equals_grouped_kernel_and_oracle(B, n, N, K, monkeypatch):
    """A batch of tensors goes through the shared-memory ring kernel; with it switched off the
    same call takes the grouped kernel.  Both must give the oracle's bytes."""
    w = _bf16((n, N, K), 100 + n, 0.02)
    w[0, 0, :16] = 0                                       # an all-zero block
    if n > 2:
        w[2] = 0                                           # an all-zero tensor: scale 1, codes 0
    wc = w.cuda()
    monkeypatch.delenv("QUADS_NO_RING_QUANT", raising=False)
    a = B.fake_quant_weights(wc)
    a_t = B.fake_quant_weights(wc, want_fq=False, sf_layout=B.SF_TILED)
    monkeypatch.setenv("QUADS_NO_RING_QUANT", "1")
    b = B.fake_quant_weights(wc)
    b_t = B.fake_quant_weights(wc, want_fq=False, sf_layout=B.SF_TILED)
    monkeypatch.delenv("QUADS_NO_RING_QUANT")
    for k in ("gs", "q", "sf", "w_fq"):
        assert torch.equal(a[k].view(torch.uint8), b[k].view(torch.uint8)), k
    idx = torch.from_numpy(_tiled_index(N, K).reshape(-1)).cuda()     # (padding bytes of the tiled layout are never written)
    for k in ("gs", "q"):
        assert torch.equal(a_t[k].view(torch.uint8), b_t[k].view(torch.uint8)), k
    assert torch.equal(a_t["sf"][:, idx], b_t["sf"][:, idx])
    wf_o, q_o, sf_o, gs_o = Q.fake_quant_weights(_f32(w))
    assert np.array_equal(a["gs"].cpu().numpy(), gs_o)
    assert np.array_equal(a["q"].cpu().numpy(), q_o)
    assert np.array_equal(a["sf"].cpu().numpy(), sf_o)
    assert np.array_equal(F.bf16_bits(_f32(a["w_fq"])), F.bf16_bits(wf_o))
    assert np.array_equal(a_t["sf"].cpu().numpy()[:, _tiled_index(N, K)], sf_o)


def test_fake_quant_batch_kernel_repeats_bit_for_bit(B):
    w = _bf16((24, 768, 2048), 5, 0.02).cuda()
    first = B.fake_quant_weights(w)
    for _ in range(5):
        again = B.fake_quant_weights(w)
        for k in ("gs", "q", "sf", "w_fq"):
            assert torch.equal(first[k].view(torch.uint8), again[k].view(torch.uint8)), k


@pytest.mark.parametrize("rows,K,seed", [(1, 16, 1), (333, 2048, 3), (2048, 4096, 4)])
def test_activation_fake_quant_decodes_what_the_rollout_operand_holds(B, rows, K, seed):
    x = _bf16((rows, K), seed, 2.0)
    if K >= 64:
        x[:, 7] *= 30
    xf, g = B.fake_quant_activations(x.cuda())
    xf_o, g_o = Q.fake_quant_activations(_f32(x))
    assert np.float32(g.item()) == g_o
    assert np.array_equal(F.bf16_bits(_f32(xf)), F.bf16_bits(xf_o))
    # ... and it is the decode of exactly the bytes quads_quantize_nvfp4 writes
    q, sf, g2 = B.quantize_nvfp4(x.cuda())
    dec = Q.dequantize_bf16(F.unpack_nibbles(q.cpu().numpy()), sf.cpu().numpy(), g2.item())
    assert np.array_equal(F.bf16_bits(dec), F.bf16_bits(_f32(xf)))
    # a given (static) scale and a row stride
    big = _bf16((max(rows, 2), 2 * K), seed + 50, 1.0).cuda()
    gs = torch.tensor([0.004], dtype=torch.float32).cuda()
    xs, _ = B.fake_quant_activations(big[:, :K], gs=gs)
    xs_o, _ = Q.fake_quant_activations(_f32(big[:, :K]), np.float32(0.004))
    assert np.array_equal(F.bf16_bits(_f32(xs)), F.bf16_bits(xs_o))


@pytest.mark.parametrize("n,N,K", [(1, 1, 16), (3, 100, 80), (4, 1536, 2048)])
def test_dequantize_gives_the_trainers_fake_quant_bit_for_bit(B, n, N, K):
    """Eq. weight-qdq-align: decoding the packed bytes on the rollout side gives
    the bf16 tensor the trainer multiplied by -- for both scale layouts, and
    equal to the oracle's decode of the same bytes."""
    w = _bf16((n, N, K), 21 + n, 0.02).cuda()
    lin = B.fake_quant_weights(w)
    til = B.fake_quant_weights(w, sf_layout=B.SF_TILED)
    d_lin = B.dequantize_nvfp4(lin["q"], lin["sf"], lin["gs"], N, K)
    d_til = B.dequantize_nvfp4(til["q"], til["sf"], til["gs"], N, K, sf_layout=B.SF_TILED)
    assert torch.equal(d_lin.view(torch.int16), lin["w_fq"].view(torch.int16))
    assert torch.equal(d_til.view(torch.int16), lin["w_fq"].view(torch.int16))
    for i in range(n):
        dec = Q.dequantize_bf16(F.unpack_nibbles(lin["q"][i].cpu().numpy()), lin["sf"][i].cpu().numpy(), lin["gs"][i].item())
        assert np.array_equal(F.bf16_bits(dec), F.bf16_bits(_f32(d_lin[i])))


@pytest.mark.parametrize("N,K", [(3072, 4096), (4096, 1536)])
def test_aqat_layer_batch_at_full_size_against_the_oracle_on_sampled_tensors(B, N, K):
    """The fake-quant + weight-sync workload in the launch configuration the benchmark times: 128
    expert tensors of one shape in one call (one cooperative launch of the ring kernel).  The batch
    is drawn on the device (seeded); the first, the last and three tensors in between are copied
    back and compared bit for bit with the oracle; trainer == rollout is checked on every tensor."""
    n = 128
    g = torch.Generator(device="cuda").manual_seed(4 * 1000003 + N)
    w = torch.empty(n, N, K, dtype=torch.bfloat16, device="cuda")
    for e0 in range(0, n, 16):
        w[e0:e0 + 16] = (torch.randn(16, N, K, device="cuda", generator=g) * 0.015).to(torch.bfloat16)
    r = B.fake_quant_weights(w)
    torch.cuda.synchronize()
    assert B.last_launch_count() == 1
    assert torch.isfinite(r["gs"]).all()
    # Eq. weight-qdq-align on all 128 tensors: decoding the packed bytes gives the trainer's bf16 bits
    dec = B.dequantize_nvfp4(r["q"], r["sf"], r["gs"], N, K)
    assert torch.equal(dec.view(torch.int16), r["w_fq"].view(torch.int16))
    del dec
    for i in (0, 41, 77, 126, 127):
        wf_o, q_o, sf_o, gs_o = Q.fake_quant_weights(_f32(w[i:i + 1]))
        assert np.array_equal(r["gs"][i:i + 1].cpu().numpy(), gs_o), i
        assert np.array_equal(r["q"][i].cpu().numpy(), q_o[0]), i
        assert np.array_equal(r["sf"][i].cpu().numpy(), sf_o[0]), i
        assert np.array_equal(F.bf16_bits(_f32(r["w_fq"][i])), F.bf16_bits(wf_o[0])), i


def test_a_bounded_wait_that_runs_out_is_reported_and_harmless(B, monkeypatch):
    """Failure detection without a fault: the test hook makes the arrival wait of the quantize kernel
    expect one arrival more than there are CTAs and shortens its bound to about a millisecond.  The
    call must still end, mark its scale as NaN, and leave the library usable: the next ordinary call
    is bit-exact against the oracle."""
    x = _bf16((1, 16), 31, 2.0).cuda()
    monkeypatch.setenv("QUADS_QUANT_COOPERATIVE", "1")        # the single-kernel path, whose CTAs wait for one another
    lib = B.lib
    lib.quads_debug_set_quantize_wait.restype = None
    lib.quads_debug_set_quantize_wait.argtypes = [B.C.c_int64, B.C.c_int32]
    lib.quads_debug_set_quantize_wait(2_000_000, 1)
    try:
        q, sf, gs = B.quantize_nvfp4(x)
        torch.cuda.synchronize()
        assert torch.isnan(gs).all()
        xf, g2 = B.fake_quant_activations(x)
        torch.cuda.synchronize()
        assert torch.isnan(g2).all()
    finally:
        lib.quads_debug_set_quantize_wait(0, 0)
    big = _bf16((333, 2048), 3, 3.0)
    q, sf, gs = B.quantize_nvfp4(big.cuda())                   # still the cooperative kernel: intact after the give-up
    c_o, s_o, g_o = Q.quantize(_f32(big))
    assert np.float32(gs.item()) == g_o and np.array_equal(sf.cpu().numpy(), s_o)
    monkeypatch.delenv("QUADS_QUANT_COOPERATIVE")
    q, sf, gs = B.quantize_nvfp4(big.cuda())                   # and the default two-launch path
    c_o, s_o, g_o = Q.quantize(_f32(big))
    assert np.float32(gs.item()) == g_o and np.array_equal(sf.cpu().numpy(), s_o)
    assert np.array_equal(q.cpu().numpy(), F.pack_nibbles(c_o))
    # with a supplied scale there is no wait at all, hook or not
    lib.quads_debug_set_quantize_wait(2_000_000, 1)
    try:
        q2, sf2, g3 = B.quantize_nvfp4(big.cuda(), gs=gs)
        torch.cuda.synchronize()
    finally:
        lib.quads_debug_set_quantize_wait(0, 0)
    assert torch.equal(q2, q) and torch.equal(sf2, sf) and g3.item() == gs.item()
