"""The allocation-free fake-quant entry point, for callers that cannot call
cudaMalloc (device memory owned by someone else's pool, or no allocation
allowed after start-up).  It must give exactly what the workspace-taking entry
point gives, on two calls in a row that share its built-in scratch array, and
refuse a batch beyond its stated capacity.  Collected last on purpose."""
import gc

import pytest
import torch

pytestmark = pytest.mark.gpu


def _outs(w):
    n, N, K = w.shape
    return (torch.empty_like(w), torch.empty(n, N, K // 2, dtype=torch.uint8, device=w.device),
            torch.empty(n, N, K // 16, dtype=torch.uint8, device=w.device),
            torch.empty(n, dtype=torch.float32, device=w.device))


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    from paper_2607_15810_b200 import binding as B
    g = torch.Generator().manual_seed(123)
    # the second batch is smaller in magnitude and count: stale amax words from
    # the first call would give it wrong (too large) tensor scales
    batches = [(torch.randn(5, 128, 256, generator=g) * 3.0).to(torch.bfloat16).cuda(),
               (torch.randn(3, 128, 256, generator=g) * 0.01).to(torch.bfloat16).cuda()]
    for w in batches:
        ref = B.fake_quant_weights(w)
        outs = _outs(w)
        gc.collect()                                   # tensors kept alive by reference cycles of earlier tests
        before = torch.cuda.memory_allocated()
        B.fake_quant_weights_noalloc(w, outs)
        assert torch.cuda.memory_allocated() == before
        torch.cuda.synchronize()
        assert torch.equal(outs[3], ref["gs"])
        assert torch.equal(outs[1], ref["q"])
        assert torch.equal(outs[2], ref["sf"])
        assert torch.equal(outs[0].view(torch.int16), ref["w_fq"].view(torch.int16))


def test_noalloc_single_tensor_and_batch_against_the_oracle():
    """One tensor takes another kernel than a batch does (both use the built-in scratch array); each
    is compared with the CPU oracle directly, and the device's free memory is the same before and
    after the calls (a cudaMalloc inside the library would show there; torch's own counter would
    not see it)."""
    import numpy as np
    from oracle import formats as F
    from oracle import nvfp4 as Q
    from paper_2607_15810_b200 import binding as B
    g = torch.Generator().manual_seed(321)
    cases = [(torch.randn(1, 200, 320, generator=g) * 0.5).to(torch.bfloat16),
             (torch.randn(4, 64, 128, generator=g) * 0.02).to(torch.bfloat16)]
    dev = [(w.cuda(), _outs(w.cuda())) for w in cases]
    for w, outs in dev:                                 # warm-up: module load, kernel attributes, symbol lookup
        B.fake_quant_weights_noalloc(w, outs)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for w, outs in dev:
        for o in outs:
            o.zero_()
        B.fake_quant_weights_noalloc(w, outs)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    for wc, (w, outs) in zip(cases, dev):
        wf_o, q_o, sf_o, gs_o = Q.fake_quant_weights(wc.to(torch.float32).numpy())
        assert np.array_equal(outs[3].cpu().numpy(), gs_o)
        assert np.array_equal(outs[1].cpu().numpy(), q_o)
        assert np.array_equal(outs[2].cpu().numpy(), sf_o)
        assert np.array_equal(F.bf16_bits(outs[0].to(torch.float32).cpu().numpy()), F.bf16_bits(wf_o))


def test_noalloc_rejects_more_tensors_than_its_scratch_holds():
    from paper_2607_15810_b200 import binding as B
    w = torch.zeros(1, 16, 64, dtype=torch.bfloat16).cuda()
    with pytest.raises(B.QuadsError) as err:
        B.fake_quant_weights_noalloc(w, _outs(w), n_tensors=B.NOALLOC_MAX_TENSORS + 1)
    assert err.value.status == -7 and "capacity" in str(err.value)
    with pytest.raises(B.QuadsError) as err:             # a negative count is a shape error, not a capacity one
        B.fake_quant_weights_noalloc(w, _outs(w), n_tensors=-1)
    assert err.value.status == -2
