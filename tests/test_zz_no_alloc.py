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


def test_noalloc_rejects_more_tensors_than_its_scratch_holds():
    from paper_2607_15810_b200 import binding as B
    w = torch.zeros(1, 16, 64, dtype=torch.bfloat16).cuda()
    with pytest.raises(B.QuadsError) as err:
        B.fake_quant_weights_noalloc(w, _outs(w), n_tensors=B.NOALLOC_MAX_TENSORS + 1)
    assert err.value.status == -7 and "capacity" in str(err.value)
