"""Seeded synthetic inputs with the shapes and value distributions of the five
benchmark workloads.  This module holds none of the method's arithmetic: it
only draws random tensors (torch CPU generators / numpy Generators, fixed
seeds), rounds them to bf16 because bf16 is the input format, and shapes the
router logits.  Both the CUDA tests and the CPU oracle read the same bytes.

Workloads (T tokens, H hidden, E experts, top-k routing, I SwiGLU width):
  dense   : X [128,512] ~ N(0,1) with channels {3,141,278,415} x20,
            W [N=256,K=512] ~ N(0, 0.02^2); 16 compensated channels.
  decode  : T=256,  H=2048, E=128, k=8, I=768,  weights std 0.02,
            20 of 2048 channels = 10 * Student-t(3).
  prefill : T=8192, same layer; router biased so experts 0..7 get 25 % of
            the assignments.
  large   : T=4096, H=4096, E=128, k=8, I=1536, weights std 0.015,
            20 of 4096 channels = 16 * Student-t(2.5).
  aqat    : 48 layers x 128 experts x (W13 [3072,4096] + W2 [4096,1536]),
            std 0.015 (one layer's tensors at a time).
"""
from dataclasses import dataclass

import numpy as np
import torch


@dataclass(frozen=True)
class MoEShape:
    name: str
    seed: int
    T: int
    H: int
    E: int
    topk: int
    I: int
    w_std: float
    n_heavy: int          # number of heavy-tailed channels
    heavy_nu: float
    heavy_scale: float
    hot_experts: int = 0  # >0: bias the router so that experts 0..hot-1 ...
    hot_share: float = 0.0  # ... receive this share of the assignments
    weight_seed: int = -1   # >= 0: draw the expert weights from this seed (a shared layer)


MOE_SHAPES = {
    "decode": MoEShape("decode", 1, 256, 2048, 128, 8, 768, 0.02, 20, 3.0, 10.0),
    "prefill": MoEShape("prefill", 2, 8192, 2048, 128, 8, 768, 0.02, 20, 3.0, 10.0, 8, 0.25, weight_seed=1),
    "large": MoEShape("large", 3, 4096, 4096, 128, 8, 1536, 0.015, 20, 2.5, 16.0),
    # small layers for tests: several tiles, ragged expert segments, empty experts
    "tiny": MoEShape("tiny", 11, 96, 256, 8, 2, 128, 0.05, 3, 3.0, 10.0),
    "small": MoEShape("small", 12, 333, 512, 16, 4, 256, 0.03, 5, 3.0, 10.0, 2, 0.4),
}

DENSE_OUTLIER_CHANNELS = (3, 141, 278, 415)

# Static per-tensor scale of the SwiGLU output h (a calibration constant the
# caller of the MoE layer supplies; values above 2688 * scale saturate).
H_GLOBAL_SCALE = {"decode": 0.25, "prefill": 0.25, "large": 0.5}


def _gen(seed, stream):
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) * 1000003 + int(stream))
    return g


def to_bf16(t):
    """float32 tensor -> bf16 tensor (the inputs of the method are bf16)."""
    return t.to(torch.bfloat16)


def dense_inputs(seed=0, T=128, K=512, N=256, w_std=0.02, outlier_scale=20.0,
                 outlier_channels=DENSE_OUTLIER_CHANNELS):
    x = torch.randn(T, K, generator=_gen(seed, 1))
    for c in outlier_channels:
        if c < K:
            x[:, c] *= outlier_scale
    w_kn = torch.randn(K, N, generator=_gen(seed, 2)) * w_std      # drawn as [K, N]
    return to_bf16(x), to_bf16(w_kn.t().contiguous())              # stored [N, K], K contiguous


def activations(shape: MoEShape):
    x = torch.randn(shape.T, shape.H, generator=_gen(shape.seed, 1))
    rng = np.random.default_rng(shape.seed * 7919 + 17)
    chans = np.sort(rng.choice(shape.H, size=shape.n_heavy, replace=False))
    heavy = rng.standard_t(shape.heavy_nu, size=(shape.T, shape.n_heavy)) * shape.heavy_scale
    x[:, torch.from_numpy(chans)] = torch.from_numpy(heavy.astype(np.float32))
    return to_bf16(x), chans


def router_logits(shape: MoEShape):
    logits = torch.randn(shape.T, shape.E, generator=_gen(shape.seed, 3))
    if shape.hot_experts > 0:
        lo, hi = 0.0, 16.0
        target = shape.hot_share
        for _ in range(40):                      # bisection on the bias
            b = 0.5 * (lo + hi)
            z = logits.clone()
            z[:, :shape.hot_experts] += b
            ids = torch.topk(z, shape.topk, dim=1).indices
            share = (ids < shape.hot_experts).float().mean().item()
            if abs(share - target) <= 0.0025:
                break
            if share < target:
                lo = b
            else:
                hi = b
        logits[:, :shape.hot_experts] += b
    return logits.contiguous()


def expert_weights(shape: MoEShape, which, experts=None):
    """bf16 weights of the experts in `experts` (default all): which='w13' gives
    [n, 2I, H] (gate rows, then up rows), which='w2' gives [n, H, I]."""
    experts = range(shape.E) if experts is None else experts
    N, K = (2 * shape.I, shape.H) if which == "w13" else (shape.H, shape.I)
    stream0 = 100 if which == "w13" else 100000
    out = torch.empty(len(experts), N, K, dtype=torch.bfloat16)
    for i, e in enumerate(experts):
        wseed = shape.weight_seed if shape.weight_seed >= 0 else shape.seed
        w = torch.randn(N, K, generator=_gen(wseed, stream0 + e)) * shape.w_std
        out[i] = to_bf16(w)
    return out


def aqat_layer_weights(layer, n_experts=128, seed=4, std=0.015, which="w13",
                       shape_w13=(3072, 4096), shape_w2=(4096, 1536)):
    """One layer of the fake-quant workload, [n_experts, N, K] bf16."""
    N, K = shape_w13 if which == "w13" else shape_w2
    stream = layer * 2 + (0 if which == "w13" else 1)
    w = torch.randn(n_experts, N, K, generator=_gen(seed, stream)) * std
    return to_bf16(w)
