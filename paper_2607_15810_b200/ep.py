"""Expert-parallel execution of the MoE layer over several GPUs, one process per GPU: every rank holds
the weights of a contiguous range of experts and the whole token batch (token-replicated expert
parallelism), calls the library once on its range and the partial sums are added with ONE all-reduce
of float32 [T, H] (NCCL over NVLink; a sum has no data-dependent routing, so no all-to-all sizes need
to be exchanged).  Quantization of x, its channel statistics and the site-13 selection are computed
from the whole batch on every rank and therefore agree; the site-2 selection is taken on each rank's
own dispatched rows.  Argument marshalling and the collective only: all arithmetic runs in the
library's kernels."""
import torch


def expert_range(rank, world, n_experts):
    """Contiguous, balanced split of the experts: (lo, hi) of `rank`."""
    base, rem = divmod(n_experts, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def shard_weights(w, lo, hi):
    """The entries of a packed-weight dict (q, sf, gs with a leading expert dimension) for experts lo..hi-1."""
    return {k: v[lo:hi].contiguous() for k, v in w.items() if v is not None}


def moe_w4a4_rac_expert_parallel(binding, x, logits, local_w13, local_w2, topk, nsel13, nsel2, a2_gs, rank, world,
                                 group=None, all_reduce=None, **kw):
    """One rank's part of the layer.  local_w13 / local_w2: this rank's experts only.  Returns the
    layer output bf16 [T, H] (identical on every rank after the all-reduce).  `all_reduce` defaults to
    torch.distributed.all_reduce on `group`."""
    T, H = x.shape
    E = logits.shape[1]
    lo, hi = expert_range(rank, world, E)
    part = torch.empty(T, H, dtype=torch.float32, device=x.device)
    binding.moe_w4a4_rac(x, logits, local_w13, local_w2, topk, nsel13, nsel2, a2_gs, expert_range=(lo, hi), out_f32=part, **kw)
    if all_reduce is None:
        import torch.distributed as dist
        dist.all_reduce(part, group=group)
    else:
        all_reduce(part)
    return part.to(torch.bfloat16)
