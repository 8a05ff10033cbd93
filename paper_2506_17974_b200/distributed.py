"""One LQ-SGD round with the workers spread over several processes / GPUs.

Algorithm 1 exchanges the quantised factors twice per iteration (its two All-Reduce steps, Section IV-A).  Each rank simulates `workers` local workers with the CUDA library; this module only
sequences the library's round pieces and the collectives between them on torch.distributed
(NCCL on GPUs): a MAX all-reduce of one scale per matrix and an all-gather of the packed b-bit
streams, per factor.  The wire therefore carries r(n+m)b bits per worker (Section IV-C) plus the
scales; every rank then forms the exact integer sum of all workers' codes itself.

`comp` is anything with the library's round interface (paper_2506_17974_b200.binding.LQSGD):
round_begin / round_pack / round_reduce / round_end / exchange_view, a `layers` list and
`is_matrix(layer)`.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch
import torch.distributed as dist

XCHG_SCALES_P, XCHG_SCALES_Q, XCHG_STREAMS_P, XCHG_STREAMS_Q = range(4)


def distributed_round(comp, grads, ghat: Sequence[torch.Tensor], group: Optional[dist.ProcessGroup] = None,
                      weights=None, lr: float = 0.0) -> None:
    """Runs one round on this rank's workers and averages over all ranks' workers."""
    world = dist.get_world_size(group)
    # the fused model update only sees this rank's share of a 1-D tensor's mean: update those here
    fused = None if weights is None else [wt if comp.is_matrix(l) else None for l, wt in enumerate(weights)]
    comp.round_begin(grads, ghat, fused, lr)
    cache = getattr(comp, "_xchg_cache", None)          # views of fixed buffers and the gather targets
    if cache is None or cache.get("world") != world:
        cache = {"world": world}
        try:
            comp._xchg_cache = cache
        except AttributeError:
            pass
    for which, scales_id, streams_id in ((0, XCHG_SCALES_P, XCHG_STREAMS_P), (1, XCHG_SCALES_Q, XCHG_STREAMS_Q)):
        scales = comp.exchange_view(scales_id)
        if scales.numel():
            dist.all_reduce(scales, op=dist.ReduceOp.MAX, group=group)       # one shared scale per factor and layer
        comp.round_pack(which)
        send = comp.exchange_view(streams_id)
        gathered = cache.get(("gathered", which))
        if gathered is None or gathered.numel() != world * send.numel() or gathered.device != send.device:
            gathered = torch.empty(world * send.numel(), dtype=send.dtype, device=send.device)
            cache[("gathered", which)] = gathered
        if send.numel():
            dist.all_gather_into_tensor(gathered, send, group=group)          # the packed codes of every worker
        comp.round_reduce(which, gathered, world)
    comp.round_end()
    for l in range(len(comp.layers)):                                         # 1-D tensors: shares of the mean
        if not comp.is_matrix(l):
            if ghat is not None and ghat[l] is not None:
                dist.all_reduce(ghat[l], op=dist.ReduceOp.SUM, group=group)
                if weights is not None and weights[l] is not None:
                    weights[l].add_(ghat[l], alpha=-lr)
            elif weights is not None and weights[l] is not None:
                raise ValueError("a 1-D tensor needs its ghat buffer when its weights are to be updated across ranks")
