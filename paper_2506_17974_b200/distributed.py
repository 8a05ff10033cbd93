"""One LQ-SGD round with the workers spread over several processes / GPUs.

Algorithm 1 exchanges the quantised factors twice per iteration (its two All-Reduce steps, Section IV-A).
Each rank simulates `workers` local workers with the CUDA library; this module only sequences the
library's round pieces and the collectives between them on torch.distributed (NCCL on GPUs): per factor a
MAX all-reduce of the scales and an all-gather of the packed b-bit streams, plus one SUM all-reduce of the
flat buffer that holds every 1-D tensor's mean - five collectives per round, whatever the number of layers.
The wire therefore carries r(n+m)b bits per worker (Section IV-C) plus the scales; every rank then forms the
exact integer sum of all workers' codes itself.  All arithmetic, the 1-D tensors' means and the model update
included, runs in the library's kernels.

`comp` is anything with the library's round interface (paper_2506_17974_b200.binding.LQSGD):
round_begin / round_pack / round_reduce / round_end / exchange_view.

distributed_round          the round of one compressor, its collectives in line with its kernels.
distributed_round_overlapped   the layer table cut in two (two compressors, see split_layers): the second half's
                           pass 1 is issued before the first half's exchange, so that the collectives of one
                           half run under the streaming passes of the other (two CUDA streams).
"""
from __future__ import annotations

import contextlib
from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

XCHG_SCALES_P, XCHG_SCALES_Q, XCHG_STREAMS_P, XCHG_STREAMS_Q, XCHG_VECTORS = range(5)


def _gather_buffer(comp, which: int, send: torch.Tensor, world: int) -> torch.Tensor:
    cache = getattr(comp, "_xchg_cache", None)          # the gather targets are kept between rounds
    if cache is None or cache.get("world") != world:
        cache = {"world": world}
        try:
            comp._xchg_cache = cache
        except AttributeError:
            pass
    buf = cache.get(("gathered", which))
    if buf is None or buf.numel() != world * send.numel() or buf.device != send.device or buf.dtype != send.dtype:
        buf = torch.empty(world * send.numel(), dtype=send.dtype, device=send.device)
        cache[("gathered", which)] = buf
    return buf


def _exchange_factor(comp, which: int, group, world: int) -> None:
    """Scales (MAX), pack, streams (all-gather), sum + dequantise + what follows in the library."""
    scales = comp.exchange_view(XCHG_SCALES_Q if which else XCHG_SCALES_P)
    if scales.numel():
        dist.all_reduce(scales, op=dist.ReduceOp.MAX, group=group)           # the scales every rank quantises with
    comp.round_pack(which)
    send = comp.exchange_view(XCHG_STREAMS_Q if which else XCHG_STREAMS_P)
    gathered = _gather_buffer(comp, which, send, world)
    if send.numel():
        dist.all_gather_into_tensor(gathered, send, group=group)             # the packed codes of every worker
    comp.round_reduce(which, gathered, world)


def _exchange_vectors(comp, group) -> None:
    vec = comp.exchange_view(XCHG_VECTORS)
    if vec.numel():
        dist.all_reduce(vec, op=dist.ReduceOp.SUM, group=group)              # every 1-D tensor's mean, one collective


def distributed_round(comp, grads, ghat: Sequence[torch.Tensor], group: Optional[dist.ProcessGroup] = None,
                      weights=None, lr: float = 0.0) -> None:
    """Runs one round on this rank's workers and averages over all ranks' workers."""
    world = dist.get_world_size(group)
    comp.round_begin(grads, ghat, weights, lr)
    _exchange_factor(comp, 0, group, world)
    _exchange_factor(comp, 1, group, world)
    _exchange_vectors(comp, group)
    comp.round_end()


def split_layers(layers: Sequence[Tuple[int, int]]) -> Tuple[List[int], List[int]]:
    """Cuts a layer table in two halves of about equal matrix size (largest first to the lighter half);
    the 1-D tensors go with the first half.  Returns the two lists of layer indices, each in table order."""
    halves, load = ([], []), [0, 0]
    mats = [(i, s) for i, s in enumerate(layers) if s[0] > 1 and s[1] > 1]
    for i, s in sorted(mats, key=lambda x: -x[1][0] * x[1][1]):
        k = 0 if load[0] <= load[1] else 1
        halves[k].append(i)
        load[k] += s[0] * s[1]
    halves[0].extend(i for i, s in enumerate(layers) if not (s[0] > 1 and s[1] > 1))
    return sorted(halves[0]), sorted(halves[1])


def distributed_round_overlapped(parts, group: Optional[dist.ProcessGroup] = None, streams=None) -> None:
    """One round over a layer table cut in two.  parts: two tuples (comp, grads, ghat[, weights, lr]), one per half
    (each comp built on its half's layers, see split_layers); streams: two CUDA streams, or None to run the same
    sequence on the current stream (CPU stand-ins).  Issue order: pass 1 of both halves, then the halves' exchanges
    in turn - a collective of one half is then in flight while the other half's kernels run.  The caller joins the
    two streams afterwards (stream.synchronize(), or wait_stream)."""
    assert len(parts) == 2
    world = dist.get_world_size(group)

    def on(k):
        return torch.cuda.stream(streams[k]) if streams is not None else contextlib.nullcontext()

    comps = []
    for k, part in enumerate(parts):
        comp, grads, ghat = part[0], part[1], part[2]
        weights, lr = (part[3], part[4]) if len(part) > 3 else (None, 0.0)
        comps.append(comp)
        with on(k):
            comp.round_begin(grads, ghat, weights, lr)
    for which in (0, 1):
        for k, comp in enumerate(comps):
            with on(k):
                _exchange_factor(comp, which, group, world)
    for k, comp in enumerate(comps):
        with on(k):
            _exchange_vectors(comp, group)
            comp.round_end()
