"""Host-side bookkeeping for spreading one decode step's keys over several ranks.

A long dense (FA) request can be evaluated in pieces: rank r holds the cache rows of its key range,
computes the piece with ``flux_attn_decode_partial``, the pieces are exchanged with one all-gather
(``B * n_q_heads * 130`` floats per rank and layer) and every rank merges them with
``flux_attn_combine``.  This module only cuts ranges and moves pieces; it holds no attention
arithmetic.  The exchange is a plain ``torch.distributed`` all-gather (NCCL on GPUs, gloo in the CPU
tests).  The second form of the exchange needs no collective: ``flux_attn_decode_partial_push`` stores a
rank's piece into every rank's gather buffer and raises a flag, ``flux_attn_combine_wait`` waits for the
flags; ``exchange_seq`` and ``buffer_set`` give the sequence number and the buffer set that form uses.
"""
from __future__ import annotations

import numpy as np
import torch


def key_ranges(ctx_len, world: int, align: int = 16) -> np.ndarray:
    """Cuts positions ``[0, n_b)`` of every request into ``world`` consecutive ranges of nearly equal size whose
    inner bounds are multiples of ``align`` (the kernels' tile of 16 keys).  Returns int32 ``[world][B][2]``
    (begin, end); ranges can be empty for short requests; together they cover ``[0, n_b)`` exactly once."""
    n = np.asarray(ctx_len, dtype=np.int64)
    assert world >= 1 and align >= 1 and (n >= 0).all()
    out = np.zeros((world, len(n), 2), dtype=np.int32)
    for r in range(world + 1):
        cut = (n * r // world + align - 1) // align * align if 0 < r < world else (n if r == world else 0 * n)
        cut = np.minimum(cut, n)
        if r < world:
            out[r, :, 0] = cut
        if r > 0:
            out[r - 1, :, 1] = cut
    return out


def all_gather_pieces(dist, part_o: torch.Tensor, part_ml: torch.Tensor, group=None):
    """All-gathers every rank's piece: ``part_o [B][Hq][D]``, ``part_ml [B][Hq][2]`` (fp32) ->
    ``([world][B][Hq][D], [world][B][Hq][2])``, rank-major, the layout ``flux_attn_combine`` takes."""
    world = dist.get_world_size(group)
    B = part_o.shape[0]
    # gathered along the first axis (the form every backend takes), then viewed rank-major
    po = torch.empty((world * B,) + tuple(part_o.shape[1:]), dtype=part_o.dtype, device=part_o.device)
    pml = torch.empty((world * B,) + tuple(part_ml.shape[1:]), dtype=part_ml.dtype, device=part_ml.device)
    dist.all_gather_into_tensor(po, part_o.contiguous(), group=group)
    dist.all_gather_into_tensor(pml, part_ml.contiguous(), group=group)
    return po.view((world,) + tuple(part_o.shape)), pml.view((world,) + tuple(part_ml.shape))


def exchange_seq(step: int) -> int:
    """Sequence number of decode step ``step`` (0, 1, 2, ...) for the pushed exchange: never 0 (a cleared flag
    array holds zeros), different for consecutive steps, inside 32 bits."""
    assert step >= 0
    return step % 0xFFFFFFFF + 1


def buffer_set(step: int, layer: int, n_layers: int) -> int:
    """Which gather buffer set (gather_o, gather_ml, flags) the exchange of (step, layer) goes through.  A set may
    be written again only when every rank has merged the previous exchange out of it.  With at least two layers,
    one set per layer is enough: a rank cannot push layer ``l`` of the next step before it has finished this
    step, hence not before every rank has pushed -- and so merged layer ``l`` of -- this step's later layers.
    A single-layer stack alternates two sets."""
    assert 0 <= layer < n_layers
    return layer if n_layers >= 2 else step % 2
