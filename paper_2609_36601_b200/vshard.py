"""Vocabulary-sharded routing: the exchange around the library's stage calls.

Every rank holds a contiguous column slice of the logit rows (as a tensor-parallel lm-head leaves them).  A
row is routed in four stages; per stage a rank reduces its slice to 16 float64 numbers per row
(`vshard_partial`, a kernel), the ranks all-gather those (128 bytes per row, rank and stage; NCCL over NVLink on
GPUs, no logits ever cross), and every rank folds the gathered partials in rank order into the same per-row
state (`vshard_combine`, a kernel).  Stage 1 (one evaluation of the trust-region constraint) repeats until no
row is still solving: two waves as a rule (each moves to the root of a fourth-order model of the constraint).  This module holds no arithmetic: it
sequences the stages, moves the partials, and reads one counter per wave.

`route_vocab_sharded` is the one-rank-per-process form over `torch.distributed`; `route_vocab_sharded_local`
runs the ranks one after the other in a single process on one device (the slices of all ranks are at hand):
the same calls in the same order, with a copy in place of the all-gather.
"""
from __future__ import annotations

import torch

from . import binding as B

MAX_WAVES = 128


def split_columns(V: int, world: int):
    """Contiguous, balanced column ranges: [(v0, V_local)] per rank, in rank order, tiling [0, V)."""
    base, extra = divmod(V, world)
    out, v0 = [], 0
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append((v0, n))
        v0 += n
    return out


def route_vocab_sharded(s_loc, t_loc, v0: int, V: int, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None,
                        grad_scale=1.0, backward=True, group=None, stream=None):
    """One rank's call: `s_loc`, `t_loc` are this rank's columns [v0, v0 + V_local) on its GPU.  Returns (out,
    dlogits_slice): the per-position outputs (identical on every rank) and this rank's columns of the gradient."""
    import torch.distributed as dist
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    dev, N = s_loc.device, s_loc.shape[0]
    si = B.vshard_in(s_loc, t_loc, v0, V, proposal, eps, temperature, seed, row_offset, mask, rank, world)
    state = torch.empty((N, B.VSHARD_STATE), dtype=torch.float64, device=dev)
    part = torch.empty((N, B.VSHARD_PARTIALS), dtype=torch.float64, device=dev)
    gathered = torch.empty((world, N, B.VSHARD_PARTIALS), dtype=torch.float64, device=dev)
    n_solving = torch.zeros(1, dtype=torch.int32, device=dev)
    out = B.alloc_outputs(N, dev)
    g = torch.empty_like(s_loc) if backward else None

    def wave(stage, with_state=True):
        B.vshard_partial(si, stage, state if with_state else None, part, g if stage == 3 else None, grad_scale, stream)
        dist.all_gather_into_tensor(gathered.view(-1), part.view(-1), group=group)
        B.vshard_combine(si, stage, gathered, state, out if stage == 3 else None, n_solving, stream)

    wave(0, with_state=False)
    waves = 0
    while int(n_solving.item()) > 0 and waves < MAX_WAVES:
        wave(1)
        waves += 1
    wave(2)
    wave(3)
    return out, g


def route_vocab_sharded_local(slices, V: int, proposal, eps, temperature=1.0, seed=0, row_offset=0, mask=None,
                              grad_scale=1.0, backward=True, stream=None, state_out=None):
    """All ranks in one process: `slices` = [(s_loc, t_loc, v0)] in rank order on one device.  Returns (out,
    [dlogits_slice per rank], waves): the calls every rank would make, one rank after the other.  `state_out`: a
    list that receives the per-row state tensor (for tests)."""
    world = len(slices)
    dev, N = slices[0][0].device, slices[0][0].shape[0]
    sis = [B.vshard_in(s, t, v0, V, proposal, eps, temperature, seed, row_offset, mask, r, world)
           for r, (s, t, v0) in enumerate(slices)]
    state = torch.empty((N, B.VSHARD_STATE), dtype=torch.float64, device=dev)
    gathered = torch.empty((world, N, B.VSHARD_PARTIALS), dtype=torch.float64, device=dev)
    n_solving = torch.zeros(1, dtype=torch.int32, device=dev)
    out = B.alloc_outputs(N, dev)
    gs = [torch.empty_like(s) if backward else None for s, _, _ in slices]

    def wave(stage, with_state=True):
        for r in range(world):            # rank r's partial lands where the all-gather would put it
            B.vshard_partial(sis[r], stage, state if with_state else None, gathered[r], gs[r] if stage == 3 else None,
                             grad_scale, stream)
        B.vshard_combine(sis[0], stage, gathered, state, out if stage == 3 else None, n_solving, stream)

    wave(0, with_state=False)
    waves = 0
    while int(n_solving.item()) > 0 and waves < MAX_WAVES:
        wave(1)
        waves += 1
    wave(2)
    wave(3)
    if state_out is not None:
        state_out.append(state)
    return out, gs, waves
