"""Sequence-sharded forward over several devices, one process per device: rank r holds a run of
consecutive tokens of every sequence.  The library computes a shard's summary (end state from a
zero entry state, total decay) and, once all ranks' summaries are known, the shard's outputs; the
one exchange between the two is an all-gather of [B, H, P, N] + [B, H] floats per rank, done here
with torch.distributed (NCCL on GPUs, gloo in the CPU tests).  Argument marshalling and the
collective only: every arithmetic step runs in the library's kernels.
"""
from __future__ import annotations

from typing import Optional

import torch


def gather_summaries(state: torch.Tensor, decay: torch.Tensor, dist=None, group=None):
    """All ranks' (state [B,H,P,N], decay [B,H]) stacked in rank order: ([R,B,H,P,N], [R,B,H]).
    Without a process group the single rank's own summary with a leading axis of 1."""
    if dist is None:
        return state.unsqueeze(0).contiguous(), decay.unsqueeze(0).contiguous()
    world = dist.get_world_size(group)
    all_state = torch.empty((world,) + tuple(state.shape), dtype=state.dtype, device=state.device)
    all_decay = torch.empty((world,) + tuple(decay.shape), dtype=decay.dtype, device=decay.device)
    dist.all_gather(list(all_state.unbind(0)), state.contiguous(), group=group)
    dist.all_gather(list(all_decay.unbind(0)), decay.contiguous(), group=group)
    return all_state, all_decay


def sequence_sharded_forward(sb, h, w, u, x, dt, h0: Optional[torch.Tensor], B: int, L: int, y, h_end,
                             workspace, dist=None, group=None, topk_idx=None, topk_w=None, stream=None):
    """One rank's part of the sharded forward.  sb: the binding module (swimba_shard_summary /
    swimba_shard_finish); u [B,L,F], x [B,L,H,P], dt [B,L,H]: this rank's tokens; h0: the state in
    front of rank 0's tokens (the same tensor values on every rank, or None); y [B,L,H,P] and h_end
    [B,H,P,N] (may be None) are written.  Returns (all_state, all_decay) as gathered."""
    rank = 0 if dist is None else dist.get_rank(group)
    world = 1 if dist is None else dist.get_world_size(group)
    H, P = x.shape[-2], x.shape[-1]
    N = h.cfg.d_state
    state = torch.empty(B, H, P, N, dtype=torch.float32, device=x.device)
    decay = torch.empty(B, H, dtype=torch.float32, device=x.device)
    sb.swimba_shard_summary(h, w, u, x, dt, B, L, state, decay, topk_idx, topk_w, workspace, stream=stream)
    if dist is not None and stream is not None:
        # the collective is ordered behind torch's current stream only; a caller's own stream is joined here
        stream.synchronize()
    all_state, all_decay = gather_summaries(state, decay, dist, group)
    sb.swimba_shard_finish(h, w, x, h0, all_state, all_decay, rank, world, B, L, y, h_end, workspace,
                           stream=stream)
    return all_state, all_decay
