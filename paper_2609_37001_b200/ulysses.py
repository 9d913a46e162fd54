"""Head-sharded attention for sequence-sharded activations (the DeepSpeed-Ulysses pattern the paper
uses to spread PSA-Search over GPUs, Section 3.3).

Every rank holds ALL heads for a contiguous chunk of L / P tokens (token order t*H*W + h*W + w).
Attention needs all tokens of a head, and heads are independent, so one all-to-all turns the layout
into "H / P heads, all L tokens" per rank, the single-GPU stripe attention runs on those heads with
their own masks, and a second all-to-all returns the outputs to the sequence-sharded layout.

This module is host-side plumbing around ``binding.psa_attn_fwd``: two ``all_to_all_single`` calls per
tensor on the process group's backend (NCCL over NVLink on GPUs; gloo in the CPU tests).  The
exchanges are not fused with the attention kernel.  L and the head count must be divisible by the
group size.
"""
from __future__ import annotations

from typing import Callable, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


def _group_size(group) -> int:
    return dist.get_world_size(group) if dist.is_initialized() else 1


def seq_to_head_shards(x: torch.Tensor, group=None) -> torch.Tensor:
    """[heads, L/P, d] on every rank (rank r holds token chunk r) -> [heads/P, L, d] (rank r holds head
    chunk r, tokens in global order)."""
    P = _group_size(group)
    if P == 1:
        return x
    nh, lc, d = x.shape
    if nh % P:
        raise ValueError("head count must be divisible by the group size")
    # chunk p of the send buffer = the heads that rank p will own
    send = x.reshape(P, nh // P, lc, d).contiguous()
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    # chunk p of the receive buffer = token chunk p of my heads
    return recv.permute(1, 0, 2, 3).reshape(nh // P, P * lc, d).contiguous()


def head_to_seq_shards(y: torch.Tensor, group=None) -> torch.Tensor:
    """Inverse of seq_to_head_shards: [heads/P, L, d] -> [heads, L/P, d]."""
    P = _group_size(group)
    if P == 1:
        return y
    nhl, L, d = y.shape
    if L % P:
        raise ValueError("token count must be divisible by the group size")
    send = y.reshape(nhl, P, L // P, d).permute(1, 0, 2, 3).contiguous()   # chunk p = token chunk p
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    return recv.reshape(P * nhl, L // P, d)                                # chunk p = head chunk p


def local_heads(n_heads: int, group=None) -> Tuple[int, int]:
    """Head range [lo, hi) this rank owns after seq_to_head_shards."""
    P = _group_size(group)
    r = dist.get_rank(group) if P > 1 else 0
    return r * (n_heads // P), (r + 1) * (n_heads // P)


def psa_attn_fwd_ulysses(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, head_params: Sequence[Sequence[int]],
                         grid: Sequence[int], tile: Sequence[int], scale: float, group=None,
                         attn_fn: Optional[Callable] = None):
    """Stripe attention on sequence-sharded inputs.  q, k, v: [heads, L/P, 128] (this rank's token
    chunk of every head); ``head_params`` lists the masks of ALL heads.  Returns (out [heads, L/P, 128],
    lse [heads, L/P]) in the same sequence-sharded layout.

    ``attn_fn(q, k, v, params, grid, tile, scale) -> (out, lse)`` defaults to ``binding.psa_attn_fwd``;
    the CPU tests pass their own."""
    if attn_fn is None:
        from . import binding
        attn_fn = binding.psa_attn_fwd
    nh = q.shape[0]
    if len(head_params) != nh:
        raise ValueError("one parameter set per head")
    P = _group_size(group)
    T, H, W = (int(x) for x in grid)
    if q.shape[1] * P != T * H * W:
        raise ValueError("local token count times group size must equal T*H*W")
    qh, kh, vh = (seq_to_head_shards(t, group) for t in (q, k, v))
    lo, hi = local_heads(nh, group)
    out_h, lse_h = attn_fn(qh, kh, vh, [tuple(p) for p in head_params[lo:hi]], grid, tile, scale)
    out = head_to_seq_shards(out_h, group)
    lse = head_to_seq_shards(lse_h.unsqueeze(-1).contiguous(), group).squeeze(-1)
    return out, lse
