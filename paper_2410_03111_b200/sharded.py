"""Decode attention over ONE context that is sharded across GPUs by position.

The method itself shards by sequence and needs no exchange.  A single context too long (or too hot) for one GPU is the
case with a real exchange step: rank r keeps the latent rows of positions [pos0_r, pos0_r + len_r) of every sequence,
attends to them alone (lorc_decode_attn_shard), and the ranks all-gather d_head + 2 numbers per (sequence, head) and
merge (lorc_merge_shards): the shard softmaxes weighted by their denominators are the softmax over the whole context.

One process per GPU; `group` is a torch.distributed process group (NCCL over NVLink on GPUs).  Every step of the
arithmetic runs in the library's kernels; this module only plans the split and moves the small results.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as _L


def shard_bounds(seq_lens, world_size: int, quantum: int = 128):
    """Split positions [0, len) of every sequence into world_size contiguous ranges.

    The cut points are multiples of `quantum` tokens (the score kernel's tile, so that no tile straddles two ranks)
    and the ranges differ by at most one quantum; ranks at the end may get nothing.  Returns two int lists
    [world_size][batch]: first position and token count of each rank's range."""
    pos0 = [[0] * len(seq_lens) for _ in range(world_size)]
    cnt = [[0] * len(seq_lens) for _ in range(world_size)]
    for s, n in enumerate(seq_lens):
        n = int(n)
        q_total = (n + quantum - 1) // quantum
        base, extra = divmod(q_total, world_size)
        start = 0
        for r in range(world_size):
            take = (base + (1 if r < extra else 0)) * quantum
            end = min(n, start + take)
            pos0[r][s] = start
            cnt[r][s] = end - start
            start = end
    return pos0, cnt


def append_owner(seq_lens, world_size: int, quantum: int = 128):
    """Which rank the NEXT token of each sequence is appended on, under the rule of shard_bounds applied after the
    append: the rank whose range ends at the new length.  Growing a context one token at a time under that rule moves
    cut points; a server that wants rows to stay where they were written instead keeps fixed cut points and lets the
    last non-empty rank grow, which shard_bounds' callers may do by passing their own ranges to ShardedDecoder."""
    owners = []
    for n in seq_lens:
        p0, cnt = shard_bounds([int(n) + 1], world_size, quantum)
        owners.append(max(r for r in range(world_size) if cnt[r][0] > 0))
    return owners


class ShardedDecoder:
    """Decode attention of one layer over position-sharded caches.

    attend / merge default to the library's entry points; they are parameters so that the exchange logic can be run
    on CPU ranks with stand-ins for the two kernels."""

    def __init__(self, ctx, n_q_heads: int, d_head: int, group=None, attend=None, merge=None):
        self.ctx, self.H_q, self.d_h, self.group = ctx, n_q_heads, d_head, group
        self.attend = attend or _L.lorc_decode_attn_shard
        self.merge = merge or _L.lorc_merge_shards
        self.world = dist.get_world_size(group)
        self._buf = {}

    def _buffers(self, batch, device):
        key = (batch, str(device))
        if key not in self._buf:
            W = self.world
            self._buf[key] = (
                torch.empty(batch, self.H_q, self.d_h, dtype=torch.bfloat16, device=device),
                torch.empty(batch, self.H_q, 2, dtype=torch.float32, device=device),
                torch.empty(W, batch, self.H_q, self.d_h, dtype=torch.bfloat16, device=device),
                torch.empty(W, batch, self.H_q, 2, dtype=torch.float32, device=device),
            )
        return self._buf[key]

    def decode(self, layer, cache, q, pos0, q_pos, out, n_splits=0, stream=None):
        """cache: this rank's shard (seq_lens = rows held here); pos0, q_pos: int32 [batch] tensors on q's device;
        out [batch, H_q, d_head] bf16 receives the attention over the whole context on every rank."""
        batch = q.shape[0]
        o_r, ml_r, o_all, ml_all = self._buffers(batch, q.device)
        self.attend(self.ctx, layer, cache, q, pos0, q_pos, o_r, ml_r, n_splits, stream)
        # flat views: the concatenation along the first axis is what every backend agrees on
        dist.all_gather_into_tensor(o_all.view(-1), o_r.view(-1), group=self.group)
        dist.all_gather_into_tensor(ml_all.view(-1), ml_r.view(-1), group=self.group)
        self.merge(self.ctx, self.world, o_all, ml_all, out, batch, stream)
        return out
