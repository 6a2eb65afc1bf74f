"""Vocabulary-parallel verification: every rank holds rows [offset, offset+V_local) of the LM head
(the tensor-parallel deployment of the paper's experiments, Sec. 4.1).

Per call each rank runs the masked head on its shard (the masks depend on indices only, so all
ranks draw the same ones without talking), the ranks all-gather one packed 64-bit word per path
(8 * B*T*K bytes per rank: a few KB over NVLink), and every rank finishes with the histogram and
the acceptance scan on the gathered words.  The collective is `torch.distributed`'s all-gather
(NCCL on GPU tensors; any backend that takes the tensors it is given works, e.g. gloo on CPU
copies).  No kernel of this library waits on another rank.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding


class VocabParallelVerifier:
    def __init__(self, ctx, W_shard: torch.Tensor, vocab_offset: int, max_rows: int, group=None,
                 gather_on_cpu: bool = False):
        """ctx: a binding.Context on this rank's device; W_shard: this rank's rows of the head."""
        self.ctx, self.group, self.gather_on_cpu = ctx, group, gather_on_cpu
        ctx.set_head(W_shard, max_rows=max_rows)
        ctx.set_vocab_offset(vocab_offset)

    def verify_batched(self, H, draft, K, p, seed, seq_base=0, rule=binding.RULE_NAIVE):
        world = dist.get_world_size(self.group) if dist.is_initialized() else 1
        mine = self.ctx.partial_best(H, K, p, seed, seq_base)
        if world == 1:
            return self.ctx.finalize_packed(mine, draft, K, rule)
        if self.gather_on_cpu:      # backends without GPU support (tests): gather host copies
            parts = [torch.empty(mine.shape, dtype=mine.dtype) for _ in range(world)]
            dist.all_gather(parts, mine.cpu(), group=self.group)
            gathered = torch.stack(parts).to(mine.device)
        else:
            gathered = torch.empty((world, mine.numel()), dtype=mine.dtype, device=mine.device)
            dist.all_gather_into_tensor(gathered, mine, group=self.group)
        return self.ctx.finalize_packed(gathered, draft, K, rule)


def shard_rows(V: int, world: int, rank: int, multiple: int = 8) -> tuple[int, int]:
    """Rows [begin, end) of the head that rank `rank` of `world` holds: equal shares rounded up to a
    multiple of `multiple` rows, the last rank taking what is left."""
    per = -(-V // world)
    per = -(-per // multiple) * multiple
    begin = min(V, rank * per)
    return begin, min(V, begin + per)
