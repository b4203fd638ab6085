"""Block-range-sharded 8-bit Adam step for data-parallel training.

Quantization blocks are independent (Section IV-B: "quantization applied independently to each
block") and the update is element-wise, so the optimizer state of a flat parameter buffer can be
split across the ranks of a data-parallel job on block boundaries with no exchange inside the
step.  Around the step sit the two collectives every sharded optimizer needs:

    reduce-scatter(gradients)  ->  dt8_adam_step on the owned block range  ->  all-gather(parameters)

`torch.distributed` supplies the collectives (NCCL on GPUs); the step itself is the CUDA library.
Each rank keeps the 8-bit states of its own range only: state memory per rank is
(n + 4n/B) * 2 / world_size bytes for Adam.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch
import torch.distributed as dist

import paper_2412_01195_b200 as dt8


def shard_layout(n: int, block_size: int, world_size: int):
    """(blocks per rank, elements per rank, padded length).  Every rank owns the same number of
    whole blocks (the collectives want equal shards); the buffer is padded with zeros up to
    world_size * elements-per-rank."""
    if n < 0 or world_size < 1:
        raise ValueError("n >= 0 and world_size >= 1")
    nb = dt8.num_blocks(n, block_size)
    blocks = (nb + world_size - 1) // world_size
    per_rank = blocks * block_size
    return blocks, per_rank, per_rank * world_size


class ShardedAdam8bit:
    """8-bit AdamW over a flat fp32 parameter buffer replicated on every rank.

    `params` holds the padded parameters (length `padded`), `grads` the local gradients of the
    same length; `step()` averages the gradients over the ranks into this rank's shard, steps the
    shard in place and gathers the updated parameters back into `params` on every rank.
    `step_fn` and `state_fn` exist so that the plumbing can be exercised without a GPU.
    """

    def __init__(self, n: int, block_size: int = 2048, device="cuda", group=None,
                 step_fn: Optional[Callable] = None, state_fn: Optional[Callable] = None):
        self.group = group
        self.rank = dist.get_rank(group) if dist.is_initialized() else 0
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        self.n, self.block_size = n, block_size
        self.blocks, self.per_rank, self.padded = shard_layout(n, block_size, self.world)
        self.params = torch.zeros(self.padded, dtype=torch.float32, device=device)
        self.grads = torch.zeros(self.padded, dtype=torch.float32, device=device)
        self._gshard = torch.empty(self.per_rank, dtype=torch.float32, device=device)
        lo = self.rank * self.per_rank
        self.shard = self.params[lo:lo + self.per_rank]          # a view: stepped in place
        make = state_fn or dt8.new_state
        self.m_codes, self.m_absmax = make(self.per_rank, block_size, True, device)
        self.r_codes, self.r_absmax = make(self.per_rank, block_size, False, device)
        self._step_fn = step_fn or dt8.dt8_adam_step
        self.steps = 0

    def state_bytes(self) -> int:
        """Bytes of optimizer state held by this rank."""
        return 2 * dt8.dt8_state_bytes(self.per_rank, self.block_size)

    def _reduce_scatter_mean(self):
        if self.world == 1:
            self._gshard.copy_(self.grads)
            return
        try:
            dist.reduce_scatter_tensor(self._gshard, self.grads, op=dist.ReduceOp.SUM, group=self.group)
        except (RuntimeError, NotImplementedError):
            # backends without reduce-scatter (gloo on CPU): all-reduce, then keep the own range
            total = self.grads.clone()
            dist.all_reduce(total, op=dist.ReduceOp.SUM, group=self.group)
            lo = self.rank * self.per_rank
            self._gshard.copy_(total[lo:lo + self.per_rank])
        self._gshard.div_(self.world)

    def step(self, lr, beta1, beta2, eps, weight_decay, flags=dt8.DEFAULT_ADAM_FLAGS) -> None:
        self.steps += 1
        self._reduce_scatter_mean()
        self._step_fn(self.shard, self._gshard, self.m_codes, self.m_absmax, self.r_codes,
                      self.r_absmax, lr, beta1, beta2, eps, weight_decay, self.steps,
                      self.block_size, flags)
        if self.world > 1:
            mine = self.shard.clone()
            try:
                dist.all_gather_into_tensor(self.params, mine, group=self.group)
            except (RuntimeError, NotImplementedError):
                parts = [torch.empty_like(mine) for _ in range(self.world)]
                dist.all_gather(parts, mine, group=self.group)
                self.params.copy_(torch.cat(parts))
