"""Block-range-sharded 8-bit Adam step for data-parallel training.

Every quantization block is quantized on its own (Section IV-B, "Tensor chunking") and the update
is element-wise, so the optimizer state of a flat parameter buffer can be split across the ranks
of a data-parallel job on block boundaries with no exchange inside the step.  Around the step sit
the two collectives every sharded optimizer needs:

    reduce-scatter(gradients)  ->  dt8_adam_step on the owned block range  ->  all-gather(parameters)

`torch.distributed` supplies the collectives (NCCL on GPUs); the step itself is the CUDA library.
Each rank keeps the 8-bit states of its own range only: state memory per rank is
(n + 4n/B) * 2 / world_size bytes for Adam.

Which collectives are issued is decided once, from the backend of the process group: NCCL has
reduce-scatter with averaging and all-gather into one tensor; gloo has neither, so there the
gradients are all-reduced and the parameters gathered as a list.  Errors of a collective are
never caught: a rank that took another path than its peers would leave them waiting.
"""
from __future__ import annotations

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
    """

    def __init__(self, n: int, block_size: int = 2048, device="cuda", group=None):
        self.group = group
        ready = dist.is_available() and dist.is_initialized()
        self.rank = dist.get_rank(group) if ready else 0
        self.world = dist.get_world_size(group) if ready else 1
        self.backend = dist.get_backend(group) if ready else "none"
        # tensor collectives (reduce_scatter_tensor with AVG, all_gather_into_tensor) are NCCL's
        self.tensor_collectives = self.backend == "nccl"
        self.n, self.block_size = n, block_size
        self.blocks, self.per_rank, self.padded = shard_layout(n, block_size, self.world)
        self.params = torch.zeros(self.padded, dtype=torch.float32, device=device)
        self.grads = torch.zeros(self.padded, dtype=torch.float32, device=device)
        self._gshard = torch.empty(self.per_rank, dtype=torch.float32, device=device)
        lo = self.rank * self.per_rank
        self.shard = self.params[lo:lo + self.per_rank]          # a view: stepped in place
        self.m_codes, self.m_absmax = self._new_state(True, device)
        self.r_codes, self.r_absmax = self._new_state(False, device)
        self.steps = 0

    def _new_state(self, signed: bool, device):
        return dt8.new_state(self.per_rank, self.block_size, signed, device)

    def _step_shard(self, lr, beta1, beta2, eps, weight_decay, flags) -> None:
        dt8.dt8_adam_step(self.shard, self._gshard, self.m_codes, self.m_absmax, self.r_codes,
                          self.r_absmax, lr, beta1, beta2, eps, weight_decay, self.steps,
                          self.block_size, flags)

    def state_bytes(self) -> int:
        """Bytes of optimizer state held by this rank."""
        return 2 * dt8.dt8_state_bytes(self.per_rank, self.block_size)

    def _reduce_scatter_mean(self) -> None:
        if self.world == 1:
            self._gshard.copy_(self.grads)
        elif self.tensor_collectives:
            dist.reduce_scatter_tensor(self._gshard, self.grads, op=dist.ReduceOp.AVG, group=self.group)
        else:
            dist.all_reduce(self.grads, op=dist.ReduceOp.SUM, group=self.group)
            lo = self.rank * self.per_rank
            torch.div(self.grads[lo:lo + self.per_rank], self.world, out=self._gshard)

    def _all_gather_params(self) -> None:
        if self.world == 1:
            return
        if self.tensor_collectives:
            # in place: this rank's shard already sits at its position of the output
            dist.all_gather_into_tensor(self.params, self.shard, group=self.group)
        else:
            parts = list(self.params.split(self.per_rank))
            dist.all_gather(parts, self.shard.clone(), group=self.group)

    def step(self, lr, beta1, beta2, eps, weight_decay, flags=dt8.DEFAULT_ADAM_FLAGS) -> None:
        self.steps += 1
        self._reduce_scatter_mean()
        self._step_shard(lr, beta1, beta2, eps, weight_decay, flags)
        self._all_gather_params()
