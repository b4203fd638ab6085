"""The multi-GPU path on CPU: world size 2 over gloo.

The step shards on quantization-block boundaries with no exchange between ranks (Section IV-B:
every block is quantized on its own).  These tests run the host-side logic of that path as two
gloo ranks: the block partition, the timing reduction the benchmark uses (barrier + maximum over
ranks), and the sharded optimizer's plumbing (reduce-scatter -> step on the owned block range ->
all-gather), whose result must equal the unsharded step on the mean gradient bit for bit.  There
is no GPU here, so the step on the shard is the CPU checker, put in by subclassing."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORLD = 2
B = 256
N = 37 * B + 91            # 38 blocks, the last one short
HP = (1e-3, 0.9, 0.999, 1e-8, 0.01)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs():
    from paper_2412_01195_b200 import synth
    w, g = synth.flat_adam_inputs(N, 11)
    return w.numpy().copy(), g.numpy().copy()


def _worker(rank: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(WORLD), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        import bench
        import oracle
        import paper_2412_01195_b200 as dt8

        nb = dt8.num_blocks(N, B)
        mine = dt8.shard_blocks(nb, rank, WORLD)
        # 1. the partition: every block owned exactly once, ranges contiguous and ordered
        owned = [None] * WORLD
        dist.all_gather_object(owned, (mine.start, mine.stop))
        assert owned[0][0] == 0 and owned[-1][1] == nb
        assert all(owned[i][1] == owned[i + 1][0] for i in range(WORLD - 1))

        # 2. the benchmark's timing reduction: barrier, then the maximum over ranks
        bench.barrier()
        slowest = bench.max_over_ranks(10.0 * (rank + 1), torch.device("cpu"))
        assert slowest == 10.0 * WORLD
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as fh:
            fh.write("ok")
    finally:
        dist.destroy_process_group()


def _cpu_sharded_class():
    """ShardedAdam8bit with the step on the shard done by the CPU checker (no GPU in this test)."""
    import oracle
    from paper_2412_01195_b200.sharded import ShardedAdam8bit

    class CpuSharded(ShardedAdam8bit):
        def _step_shard(self, lr, beta1, beta2, eps, weight_decay, flags):
            oracle.adam_step(self.shard.numpy(), self._gshard.numpy(), self.m_codes.numpy(),
                             self.m_absmax.numpy(), self.r_codes.numpy(), self.r_absmax.numpy(), lr,
                             beta1, beta2, eps, weight_decay, self.steps, self.block_size, flags)
    return CpuSharded


def _sharded_worker(rank: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(WORLD), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=WORLD)
    try:
        import oracle
        from paper_2412_01195_b200 import synth
        from paper_2412_01195_b200.sharded import shard_layout

        blocks, per_rank, padded = shard_layout(N, B, WORLD)
        assert per_rank == blocks * B and padded == WORLD * per_rank >= N
        opt = _cpu_sharded_class()(N, B, device="cpu")
        assert opt.backend == "gloo" and not opt.tensor_collectives      # the path is chosen once, by backend
        w0 = synth.normal(N, 0.02, 21)
        opt.params[:N].copy_(w0)
        # reference: the unsharded step on the gradient averaged over the ranks
        w_ref = np.zeros(padded, np.float32)
        w_ref[:N] = w0.numpy()
        nb = oracle.num_blocks(padded, B)
        mc, ma = np.full(padded, 127, np.uint8), np.zeros(nb, np.float32)
        rc, ra = np.zeros(padded, np.uint8), np.zeros(nb, np.float32)
        for t in (1, 2, 3):
            local = [synth.normal(N, 1e-3, 100 * t + r) for r in range(WORLD)]
            opt.grads.zero_()
            opt.grads[:N].copy_(local[rank])
            opt.step(*HP)
            mean = np.zeros(padded, np.float32)
            mean[:N] = ((local[0] + local[1]) / WORLD).numpy()
            oracle.adam_step(w_ref, mean, mc, ma, rc, ra, *HP, t, B)
        assert np.array_equal(opt.params.numpy(), w_ref), "gathered parameters differ"
        lo = rank * per_rank
        assert np.array_equal(opt.m_codes.numpy(), mc[lo:lo + per_rank])
        assert np.array_equal(opt.r_absmax.numpy(), ra[lo // B:(lo + per_rank) // B])
        assert opt.state_bytes() == 2 * (per_rank + 4 * blocks)
        # the shard is the block range shard_blocks() names when the blocks divide evenly
        import paper_2412_01195_b200 as dt8
        mine = dt8.shard_blocks(padded // B, rank, WORLD)
        assert (mine.start, mine.stop) == (rank * blocks, (rank + 1) * blocks)

        # a failing collective is not swallowed: it reaches the caller on every rank
        import torch.distributed as dist_mod
        real = dist_mod.all_reduce

        def broken(*a, **k):
            raise RuntimeError("collective failed")
        dist_mod.all_reduce = broken
        try:
            with pytest.raises(RuntimeError, match="collective failed"):
                opt.step(*HP)
        finally:
            dist_mod.all_reduce = real
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as fh:
            fh.write("ok")
    finally:
        dist.destroy_process_group()


def test_sharded_adam_reduce_scatter_step_all_gather(tmp_path):
    """reduce-scatter(grads) -> step on the owned blocks -> all-gather(params), two gloo ranks,
    with the CPU checker standing in for the CUDA step: equals the unsharded step on the mean
    gradient bit for bit."""
    mp.spawn(_sharded_worker, args=(_free_port(), str(tmp_path)), nprocs=WORLD, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(WORLD))


def test_two_ranks_shard_blocks_and_agree_with_the_unsharded_step(tmp_path):
    mp.spawn(_worker, args=(_free_port(), str(tmp_path)), nprocs=WORLD, join=True)
    assert all(os.path.exists(tmp_path / f"ok{r}") for r in range(WORLD))


def test_reference_arm_runs_on_rank_zero_only(monkeypatch, capsys):
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")

    class Args:
        steps, warmup = 1, 1
    assert bench.run_reference(Args()) is None
    assert capsys.readouterr().out == ""
