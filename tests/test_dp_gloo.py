"""The N > 1 path on CPU: two gloo ranks exercise sharding, the max-over-ranks timing rule, the theta
broadcast and the whole-job rate, and check that shards of the generator tile the job without overlap."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2601_12698_b200 import dp, synth
    import oracle
    device = torch.device("cpu")
    assert dp.env_world() == (rank, world, rank)
    assert dp.init(backend="gloo", device=device) is True
    shard = dp.weak_shard(96, rank, world)
    assert (shard.row_begin, shard.row_end, shard.rows) == (rank * 96, (rank + 1) * 96, 96)
    # this rank's rows of the (world * 96)-row job, and its own oracle pass: no data crosses ranks
    x = synth.make_rows(synth.TENSOR_X, shard.row_begin, shard.row_end, 256, "bf16", seed=5).contiguous()
    r = synth.make_rows(synth.TENSOR_R, shard.row_begin, shard.row_end, 256, "bf16", seed=5).contiguous()
    w = synth.make_weight(256, "bf16", seed=5)
    y, ro = oracle.add_rmsnorm(x, r, w, 1e-6)
    torch.save({"x": x, "y": y, "ro": ro}, os.path.join(out_dir, f"rank{rank}.pt"))
    dp.barrier(device)
    # the slowest rank sets the time; the rate counts every rank's units
    ms = dp.max_over_ranks(10.0 + 5.0 * rank, device)
    assert ms == 10.0 + 5.0 * (world - 1)
    assert dp.sum_over_ranks(1.0, device) == float(world)
    rate = dp.whole_job_rate(units_per_rank_per_step=1000.0, steps=4, world=world, max_ms=ms)
    assert abs(rate - 1000.0 * 4 * world / (ms * 1e-3)) < 1e-6
    # rank 0 chooses theta, everyone launches the same one
    theta = [256, 1, 16, 1, 2, 0, 1] if rank == 0 else [0] * 7
    assert dp.broadcast_ints(theta, device) == [256, 1, 16, 1, 2, 0, 1]
    dp.barrier(device)
    dp.shutdown()


def test_two_gloo_ranks(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    sys.path.insert(0, ROOT)
    from paper_2601_12698_b200 import synth
    import oracle
    parts = [torch.load(os.path.join(tmp_path, f"rank{k}.pt")) for k in range(2)]
    # the two shards are the two halves of one 192-row job, and sharding does not change any row's result
    x_all = synth.make_rows(synth.TENSOR_X, 0, 192, 256, "bf16", seed=5).contiguous()
    r_all = synth.make_rows(synth.TENSOR_R, 0, 192, 256, "bf16", seed=5).contiguous()
    assert torch.equal(torch.cat([p["x"] for p in parts]), x_all)
    y_all, ro_all = oracle.add_rmsnorm(x_all, r_all, synth.make_weight(256, "bf16", seed=5), 1e-6)
    assert torch.equal(torch.cat([p["y"] for p in parts]), y_all)
    assert torch.equal(torch.cat([p["ro"] for p in parts]), ro_all)


def test_shard_arithmetic():
    from paper_2601_12698_b200 import dp
    for total, world in ((16384, 8), (10, 4), (3, 8), (0, 2)):
        shards = [dp.strong_shard(total, k, world) for k in range(world)]
        assert shards[0].row_begin == 0 and shards[-1].row_end == total
        assert all(a.row_end == b.row_begin for a, b in zip(shards, shards[1:]))
        assert max(s.rows for s in shards) - min(s.rows for s in shards) <= 1
    with pytest.raises(ValueError):
        dp.weak_shard(4, 2, 2)
    assert dp.env_world() == (0, 1, 0) or "RANK" in os.environ
    # single process: the helpers are the identity
    cpu = torch.device("cpu")
    assert dp.max_over_ranks(3.5, cpu) == 3.5 and dp.broadcast_ints([1, 2], cpu) == [1, 2]
