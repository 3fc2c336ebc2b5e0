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


# ---- the tensor-parallel form of the norm: host logic of the group on CPU --------------------------------------

def _tp_worker(rank: int, world: int, port: int, shared: dict, out_dir: str):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch.distributed as dist
    from paper_2601_12698_b200 import dp
    import oracle
    device = torch.device("cpu")
    assert dp.init(backend="gloo", device=device) is True
    n_rows, hidden = shared["r"].shape
    calls = []

    # Stand-in for the CUDA entry point with the same signature: the oracle on the requested rows, written to every
    # destination.  Shared-memory tensors stand in for peer-mapped GPU memory.
    met_on = []  # the stream each meeting of the group was issued on

    def sync(stream):
        met_on.append(stream)
        dist.barrier()

    def launch(theta, x_parts, r, w, y_outs, r_outs, row_begin, row_count, eps, stream):
        # the launch sits between two meetings and on the very stream the first one was issued on
        assert len(met_on) % 2 == 1 and stream is met_on[-1]
        calls.append((tuple(theta), row_begin, row_count, len(x_parts), len(y_outs), len(r_outs)))
        rows = slice(row_begin, row_begin + row_count)
        stacked = torch.stack([p[rows] for p in x_parts]).contiguous()
        y, ro = oracle.allreduce_add_rmsnorm(stacked, r[rows].contiguous(), w, eps)
        for dst in y_outs:
            dst[rows] = y
        for dst in r_outs:
            dst[rows] = ro

    # every rank fills its own partial, then the group runs the fused operator
    g = torch.Generator().manual_seed(100 + rank)
    shared["x"][rank].copy_(torch.randn(n_rows, hidden, generator=g).to(torch.bfloat16))
    ranks_seen = dp.gather_in_rank_order(("rank", rank))
    assert ranks_seen == [("rank", k) for k in range(world)]
    op = dp.FusedAllreduceNorm(rank, world, n_rows, list(shared["x"]), list(shared["y"]), list(shared["r_out"]), launch,
                               sync=sync)
    side_stream = object()  # stands for a CUDA stream that is not the current one
    sh = op((256, 1, 16, 1, 0, 0, 1), shared["r"], shared["w"], 1e-6, stream=side_stream)
    assert met_on == [side_stream, side_stream]                             # both meetings on the launch stream
    assert (sh.row_begin, sh.row_end) == ((0, 19), (19, 37))[rank]          # 37 rows over two ranks: 19 + 18
    assert calls == [((256, 1, 16, 1, 0, 0, 1), sh.row_begin, sh.rows, world, world, 1)]
    # after the second meeting this rank's y holds every row, its r_out the rows of its own block
    torch.save({"y": shared["y"][rank].clone(), "ro": shared["r_out"][rank].clone(), "rows": (sh.row_begin, sh.row_end)},
               os.path.join(out_dir, f"tp{rank}.pt"))
    # the same again with the residual sent to every rank
    dp.barrier(device)
    op.gather_residual = True
    op((256, 1, 16, 1, 0, 0, 1), shared["r"], shared["w"], 1e-6)
    assert calls[-1][-1] == world and met_on[2:] == [None, None]
    torch.save({"ro_all": shared["r_out"][rank].clone()}, os.path.join(out_dir, f"tpg{rank}.pt"))
    # the default meeting (a one-element all-reduce of the process group) in place of the test's barrier
    dp.barrier(device)
    met_on.append(None)  # keep the launch's "between two meetings" check in step
    op.sync = None
    op((256, 1, 16, 1, 0, 0, 1), shared["r"], shared["w"], 1e-6)
    assert int(op._flag.item()) == 0 and len(calls) == 3
    dp.barrier(device)
    dp.shutdown()


def test_two_gloo_ranks_tensor_parallel_norm(tmp_path):
    sys.path.insert(0, ROOT)
    import oracle
    world, n_rows, hidden = 2, 37, 64
    g = torch.Generator().manual_seed(9)
    shared = {
        "x": [torch.zeros(n_rows, hidden, dtype=torch.bfloat16).share_memory_() for _ in range(world)],
        "y": [torch.zeros(n_rows, hidden, dtype=torch.bfloat16).share_memory_() for _ in range(world)],
        "r_out": [torch.zeros(n_rows, hidden, dtype=torch.bfloat16).share_memory_() for _ in range(world)],
        "r": torch.randn(n_rows, hidden, generator=g).to(torch.bfloat16).share_memory_(),
        "w": (1 + 0.1 * torch.randn(hidden, generator=g)).to(torch.bfloat16).share_memory_(),
    }
    mp.spawn(_tp_worker, args=(world, _free_port(), shared, str(tmp_path)), nprocs=world, join=True)
    got = [torch.load(os.path.join(tmp_path, f"tp{k}.pt")) for k in range(world)]
    y_ref, r_ref = oracle.allreduce_add_rmsnorm(torch.stack(shared["x"]).contiguous(), shared["r"], shared["w"], 1e-6)
    for k in range(world):
        assert torch.equal(got[k]["y"].view(torch.int16), y_ref.view(torch.int16))
        lo, hi = got[k]["rows"]
        assert torch.equal(got[k]["ro"][lo:hi].view(torch.int16), r_ref[lo:hi].view(torch.int16))
        outside = torch.cat([got[k]["ro"][:lo], got[k]["ro"][hi:]])
        assert bool((outside == 0).all())                                   # another rank's rows were not sent here
        gathered = torch.load(os.path.join(tmp_path, f"tpg{k}.pt"))["ro_all"]
        assert torch.equal(gathered.view(torch.int16), r_ref.view(torch.int16))


def test_fused_allreduce_norm_argument_checks():
    sys.path.insert(0, ROOT)
    from paper_2601_12698_b200 import dp
    t = [torch.zeros(4, 8)] * 2
    with pytest.raises(ValueError):
        dp.FusedAllreduceNorm(0, 3, 4, t + t[:1], t + t[:1], t + t[:1], None)     # a group of three
    with pytest.raises(ValueError):
        dp.FusedAllreduceNorm(0, 2, 4, t, t[:1], t, None)                           # a destination missing
    with pytest.raises(ValueError):
        dp.FusedAllreduceNorm(2, 2, 4, t, t, t, None)                               # rank outside the group
    assert dp.gather_in_rank_order("alone") == ["alone"]
    # the blocks of rows tile the job for every group size
    for world in (2, 4, 8):
        for n_rows in (1, 7, 64, 1001):
            blocks = [dp.FusedAllreduceNorm(k, world, n_rows, [None] * world, [None] * world, [None] * world, None).shard
                      for k in range(world)]
            assert blocks[0].row_begin == 0 and blocks[-1].row_end == n_rows
            assert all(a.row_end == b.row_begin for a, b in zip(blocks, blocks[1:]))
