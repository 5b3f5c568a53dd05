"""The N > 1 path on CPU: two gloo ranks shard a batch, each verifies its block (the oracle stands in
for the device here), and the gathered result equals the unsharded one."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2606_12370_b200.shard import max_over_ranks, shard_range


def test_shard_range_covers_in_order():
    for batch in (0, 1, 5, 64, 1023):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                b, e = shard_range(batch, r, world)
                assert b == prev and e >= b
                prev = e
            assert prev == batch
            sizes = [shard_range(batch, r, world)[1] - shard_range(batch, r, world)[0] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_shard_range_balances_rows():
    rng = np.random.default_rng(0)
    lens = rng.integers(1, 5, size=1024)
    w = 2 * lens + 1
    for world in (2, 4, 8):
        loads, prev = [], 0
        for r in range(world):
            b, e = shard_range(1024, r, world, lens)
            assert b == prev
            prev = e
            loads.append(int(w[b:e].sum()))
        assert prev == 1024
        assert max(loads) - min(loads) <= 2 * int(w.max())
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)
    with pytest.raises(ValueError):
        shard_range(4, 0, 2, [1, 2, 3])


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bebop_gen as G
        import oracle
        cfg = G.get_config("tiny", B=6)
        x = G.make_inputs(cfg, "cpu")
        lens = [3, 1, 2, 3, 0, 2]
        b, e = shard_range(cfg.B, rank, world, lens)
        sl = slice(b, e)
        res = oracle.verify(x["target"][sl].numpy(), x["draft"][sl].numpy(), x["draft_tokens"][sl].numpy(),
                            x["u_accept"][sl].numpy(), x["u_final"][sl].numpy(),
                            draft_len=np.asarray(lens[b:e], dtype=np.int32), temperature_all=1.0, nthreads=1)
        mine = torch.full((cfg.B, cfg.K + 2), -9, dtype=torch.int64)
        mine[sl, 0] = torch.from_numpy(res["accept_len"].astype(np.int64))
        mine[sl, 1:] = torch.from_numpy(res["out_tokens"].astype(np.int64))
        dist.all_reduce(mine, op=dist.ReduceOp.MAX)          # blocks are disjoint, the rest is -9
        times = max_over_ranks([1.0 + rank, 5.0 - rank], dist)
        if rank == 0:
            full = oracle.verify(x["target"].numpy(), x["draft"].numpy(), x["draft_tokens"].numpy(),
                                 x["u_accept"].numpy(), x["u_final"].numpy(),
                                 draft_len=np.asarray(lens, dtype=np.int32), temperature_all=1.0, nthreads=1)
            ok = (mine[:, 0].numpy() == full["accept_len"]).all() and (mine[:, 1:].numpy() == full["out_tokens"]).all()
            ret["ok"] = bool(ok)
            ret["times"] = times
    finally:
        dist.destroy_process_group()


def _bench_worker(rank, world, port, ret):
    """Two ranks go through bench.py's own per-rank function (strong scaling over a small ragged batch); the oracle
    stands in for the device step."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        import oracle
        over = {"B": 13, "V": 640}
        wl = bench.rank_workload(rank, world, "strong", "cpu", over)
        x, cfg = wl["x"], wl["cfg"]
        res = oracle.verify(x["target"].float().numpy(), x["draft"].float().numpy(), x["draft_tokens"].numpy(),
                            x["u_accept"].numpy(), x["u_final"].numpy(), draft_len=x["draft_len"].numpy(),
                            temperature=x["temperature"].numpy(), nthreads=1)
        mine = torch.full((cfg.B, cfg.K + 2), -9, dtype=torch.int64)
        sl = slice(wl["begin"], wl["end"])
        mine[sl, 0] = torch.from_numpy(res["accept_len"].astype(np.int64))
        mine[sl, 1:] = torch.from_numpy(res["out_tokens"].astype(np.int64))
        dist.all_reduce(mine, op=dist.ReduceOp.MAX)
        tot = torch.tensor([wl["positions"], wl["rows"], wl["nseq"]], dtype=torch.float64)
        dist.all_reduce(tot)
        edges = torch.zeros(world, 2, dtype=torch.int64)
        edges[rank, 0], edges[rank, 1] = wl["begin"], wl["end"]
        dist.all_reduce(edges)
        if rank == 0:
            whole = bench.rank_workload(0, 1, "strong", "cpu", over)
            xf = whole["x"]
            full = oracle.verify(xf["target"].float().numpy(), xf["draft"].float().numpy(), xf["draft_tokens"].numpy(),
                                 xf["u_accept"].numpy(), xf["u_final"].numpy(), draft_len=xf["draft_len"].numpy(),
                                 temperature=xf["temperature"].numpy(), nthreads=1)
            ret["same"] = bool((mine[:, 0].numpy() == full["accept_len"]).all() and (mine[:, 1:].numpy() == full["out_tokens"]).all())
            ret["totals"] = [float(v) for v in tot] == [float(whole["positions"]), float(whole["rows"]), float(whole["nseq"])]
            ret["cover"] = edges[0, 0].item() == 0 and edges[-1, 1].item() == cfg.B and all(
                edges[r, 1].item() == edges[r + 1, 0].item() for r in range(world - 1))
            rows = [int((2 * xf["draft_len"][edges[r, 0]:edges[r, 1]].long() + 1).sum()) for r in range(world)]
            ret["balanced"] = max(rows) - min(rows) <= 2 * (2 * cfg.K + 1)
    finally:
        dist.destroy_process_group()


def test_bench_rank_function_strong_scaling_two_ranks():
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_bench_worker, args=(2, _free_port(), ret), nprocs=2, join=True)
    assert ret["same"] and ret["totals"] and ret["cover"] and ret["balanced"], dict(ret)


def test_two_ranks_equal_one():
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(2, _free_port(), ret), nprocs=2, join=True)
    assert ret["ok"] is True
    assert ret["times"] == [2.0, 5.0]
