"""The N > 1 path on CPU: two gloo ranks each own a shard (by KV head, and by problem) and need nothing from the
other rank to compute it; gathered shards reproduce the unsharded result.  The per-shard arithmetic here is the
CPU oracle (this test has no GPU); what is under test is the sharding logic bench.py and a multi-GPU caller use.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, ret):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    os.environ["OMP_NUM_THREADS"] = "2"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2602_14209_b200 import workloads as W
    w = W.Workload("shard", H_q=8, H_kv=4, N=300, B=8, k=32, T=2, P=3, n_heavy=16, seed=4)
    f = lambda t: t.float().numpy()
    # (a) one layer split by KV head
    pr = W.make_problem(w, 0)
    hs, qs = W.shard_by_kv_head(w.H_q, w.H_kv, world, rank)
    r = oracle.run_block(f(pr["q"][:, qs]), f(pr["kc"][hs]), f(pr["vc"][hs]), f(pr["kb"][:, hs]), f(pr["vb"][:, hs]), w.k)
    mine = torch.from_numpy(np.concatenate([r["O_exact"].ravel(), r["O_sparse"][0].ravel(), r["idx"].ravel().astype(np.float64)]))
    gathered = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)          # only to compare; the path itself exchanged nothing
    # (b) problems split round-robin
    my_problems = W.shard_problems(w.P, world, rank)
    counts = torch.tensor([len(my_problems)])
    dist.all_reduce(counts)
    if rank == 0:
        full = oracle.run_block(f(pr["q"]), f(pr["kc"]), f(pr["vc"]), f(pr["kb"]), f(pr["vb"]), w.k)
        per = w.H_q // world * w.B * w.d
        O_e = np.concatenate([g[:per].numpy() for g in gathered]).reshape(w.H_q, w.B, w.d)
        O_s = np.concatenate([g[per:2 * per].numpy() for g in gathered]).reshape(w.H_q, w.B, w.d)
        idx = np.concatenate([g[2 * per:].numpy() for g in gathered]).reshape(w.H_kv, w.k).astype(np.int32)
        ok = (np.array_equal(O_e, full["O_exact"]) and np.array_equal(O_s, full["O_sparse"][0])
              and np.array_equal(idx, full["idx"]) and int(counts) == w.P)
        ret.put(bool(ok))
    dist.barrier()
    dist.destroy_process_group()


def test_kv_head_and_problem_sharding_world_size_2():
    import oracle
    oracle.build()
    ctx = mp.get_context("spawn")
    ret = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, ret)) for r in range(2)]
    for p in procs:
        p.start()
    ok = ret.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok


def test_shard_helpers():
    from paper_2602_14209_b200 import workloads as W
    import pytest
    assert W.shard_by_kv_head(28, 4, 2, 1) == (slice(2, 4), slice(14, 28))
    assert W.shard_by_kv_head(32, 8, 8, 3) == (slice(3, 4), slice(12, 16))
    with pytest.raises(ValueError):
        W.shard_by_kv_head(28, 4, 3, 0)
    assert sorted(sum((W.shard_problems(28, 4, r) for r in range(4)), [])) == list(range(28))
