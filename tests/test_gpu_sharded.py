"""KV-head sharding on the GPU: every stage of the path is independent per KV head (Eq. 2 / Eq. 4 sum only inside
group(h)), so a rank that owns KV heads [a, b) runs the library on a strided view of the cache and on its own query
heads, and needs nothing from its peers.

One GPU is enough to check that: the shards of a world of 2 and of 4 are run one after the other, each through the
C ABI on the views a rank would pass, and every shard must match the oracle on its own heads.  With two or more GPUs
visible, the second test runs one process per GPU and rank 0 checks the gathered result against the unsharded oracle.
"""
import os
import socket

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H


@pytest.mark.parametrize("world", [2, 4])
def test_each_kv_head_shard_matches_the_oracle(oracle_mod, world):
    from paper_2602_14209_b200 import build
    build.build()
    w = W.Workload("sharded", H_q=28, H_kv=4, N=3000, B=32, k=256, T=2, P=2, n_heavy=32, ragged_min=900, seed=8)
    batch = W.make_batch(w, device="cuda")
    full = H.run_gpu_block(batch, w)
    idx_parts, out_parts = [], []
    for rank in range(world):
        w_r, b_r = W.shard_batch_by_kv_head(batch, w, world, rank)
        assert not b_r["kc"].is_contiguous() and b_r["kc"].data_ptr() == batch["kc"][:, rank * (w.H_kv // world)].data_ptr()
        res = H.run_gpu_block(b_r, w_r)
        assert res["status"] == 0
        for p in range(w.P):
            H.check_problem(oracle_mod, b_r, res, w_r, p)
        idx_parts.append(res["indices"])
        out_parts.append(res["outs"][1])
    # reassembled shards against the unsharded run: same selected sets, outputs within the output tolerance
    assert np.array_equal(np.concatenate(idx_parts, axis=1), full["indices"])
    assert np.abs(np.concatenate(out_parts, axis=1) - full["outs"][1]).max() <= H.O_MAX_ABS


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, ret):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)          # plumbing for the comparison only
    torch.cuda.set_device(rank)
    import sys
    sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
    import gpu_harness as Hh
    w = W.Workload("sharded_mp", H_q=32, H_kv=8, N=2500, B=32, k=128, T=2, P=2, n_heavy=32, seed=9)
    batch = W.make_batch(w, device=f"cuda:{rank}")                       # same seed on every rank: same tensors
    w_r, b_r = W.shard_batch_by_kv_head(batch, w, world, rank)
    res = Hh.run_gpu_block(b_r, w_r)
    mine = torch.from_numpy(res["outs"][0]).contiguous()
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine)
    if rank == 0:
        import oracle
        oracle.build()
        f = lambda t: t.float().cpu().numpy()
        got = np.concatenate([p.numpy() for p in parts], axis=1)
        ok = True
        for p in range(w.P):
            O = oracle.exact_block_attn(f(batch["q"][0, p]), f(batch["kc"][p]), f(batch["vc"][p]), f(batch["kb"][0, p]), f(batch["vb"][0, p]))
            err = np.abs(got[p] - O)
            ok = ok and err.max() <= Hh.O_MAX_ABS and err.mean() <= Hh.O_MEAN_ABS
        ret.put(bool(ok))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.skipif(torch.cuda.device_count() < 2, reason="needs two GPUs")
def test_one_process_per_gpu_reassembles_to_the_unsharded_oracle():
    import torch.multiprocessing as mp
    world = 2
    ctx = mp.get_context("spawn")
    ret = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, ret)) for r in range(world)]
    for p in procs:
        p.start()
    ok = ret.get(timeout=300)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ok
