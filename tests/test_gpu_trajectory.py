"""Consecutive blocks end to end (Algorithm 1 including its last line, the cache append): each block runs Step 1,
selection and the reuse steps on the GPU, then appends its final K/V to the cache; the next block sees the longer
prefix.  The oracle follows with plain array concatenation."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
from paper_2602_14209_b200.pipeline import BlockAttention
import gpu_harness as H


@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
def test_three_blocks_with_cache_append(oracle_mod, paged):
    w = W.Workload("traj", H_q=8, H_kv=2, N=600, B=32, k=96, T=3, P=3, n_heavy=16, ragged_min=100, page_size=64, seed=31)
    n_blocks, cap = 3, 600 + 3 * 32 + 5                                   # capacity N_max leaves room for three blocks
    base = W.make_batch(w, device="cuda")
    lens0 = base["seq_lens"].tolist()
    lens0[2] = 0                                                          # one sequence starts with an empty prefix
    P, H_kv, d = w.P, w.H_kv, w.d
    kc = torch.zeros(P, H_kv, cap, d, dtype=torch.bfloat16, device="cuda")
    vc = torch.zeros_like(kc)
    for p in range(P):
        kc[p, :, :lens0[p]] = base["kc"][p, :, :lens0[p]]
        vc[p, :, :lens0[p]] = base["vc"][p, :, :lens0[p]]
    seq_lens = torch.tensor(lens0, dtype=torch.int32, device="cuda")
    if paged:
        # every logical page up to the capacity is mapped up front (page allocation is the caller's job)
        k_pool, v_pool, table, _ = W.to_paged(kc, vc, [cap] * P, 64, seed=1)
        kv = mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=seq_lens, block_table=table, N_max=cap)
    else:
        kv = mb.KVCache(kc, vc, w.H_q, w.B, seq_lens=seq_lens)
    ba = BlockAttention(kv, w.k)
    f = lambda t: t.float().cpu().numpy()
    # the oracle's own copy of the cache, grown by concatenation
    ref_k = [f(kc[p, :, :lens0[p]]) for p in range(P)]
    ref_v = [f(vc[p, :, :lens0[p]]) for p in range(P)]
    for b in range(n_blocks):
        blk = W.make_batch(dataclasses.replace(w, seed=100 + b, N=64, ragged_min=0), device="cuda")   # this block's q, K, V per step
        outs = [torch.empty_like(ba.out) for _ in range(w.T)]
        ba.run_block([blk["q"][t] for t in range(w.T)], [blk["kb"][t] for t in range(w.T)], [blk["vb"][t] for t in range(w.T)], outs)
        mb.mage_append_block(kv, blk["kb"][w.T - 1], blk["vb"][w.T - 1], seq_lens, ba.status)
        torch.cuda.synchronize()
        assert int(ba.status.item()) == 0
        idx, k_eff = ba.indices.cpu().numpy(), ba.k_eff.cpu().numpy()
        for p in range(P):
            n = ref_k[p].shape[1]
            assert k_eff[p] == min(w.k, n)
            r = oracle_mod.run_block(f(blk["q"][:, p]), ref_k[p], ref_v[p], f(blk["kb"][:, p]), f(blk["vb"][:, p]), w.k)
            err = np.abs(f(outs[0][p]) - r["O_exact"])
            assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (b, p, err.max())
            if n:
                sc = r["score"]
                for h in range(H_kv):
                    H.check_topk_band(sc[h], idx[p, h], w.k, n)
            for t in range(1, w.T):
                Os = oracle_mod.sparse_block_attn(f(blk["q"][t, p]), ref_k[p], ref_v[p], f(blk["kb"][t, p]), f(blk["vb"][t, p]), idx[p], int(k_eff[p]))
                e = np.abs(f(outs[t][p]) - Os)
                assert e.max() <= H.O_MAX_ABS and e.mean() <= H.O_MEAN_ABS, (b, p, t, e.max())
            ref_k[p] = np.concatenate([ref_k[p], f(blk["kb"][w.T - 1, p])], axis=1)
            ref_v[p] = np.concatenate([ref_v[p], f(blk["vb"][w.T - 1, p])], axis=1)
        assert seq_lens.tolist() == [lens0[p] + (b + 1) * w.B for p in range(P)]
    # the cache now holds exactly the oracle's concatenation (bit-exact copies); rows beyond stay as they were
    if not paged:
        for p in range(P):
            n = ref_k[p].shape[1]
            assert np.array_equal(f(kc[p, :, :n]), ref_k[p]) and np.array_equal(f(vc[p, :, :n]), ref_v[p])
            assert (kc[p, :, n:] == 0).all()
    # no room left for a fourth block in sequence 0 once the lengths are pushed to the limit: flagged, nothing changes
    seq_lens[0] = cap - 10
    before = seq_lens.clone()
    ba.status.zero_()
    mb.mage_append_block(kv, blk["kb"][0], blk["vb"][0], seq_lens, ba.status)
    torch.cuda.synchronize()
    assert int(ba.status.item()) & mb.DEV_CACHE_FULL
    assert int(seq_lens[0]) == int(before[0]) and int(seq_lens[1]) == int(before[1]) + w.B
