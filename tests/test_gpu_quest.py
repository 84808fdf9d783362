"""The Quest-style per-block page estimator (the paper's comparison system) through the C ABI against its oracle
restatement: page summaries bit for bit, page scores within fp32 accumulation error, the selected pages by the band rule,
the expanded index set consumed by the reuse step.  Contiguous and paged caches, ragged lengths, N < 16, k > N."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H

PAGE = mb.QUEST_PAGE
SCORE_ABS_REL = 2e-5            # |gpu - oracle| <= this * max|score| (fp32 sums of 128 signed products, twice, against fp64)


def _run_quest(batch, w, paged, step=0):
    lens = batch["seq_lens"].tolist()
    if paged:
        k_pool, v_pool, table, _ = W.to_paged(batch["kc"], batch["vc"], lens, 64, seed=w.seed)
        kv = mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"], block_table=table, N_max=batch["N_max"])
    else:
        kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"])
    n_pages_max = max(1, (kv.N_max + PAGE - 1) // PAGE)
    pmin = torch.full((kv.P, kv.H_kv, n_pages_max, kv.d), 99.0, dtype=torch.bfloat16, device="cuda")
    pmax = torch.full_like(pmin, -99.0)
    scores = torch.full((kv.P, kv.H_kv, n_pages_max), -5.0, dtype=torch.float32, device="cuda")
    idx = torch.full((kv.P, kv.H_kv, w.k), -7, dtype=torch.int32, device="cuda")
    keff = torch.full((kv.P,), -7, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mb.mage_quest_build(kv, pmin, pmax, status)
    mb.mage_quest_select(kv, batch["q"][step], pmin, pmax, w.k, scores, idx, keff, mb.quest_workspace(kv, w.k))
    out = torch.empty(kv.P, kv.H_q, kv.B, kv.d, dtype=torch.bfloat16, device="cuda")
    mb.mage_sparse_block_attn(kv, batch["q"][step], batch["kb"][step], batch["vb"][step], idx, keff, w.k, kv.d ** -0.5, out,
                              kv.new_workspace(w.k), status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return pmin.float().cpu().numpy(), pmax.float().cpu().numpy(), scores.cpu().numpy(), idx.cpu().numpy(), keff.cpu().numpy(), out.float().cpu().numpy()


def _check(oracle_mod, batch, w, got, step=0):
    pmin, pmax, scores, idx, keff, out = got
    f = lambda t: t.float().cpu().numpy()
    lens = batch["seq_lens"].tolist()
    k_pages = w.k // PAGE
    for p, n in enumerate(lens):
        n_pages = n // PAGE
        Kc, Vc = f(batch["kc"][p, :, :n]), f(batch["vc"][p, :, :n])
        kmin, kmax = oracle_mod.quest_page_summaries(Kc)
        assert np.array_equal(pmin[p, :, :n_pages], kmin) and np.array_equal(pmax[p, :, :n_pages], kmax)
        assert (pmin[p, :, n_pages:] == 99.0).all()                         # nothing written beyond the whole pages
        sc = oracle_mod.quest_page_scores(f(batch["q"][step, p]), kmin, kmax)
        assert keff[p] == PAGE * min(k_pages, n_pages)
        if n_pages:
            scale = np.abs(sc).max()
            assert np.abs(scores[p, :, :n_pages] - sc).max() <= SCORE_ABS_REL * scale
        assert (scores[p, :, n_pages:] == -5.0).all()
        n_sel = min(k_pages, n_pages)
        for h in range(w.H_kv):
            sel = idx[p, h, : n_sel * PAGE]
            assert (idx[p, h, n_sel * PAGE:] == -1).all()
            pages = sel.reshape(n_sel, PAGE)
            assert (pages == pages[:, :1] + np.arange(PAGE)[None, :]).all() and (pages[:, 0] % PAGE == 0).all()   # whole pages
            chosen = pages[:, 0] // PAGE
            assert (np.diff(chosen) > 0).all() and (chosen < max(n_pages, 1)).all()
            if 0 < n_sel < n_pages:                                         # band rule on the page scores
                tau = np.partition(sc[h], n_pages - n_sel)[n_pages - n_sel]
                band = SCORE_ABS_REL * scale
                mask = np.zeros(n_pages, dtype=bool)
                mask[chosen] = True
                assert mask[sc[h] > tau + band].all() and not mask[sc[h] < tau - band].any()
        # the reuse step on that index set against the oracle's sparse attention on the same set
        O = oracle_mod.sparse_block_attn(f(batch["q"][step, p]), Kc, Vc, f(batch["kb"][step, p]), f(batch["vb"][step, p]), idx[p], int(keff[p]))
        err = np.abs(out[p] - O)
        assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS


@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
@pytest.mark.parametrize("shape", [(8, 2, 32, 3000, 256, 3), (28, 4, 32, 2049, 512, 2), (8, 2, 16, 10, 32, 2), (32, 8, 32, 700, 2048, 2)],
                         ids=lambda s: "x".join(map(str, s)))
def test_quest_path_matches_its_oracle(oracle_mod, shape, paged):
    from paper_2602_14209_b200 import build
    build.build()
    H_q, H_kv, B, N, k, P = shape
    w = W.Workload("quest", H_q=H_q, H_kv=H_kv, N=N, B=B, k=k, T=2, P=P, n_heavy=min(32, N), ragged_min=max(1, N // 5) if P > 1 else 0, seed=6)
    batch = W.make_batch(w, device="cuda")
    _check(oracle_mod, batch, w, _run_quest(batch, w, paged, step=1), step=1)


def test_quest_against_exact_selection_on_the_planted_workload(oracle_mod):
    """Sanity figure, not a parity bar: on the planted-heavy-key recipe the page estimator finds fewer of the exact
    per-block top-k entries than the exact score does (which finds all of them by definition) -- the accuracy gap of
    Section 3.1, Fig. 1b, on synthetic inputs."""
    w = dataclasses.replace(W.CONFIGS["cfg2_qwen_32k"], N=8192, k=512)
    batch = W.make_batch(w, device="cuda", steps=1)
    got = _run_quest(batch, w, False)
    f = lambda t: t.float().cpu().numpy()
    exact_idx, k_eff = oracle_mod.topk(oracle_mod.block_score(f(batch["q"][0, 0]), f(batch["kc"][0])), w.k)
    acc = oracle_mod.recall(exact_idx, got[3][0], k_eff)
    print("estimation accuracy of the page estimator against the exact per-block top-k:", acc)
    assert ((acc >= 0.0) & (acc < 1.0)).all()
