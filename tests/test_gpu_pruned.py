"""mage_exact_select_pruned: Step 1 + selection with the score pass restricted to the key tiles that can hold a selected
key.  Whatever it prunes, its output, index sets and k_eff must be those of mage_exact_select + mage_topk, and the
oracle's; entries of `scores` are exact where scored and zero where pruned, and every pruned entry's oracle score lies
below the k-th largest oracle score."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H


def _run_both(batch, w, paged=False, dense_above=0.5):
    lens = batch["seq_lens"].tolist()
    if paged:
        k_pool, v_pool, table, _ = W.to_paged(batch["kc"], batch["vc"], lens, 64, seed=w.seed)
        kv = mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"], block_table=table, N_max=batch["N_max"])
    else:
        kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"])
    plain = H.run_gpu_block(batch, w, paged=paged, steps=1)
    mk = lambda shape, dt, fill: torch.full(shape, fill, dtype=dt, device="cuda")
    out = mk((kv.P, kv.H_q, kv.B, kv.d), torch.bfloat16, float("nan"))
    scores = mk((kv.P, kv.H_kv, max(kv.N_max, 1)), torch.float32, -1.0)
    idx, keff = mk((kv.P, kv.H_kv, w.k), torch.int32, -9), mk((kv.P,), torch.int32, -9)
    tiles = mk((kv.P, kv.H_kv), torch.int32, -9)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    mb.mage_exact_select_pruned(kv, batch["q"][0], batch["kb"][0], batch["vb"][0], kv.d ** -0.5, w.k, out, scores, idx, keff,
                                mb.pruned_workspace(kv, w.k), tiles_scored=tiles, dense_above=dense_above, dev_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return plain, {"outs": [out.float().cpu().numpy()], "scores": scores.cpu().numpy(), "indices": idx.cpu().numpy(), "k_eff": keff.cpu().numpy(),
                   "status": 0, "k": w.k, "tiles": tiles.cpu().numpy()}


def _check(oracle_mod, batch, w, plain, got, problems=None, heads=None):
    lens = batch["seq_lens"].tolist()
    assert np.array_equal(got["indices"], plain["indices"]) and np.array_equal(got["k_eff"], plain["k_eff"])
    assert np.array_equal(got["outs"][0], plain["outs"][0])
    f = lambda t: t.float().cpu().numpy()
    for p in (range(w.P) if problems is None else problems):
        n = lens[p]
        sc_got, sc_plain = got["scores"][p, :, :n], plain["scores"][p, :, :n]
        scored = sc_got != 0.0
        assert np.array_equal(sc_got[scored], sc_plain[scored])                 # exact (the same bits) where scored
        assert (got["scores"][p, :, n:] == -1.0).all()                           # untouched beyond the prefix
        for h in (range(w.H_kv) if heads is None else heads):
            # oracle: the index set by the band rule, and every pruned key strictly below the k-th largest oracle score
            sc = oracle_mod.block_score(f(batch["q"][0, p, h * w.G:(h + 1) * w.G]), f(batch["kc"][p, h:h + 1, :n]))[0] if n else np.zeros(0)
            H.check_topk_band(sc, got["indices"][p, h], w.k, n)
            if 0 < min(w.k, n) < n:
                tau = np.partition(sc, n - w.k)[n - w.k]
                assert (sc[~scored[h]] < tau).all()
            tiles_head = (n + 127) // 128
            assert len(set((np.nonzero(scored[h])[0] // 128).tolist())) <= got["tiles"][p, h] <= tiles_head


@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
@pytest.mark.parametrize("shape", [(8, 2, 32, 3000, 256, 3), (28, 4, 32, 5000, 512, 2), (14, 2, 64, 900, 64, 1), (8, 2, 32, 100, 256, 2), (8, 2, 16, 0, 32, 1)],
                         ids=lambda s: "x".join(map(str, s)))
def test_flat_attention_prunes_nothing_and_changes_nothing(oracle_mod, shape, paged):
    from paper_2602_14209_b200 import build
    build.build()
    H_q, H_kv, B, N, k, P = shape
    w = W.Workload("pruned_flat", H_q=H_q, H_kv=H_kv, N=N, B=B, k=k, T=1, P=P, n_heavy=min(32, N), ragged_min=max(1, N // 4) if P > 1 else 0, seed=14)
    batch = W.make_batch(w, device="cuda")
    plain, got = _run_both(batch, w, paged)
    _check(oracle_mod, batch, w, plain, got)
    lens = batch["seq_lens"].tolist()
    for p, n in enumerate(lens):                                                  # flat scores: every tile had to be scored
        assert (got["tiles"][p] == (n + 127) // 128).all()


@pytest.mark.parametrize("dense_above", [0.5, 0.0])
def test_concentrated_attention_scores_a_fraction_of_the_tiles(oracle_mod, dense_above):
    """Planted keys strong enough to hold most of the mass: only the tiles that contain one are scored (dense_above = 0.5),
    or -- with the switch back to the dense pass forced by dense_above = 0 -- all of them; the selection is the same."""
    w = dataclasses.replace(W.CONFIGS["concentrated_qwen_128k_x28"], N=32768, P=3, T=1, n_heavy=512, k=256, seed=3)
    batch = W.make_batch(w, device="cuda")
    plain, got = _run_both(batch, w, dense_above=dense_above)
    _check(oracle_mod, batch, w, plain, got, heads=[1])
    tiles_head = w.N // 128
    print("tiles scored per head (of", tiles_head, "):", got["tiles"].tolist())
    if dense_above > 0:
        assert (got["tiles"] < 0.5 * tiles_head).all()
        for p in range(w.P):                                                      # the planted positions were all scored, and selected
            for h in range(w.H_kv):
                heavy = batch["heavy"][p][h].numpy()
                assert (got["scores"][p, h, heavy] > 0).all()
                assert len(set(heavy.tolist()) & set(got["indices"][p, h].tolist())) == w.k      # every selected key is a planted one
    else:
        assert (got["tiles"] == tiles_head).all()
