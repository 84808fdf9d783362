"""The five benchmark configurations at full size, in the batched launch configuration bench.py uses.

Where the oracle cannot cover every output in seconds, sampled (problem, KV head) pairs are compared element by
element and properties that hold at any size are checked everywhere (score rows sum to one, indices ascending and
in range, outputs finite, no device status bit).
"""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H


def _global_properties(batch, res, w):
    lens = batch["seq_lens"].tolist()
    assert res["status"] == 0
    for o in res["outs"]:
        assert np.isfinite(o).all()
    for p, n in enumerate(lens):
        k_eff = min(res["k"], n)
        assert res["k_eff"][p] == k_eff
        if n == 0:
            continue
        sums = res["scores"][p, :, :n].astype(np.float64).sum(axis=1)
        np.testing.assert_allclose(sums, 1.0, rtol=2e-5)
        idx = res["indices"][p, :, :k_eff]
        assert (idx >= 0).all() and (idx < n).all() and (np.diff(idx, axis=1) > 0).all()
        assert (res["indices"][p, :, k_eff:] == -1).all()


def test_cfg2_qwen_32k_every_head(oracle_mod):
    w = W.CONFIGS["cfg2_qwen_32k"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w)
    _global_properties(batch, res, w)
    d = H.check_problem(oracle_mod, batch, res, w, 0, sparse_steps=(1, w.T - 1))
    print("cfg2", d)
    # planted heavy positions dominate the selection
    for h in range(w.H_kv):
        hit = len(set(res["indices"][0, h].tolist()) & set(batch["heavy"][0][h].tolist()))
        assert hit > 0.5 * w.k


def test_cfg3_qwen_128k_28_layers_sampled(oracle_mod):
    """Every layer of the 28-layer batch, one KV head per layer (h = layer mod 4), element by element: Step 1 and the
    first and last reuse steps."""
    w = W.CONFIGS["cfg3_qwen_128k_x28"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w)
    _global_properties(batch, res, w)
    worst = {}
    for p in range(w.P):
        d = H.check_problem(oracle_mod, batch, res, w, p, heads=[p % w.H_kv], sparse_steps=(1, w.T - 1))
        for key, v in d.items():
            worst[key] = max(worst.get(key, 0), v)
    print("cfg3 worst over 28 (layer, head) pairs", worst)


@pytest.mark.parametrize("B,k", [(4, 128), (16, 1024), (32, 512), (64, 2048)])
def test_cfg4_budget_block_sweep_cells_with_recall(oracle_mod, B, k):
    w = W.cfg4_variant(B, k)
    T = min(w.T, 3)
    batch = W.make_batch(w, device="cuda", steps=T)
    res = H.run_gpu_block(batch, w)
    _global_properties(batch, res, w)
    h = 1
    d = H.check_problem(oracle_mod, batch, res, w, 0, heads=[h], sparse_steps=range(1, T))
    # Eq. 3 on the drifted queries, oracle-computed: recall of the Step-1 set against each later step's exact set
    f = lambda t: t.float().cpu().numpy()
    G = w.G
    Kc = f(batch["kc"][0, h:h + 1])
    idx1, k_eff = oracle_mod.topk(oracle_mod.block_score(f(batch["q"][0, 0, h * G:(h + 1) * G]), Kc), k)
    recalls = []
    for t in range(1, T):
        idx_t, _ = oracle_mod.topk(oracle_mod.block_score(f(batch["q"][t, 0, h * G:(h + 1) * G]), Kc), k)
        recalls.append(float(oracle_mod.recall(idx1, idx_t, k_eff)[0]))
    print(f"cfg4 B={B} k={k}", d, "recall(step1 -> later steps)", recalls)
    assert all(0.0 < r <= 1.0 for r in recalls) or T == 1


def test_cfg5_llama_ragged_paged_sampled(oracle_mod):
    """Every sequence of the ragged paged batch, one KV head per sequence (h = sequence mod 8), element by element."""
    w = W.CONFIGS["cfg5_llama_ragged_paged"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w, paged=True)
    _global_properties(batch, res, w)
    lens = batch["seq_lens"].tolist()
    worst = {}
    for p in range(w.P):
        d = H.check_problem(oracle_mod, batch, res, w, p, heads=[p % w.H_kv], sparse_steps=(1, w.T - 1))
        for key, v in d.items():
            worst[key] = max(worst.get(key, 0), v)
    print("cfg5 lens", lens, "worst over 16 (sequence, head) pairs", worst)


def test_topk_overlaps_main_stream_work():
    """The select stream runs mage_topk while the main stream keeps working; one join before the first reuse step."""
    w = dataclasses.replace(W.CONFIGS["cfg2_qwen_32k"], P=8)
    batch = W.make_batch(w, device="cuda", steps=2)
    kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"])
    from paper_2602_14209_b200.pipeline import BlockAttention
    ba = BlockAttention(kv, w.k)
    other = BlockAttention(kv, w.k)                 # a second batch whose sparse steps keep the main stream busy
    other.run_block([batch["q"][0], batch["q"][1]], [batch["kb"][0], batch["kb"][1]], [batch["vb"][0], batch["vb"][1]])
    torch.cuda.synchronize()
    main = torch.cuda.current_stream()
    ev = {k: torch.cuda.Event(enable_timing=True) for k in ("scores", "topk_done", "main_done")}
    ba.exact_select(batch["q"][0], batch["kb"][0], batch["vb"][0])
    ev["scores"].record(main)
    ba.select_async(main)
    ev["topk_done"].record(ba.select_stream)
    for _ in range(40):
        other.sparse_step(batch["q"][1], batch["kb"][1], batch["vb"][1])
    ev["main_done"].record(main)
    ba.join(main)
    out = ba.sparse_step(batch["q"][1], batch["kb"][1], batch["vb"][1])
    torch.cuda.synchronize()
    t_topk = ev["scores"].elapsed_time(ev["topk_done"])
    t_main = ev["scores"].elapsed_time(ev["main_done"])
    print("topk finished", t_topk, "ms after the scores; main-stream filler finished after", t_main, "ms")
    assert t_topk < t_main, "top-k did not overlap the main stream's work"
    assert torch.isfinite(out.float()).all() and int(ba.status.item()) == 0
