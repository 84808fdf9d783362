"""Keys and queries in 8 bits (e4m3) through the C ABI against the oracle's statement of the variant: the codes of the
cache and the scales bit for bit; exact pass, block scores, selection and reuse step against the by-definition routines
run on the oracle's codes, with the tolerances of the 16-bit path.  Contiguous and paged caches, ragged lengths, one and
two M-tiles, short and empty prefixes, rows appended under an existing scale, refused descriptions."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H


def _cache(batch, w, paged):
    lens = batch["seq_lens"].tolist()
    if paged:
        k_pool, v_pool, table, _ = W.to_paged(batch["kc"], batch["vc"], lens, 64, seed=w.seed)
        return mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"], block_table=table, N_max=batch["N_max"]), table
    return mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"]), None


def _codes_of(k8, kv, table, p, h, n):
    """The GPU's codes of rows [0, n) of head (p, h) as float64 grid values."""
    codes = k8.codes.view(torch.float8_e4m3fn)
    if table is None:
        return codes[p, h, :n].float().cpu().numpy().astype(np.float64)
    page = kv.c.page_size
    if n == 0:
        return np.zeros((0, kv.d))
    j = torch.arange(n, device=codes.device)
    pages = table[p].long()[j // page]
    return codes[pages, h, j % page].float().cpu().numpy().astype(np.float64)


def _run(batch, w, paged, k, steps=(0, 1)):
    kv, table = _cache(batch, w, paged)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    k8 = mb.K8Keys(kv)
    k8.codes.fill_(0x7F)                                   # NaN codes wherever nothing is written
    k8.quantize(0, status)
    out = torch.full((kv.P, kv.H_q, kv.B, kv.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    scores = torch.full((kv.P, kv.H_kv, max(1, kv.N_max)), -1.0, dtype=torch.float32, device="cuda")
    idx = torch.full((kv.P, kv.H_kv, k), -7, dtype=torch.int32, device="cuda")
    keff = torch.full((kv.P,), -7, dtype=torch.int32, device="cuda")
    ws = kv.new_workspace(k)
    mb.mage_exact_select_k8(kv, k8, batch["q"][steps[0]], batch["kb"][steps[0]], batch["vb"][steps[0]], kv.d ** -0.5, out, scores, ws, status)
    mb.mage_topk(scores, batch["seq_lens"], kv.P, kv.H_kv, kv.N_max, k, idx, keff)
    out_sp = torch.full_like(out, float("nan"))
    mb.mage_sparse_block_attn_k8(kv, k8, batch["q"][steps[1]], batch["kb"][steps[1]], batch["vb"][steps[1]], idx, keff, k, kv.d ** -0.5, out_sp, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return {"kv": kv, "k8": k8, "table": table, "out": out.float().cpu().numpy(), "scores": scores.cpu().numpy(), "idx": idx.cpu().numpy(),
            "keff": keff.cpu().numpy(), "out_sp": out_sp.float().cpu().numpy(), "k_scale": k8.k_scale.cpu().numpy()}


def _check(o, batch, w, res, k, steps=(0, 1), pairs=None):
    """Compare with the oracle, head by head; pairs = [(problem, KV head), ...] restricts the comparison (default: all)."""
    f = lambda t: t.float().cpu().numpy()
    G = w.G
    diag = {"o_max": 0.0, "score_rel": 0.0, "swaps": 0, "sp_max": 0.0}
    for p, n in enumerate(batch["seq_lens"].tolist()):
        heads = [h for h in range(w.H_kv) if pairs is None or (p, h) in pairs]
        assert res["keff"][p] == min(k, n)
        if n == 0:
            assert (res["idx"][p] == -1).all()
        for h in heads:
            g = slice(h * G, (h + 1) * G)
            Kc, Vc = f(batch["kc"][p, h:h + 1, :n]), f(batch["vc"][p, h:h + 1, :n])
            Q0, Kb0, Vb0 = f(batch["q"][steps[0], p, g]), f(batch["kb"][steps[0], p, h:h + 1]), f(batch["vb"][steps[0], p, h:h + 1])
            Qc, Kcc, Kbc, s_q, s_k = o.k8_quantize_block(Q0, Kc, Kb0)
            # the cache's codes and scales are the oracle's, bit for bit
            assert res["k_scale"][p, h] == s_k[0]
            got = _codes_of(res["k8"], res["kv"], res["table"], p, h, n)
            assert np.array_equal(got, Kcc[0]) and np.array_equal(np.signbit(got), np.signbit(Kcc[0]))
            O = o.k8_exact_block_attn(Qc, Kcc, Vc, Kbc, Vb0, s_q, s_k)
            err = np.abs(res["out"][p, g] - O)
            assert np.isfinite(res["out"][p, g]).all() and err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (p, h, err.max(), err.mean())
            diag["o_max"] = max(diag["o_max"], err.max())
            if n > 0:
                sc = o.k8_block_score(Qc, Kcc, s_q, s_k)[0]
                rel = np.max(np.abs(res["scores"][p, h, :n] - sc) / sc)
                assert rel <= H.SCORE_REL, (p, h, rel)
                diag["score_rel"] = max(diag["score_rel"], rel)
                assert (res["scores"][p, h, n:] == -1.0).all()
                diag["swaps"] += H.check_topk_band(sc, res["idx"][p, h], k, n)
            # reuse step: its own queries and block keys are coded at the call; the cache codes are the same
            Q1, Kb1, Vb1 = f(batch["q"][steps[1], p, g]), f(batch["kb"][steps[1], p, h:h + 1]), f(batch["vb"][steps[1], p, h:h + 1])
            Qc1, _, Kbc1, s_q1, _ = o.k8_quantize_block(Q1, Kc, Kb1)
            Os = o.k8_sparse_block_attn(Qc1, Kcc, Vc, Kbc1, Vb1, res["idx"][p, h:h + 1], int(res["keff"][p]), s_q1, s_k)
            e = np.abs(res["out_sp"][p, g] - Os)
            assert np.isfinite(res["out_sp"][p, g]).all() and e.max() <= H.O_MAX_ABS and e.mean() <= H.O_MEAN_ABS, (p, h, e.max(), e.mean())
            diag["sp_max"] = max(diag["sp_max"], e.max())
    return diag


CASES = [
    # name, H_q, H_kv, N, B, P, ragged_min, k
    ("two_mtiles_ragged", 14, 2, 1500, 32, 2, 300, 256),        # G*B = 224: two M-tiles; ragged tails inside a tile
    ("one_mtile", 8, 2, 1024, 32, 2, 0, 128),                   # G*B = 128: tile-parity mode, whole tiles only
    ("short_prefix", 4, 1, 90, 16, 1, 0, 128),                  # N < one tile and k > N
    ("rows_48", 6, 2, 700, 16, 3, 200, 64),                     # G*B = 48: a partly filled M-tile
    ("rows_448", 14, 2, 900, 64, 1, 0, 128),                    # G*B = 448: two row groups (queries coded by the kernel in front)
]


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_k8_block_against_oracle(oracle_mod, case, paged):
    name, H_q, H_kv, N, B, P, ragged_min, k = case
    w = W.Workload(name, H_q=H_q, H_kv=H_kv, N=N, B=B, k=k, T=2, P=P, n_heavy=min(64, N // 2), ragged_min=ragged_min, seed=11)
    batch = W.make_batch(w, device="cuda", steps=2)
    res = _run(batch, w, paged, k)
    diag = _check(oracle_mod, batch, w, res, k)
    print(name, "paged" if paged else "contiguous", diag)


def _global_properties(batch, res, k):
    """What holds at any size: finite outputs, score rows that sum to one, index rows ascending, in range, -1 padded."""
    assert np.isfinite(res["out"]).all() and np.isfinite(res["out_sp"]).all()
    for p, n in enumerate(batch["seq_lens"].tolist()):
        k_eff = min(k, n)
        assert res["keff"][p] == k_eff
        np.testing.assert_allclose(res["scores"][p, :, :n].astype(np.float64).sum(axis=1), 1.0, rtol=2e-5)
        idx = res["idx"][p, :, :k_eff]
        assert (idx >= 0).all() and (idx < n).all() and (np.diff(idx, axis=1) > 0).all() and (res["idx"][p, :, k_eff:] == -1).all()


def test_k8_cfg2_qwen_32k_every_head(oracle_mod):
    w = W.CONFIGS["cfg2_qwen_32k"]
    batch = W.make_batch(w, device="cuda", steps=2)
    res = _run(batch, w, False, w.k)
    _global_properties(batch, res, w.k)
    print("cfg2 k8", _check(oracle_mod, batch, w, res, w.k))
    # the planted heavy positions still dominate the selection made from 8-bit keys and queries
    for h in range(w.H_kv):
        assert len(set(res["idx"][0, h].tolist()) & set(batch["heavy"][0][h].tolist())) > 0.5 * w.k


def test_k8_cfg3_qwen_128k_28_layers_sampled(oracle_mod):
    """The benchmark workload in its batched launch: properties everywhere, four (layer, head) pairs element by element."""
    w = W.CONFIGS["cfg3_qwen_128k_x28"]
    batch = W.make_batch(w, device="cuda", steps=2)
    res = _run(batch, w, False, w.k)
    _global_properties(batch, res, w.k)
    print("cfg3 k8", _check(oracle_mod, batch, w, res, w.k, pairs=[(0, 0), (9, 1), (18, 2), (27, 3)]))


def test_k8_block_keys_clamp_at_the_cache_scale(oracle_mod):
    """Block keys four times larger than anything in the cache: their codes clamp at 448 on both sides."""
    w = W.Workload("clamp", H_q=8, H_kv=2, N=640, B=32, k=128, T=2, P=1, n_heavy=32, seed=12)
    batch = W.make_batch(w, device="cuda", steps=2)
    batch["kb"] = (batch["kb"].float() * 4).to(torch.bfloat16)
    res = _run(batch, w, False, w.k)
    _check(oracle_mod, batch, w, res, w.k)


def test_k8_empty_prefix(oracle_mod):
    w = W.Workload("empty", H_q=8, H_kv=2, N=256, B=32, k=64, T=2, P=2, n_heavy=16, seed=13)
    batch = W.make_batch(w, device="cuda", steps=2)
    batch["seq_lens"] = torch.tensor([0, 200], dtype=torch.int32, device="cuda")
    res = _run(batch, w, False, w.k)
    assert res["k_scale"][0].tolist() == [1.0, 1.0]             # no rows: scale 1
    _check(oracle_mod, batch, w, res, w.k)


def test_k8_appended_rows_keep_the_scale(oracle_mod):
    """Rows added after the first quantisation are coded under the head's existing scale (and clamp if they exceed it)."""
    w = W.Workload("append", H_q=4, H_kv=2, N=512, B=32, k=64, T=2, P=2, n_heavy=16, seed=14)
    batch = W.make_batch(w, device="cuda", steps=2)
    n0 = 300
    kc = batch["kc"].clone()
    kc[:, :, n0:] = (kc[:, :, n0:].float() * 3).to(torch.bfloat16)           # the later rows are larger
    lens0 = torch.full((w.P,), n0, dtype=torch.int32, device="cuda")
    kv0 = mb.KVCache(kc, batch["vc"], w.H_q, w.B, seq_lens=lens0)
    k8 = mb.K8Keys(kv0)
    k8.codes.fill_(0x7F)
    k8.quantize(0)
    scale0 = k8.k_scale.clone()
    lens0.fill_(w.N)                                                          # the cache grew
    k8.quantize(n0)
    torch.cuda.synchronize()
    assert torch.equal(scale0, k8.k_scale)
    codes = k8.codes.view(torch.float8_e4m3fn).float().cpu().numpy().astype(np.float64)
    kc_h = kc.float().cpu().numpy()
    for p in range(w.P):
        for h in range(w.H_kv):
            s = oracle_mod.k8_scale(kc_h[p, h, :n0])
            assert s == scale0[p, h].item()
            assert np.array_equal(codes[p, h], oracle_mod.k8_codes(kc_h[p, h], s))
            assert np.abs(codes[p, h, n0:]).max() == 448.0                    # some of the larger rows clamp


def test_k8_refusals():
    w = W.Workload("ref", H_q=8, H_kv=2, N=256, B=32, k=64, T=2, P=1, n_heavy=16, seed=15)
    batch = W.make_batch(w, device="cuda", steps=2)
    kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"], flags=mb.FLAG_SIMT_KERNELS)
    k8 = mb.K8Keys(kv).quantize()
    out = torch.empty(kv.P, kv.H_q, kv.B, kv.d, dtype=torch.bfloat16, device="cuda")
    scores = torch.empty(kv.P, kv.H_kv, kv.N_max, dtype=torch.float32, device="cuda")
    n0 = mb.launch_count()
    with pytest.raises(mb.MageError) as e:
        mb.mage_exact_select_k8(kv, k8, batch["q"][0], batch["kb"][0], batch["vb"][0], kv.d ** -0.5, out, scores, kv.new_workspace(64))
    assert e.value.code == -2 and mb.launch_count() == n0      # nothing launched
    kv2 = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"])
    bad = mb.K8Keys(kv2)
    bad.c.scratch = None
    with pytest.raises(mb.MageError) as e:
        mb.mage_exact_select_k8(kv2, bad, batch["q"][0], batch["kb"][0], batch["vb"][0], kv.d ** -0.5, out, scores, kv2.new_workspace(64))
    assert e.value.code == -1
    torch.cuda.synchronize()


def test_k8_through_block_attention_matches_the_direct_calls():
    """pipeline.BlockAttention(k8=...) issues the same calls (Step 1 with events, top-k on the select stream, reuse steps)."""
    from paper_2602_14209_b200.pipeline import BlockAttention
    w = W.Workload("pipe", H_q=14, H_kv=2, N=1200, B=32, k=256, T=3, P=2, n_heavy=64, ragged_min=500, seed=16)
    batch = W.make_batch(w, device="cuda", steps=3)
    res = _run(batch, w, False, w.k)                                   # direct calls: Step 1 on step 0, reuse step on step 1
    kv = res["kv"]
    ba = BlockAttention(kv, w.k, k8=res["k8"])
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    outs = ba.run_block([batch["q"][t] for t in range(3)], [batch["kb"][t] for t in range(3)], [batch["vb"][t] for t in range(3)], events=ev)
    torch.cuda.synchronize()
    assert int(ba.status.item()) == 0
    assert np.array_equal(ba.indices.cpu().numpy(), res["idx"]) and np.array_equal(ba.k_eff.cpu().numpy(), res["keff"])
    n = batch["seq_lens"].tolist()
    for p in range(w.P):
        assert np.array_equal(ba.scores[p, :, :n[p]].cpu().numpy(), res["scores"][p, :, :n[p]])
    assert ev[0].elapsed_time(ev[3]) > 0
    outs2 = [torch.empty_like(ba.out) for _ in range(3)]
    ba.run_block([batch["q"][t] for t in range(3)], [batch["kb"][t] for t in range(3)], [batch["vb"][t] for t in range(3)], outs2)
    torch.cuda.synchronize()
    assert np.array_equal(outs2[0].float().cpu().numpy(), res["out"]) and np.array_equal(outs2[1].float().cpu().numpy(), res["out_sp"])
    with pytest.raises(NotImplementedError):
        ba.exact_attn(batch["q"][0], batch["kb"][0], batch["vb"][0])


def test_k8_bad_indices_and_pages_are_skipped_and_tails_may_hold_anything(oracle_mod):
    """The 8-bit calls treat host-made faults like the 16-bit ones: an out-of-range index or page id sets a status bit and the
    key takes no part in the softmax; value rows and key codes beyond the prefix are NaN patterns here."""
    o = oracle_mod
    w = W.Workload("bad8", H_q=8, H_kv=2, N=640, B=32, k=64, T=2, n_heavy=16, page_size=64, seed=2)
    batch = W.make_batch(w, device="cuda", steps=2)
    n = 600                                                                  # not a multiple of 64: a ragged last tile
    batch["seq_lens"] = torch.tensor([n], dtype=torch.int32, device="cuda")
    batch["vc"][:, :, n:] = float("nan")
    f = lambda t: t.float().cpu().numpy()
    Kc, Vc = f(batch["kc"][0, :, :n]), f(batch["vc"][0, :, :n])
    for paged in (False, True):
        res = _run(batch, w, paged, w.k)
        kv, k8 = res["kv"], res["k8"]
        idx = torch.from_numpy(res["idx"]).cuda()
        keff = torch.from_numpy(res["keff"]).cuda()
        idx[0, 0, 5] = 1 << 28
        idx[0, 1, 0] = -7
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.full((kv.P, kv.H_q, kv.B, kv.d), float("nan"), dtype=torch.bfloat16, device="cuda")
        mb.mage_sparse_block_attn_k8(kv, k8, batch["q"][1], batch["kb"][1], batch["vb"][1], idx, keff, w.k, kv.d ** -0.5, out, kv.new_workspace(w.k), status)
        torch.cuda.synchronize()
        assert int(status.item()) == mb.DEV_BAD_INDEX
        idx_left = np.stack([np.delete(res["idx"][0, 0], 5), np.delete(res["idx"][0, 1], 0)])
        Qc1, Kcc, Kbc1, s_q1, s_k = o.k8_quantize_block(f(batch["q"][1, 0]), Kc, f(batch["kb"][1, 0]))
        O = o.k8_sparse_block_attn(Qc1, Kcc, Vc, Kbc1, f(batch["vb"][1, 0]), idx_left, w.k - 1, s_q1, s_k)
        err = np.abs(out.float().cpu().numpy()[0] - O)
        assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (paged, err.max(), err.mean())
    # a page id out of range in Step 1 (paged run above): its 64 keys are skipped by the attention and get score 0
    res["table"][0, 3] = 10 ** 6
    status.zero_()
    scores = torch.full((kv.P, kv.H_kv, kv.N_max), -1.0, dtype=torch.float32, device="cuda")
    mb.mage_exact_select_k8(kv, k8, batch["q"][0], batch["kb"][0], batch["vb"][0], kv.d ** -0.5, out, scores, kv.new_workspace(w.k), status)
    torch.cuda.synchronize()
    assert int(status.item()) == mb.DEV_BAD_PAGE
    keep = np.r_[0:192, 256:n]
    Qc, Kcc, Kbc, s_q, s_k = o.k8_quantize_block(f(batch["q"][0, 0]), Kc, f(batch["kb"][0, 0]))   # scales from the whole prefix, as the GPU's
    O = o.k8_exact_block_attn(Qc, Kcc[:, keep], Vc[:, keep], Kbc, f(batch["vb"][0, 0]), s_q, s_k)
    err = np.abs(out.float().cpu().numpy()[0] - O)
    assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (err.max(), err.mean())
    sc = o.k8_block_score(Qc, Kcc[:, keep], s_q, s_k)
    got = scores.cpu().numpy()[0].astype(np.float64)
    assert (got[:, 192:256] == 0.0).all() and (got[:, n:] == -1.0).all()
    assert np.max(np.abs(got[:, keep] - sc) / sc) <= H.SCORE_REL


def test_k8_zero_queries_and_zero_keys(oracle_mod):
    """amax = 0 takes scale 1 on both sides: an all-zero query head gives uniform attention, an all-zero key head too."""
    w = W.Workload("zeros", H_q=8, H_kv=2, N=300, B=32, k=64, T=2, P=1, n_heavy=16, seed=17)
    batch = W.make_batch(w, device="cuda", steps=2)
    batch["q"][:, :, :4] = 0                      # the four query heads of KV head 0, both steps
    batch["kc"][:, 1] = 0                         # every cached key of KV head 1
    res = _run(batch, w, False, w.k)
    assert res["k_scale"][0, 1] == 1.0
    _check(oracle_mod, batch, w, res, w.k)
    # uniform over the prefix for head 0: every score is 1 / N
    assert np.allclose(res["scores"][0, 0, :300], 1.0 / 300, rtol=1e-5)
