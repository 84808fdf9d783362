"""GPU-vs-oracle parity through the C ABI (binding -> libmage.so), element by element on seeded inputs."""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H

IMPLS = [pytest.param(0, id="default"), pytest.param(mb.FLAG_SIMT_KERNELS, id="simt")]


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2602_14209_b200 import build
    build.build()
    assert torch.cuda.is_available()
    mb.load()


@pytest.mark.parametrize("flags", IMPLS)
def test_cfg1_small_all_elements(oracle_mod, flags):
    w = W.CONFIGS["cfg1_small"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w, flags=flags)
    d = H.check_problem(oracle_mod, batch, res, w, 0)
    print("cfg1", d)
    assert res["launches"] > 0


SMALL = [
    # (H_q, H_kv, B, N, k, T)  -- ragged tails, N < k, N < one tile, every G and B the sweep uses
    (8, 2, 32, 1000, 256, 2), (7, 1, 32, 777, 64, 2), (28, 4, 4, 1500, 128, 2), (28, 4, 16, 2049, 300, 2),
    (14, 2, 64, 1300, 2048, 2), (4, 4, 1, 130, 16, 2), (8, 2, 32, 100, 256, 2), (8, 2, 32, 0, 32, 2),
    (32, 8, 32, 4097, 512, 3), (8, 1, 64, 3000, 1024, 2),
]


@pytest.mark.parametrize("flags", IMPLS)
@pytest.mark.parametrize("shape", SMALL, ids=lambda s: "x".join(map(str, s)))
def test_small_and_ragged_shapes(oracle_mod, flags, shape):
    H_q, H_kv, B, N, k, T = shape
    w = W.Workload("small", H_q=H_q, H_kv=H_kv, N=N, B=B, k=k, T=T, n_heavy=min(32, N), seed=3)
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w, flags=flags)
    H.check_problem(oracle_mod, batch, res, w, 0)


@pytest.mark.parametrize("flags", IMPLS)
def test_batched_ragged_contiguous_and_paged_agree_with_oracle(oracle_mod, flags):
    w = W.Workload("ragged", H_q=8, H_kv=2, N=3000, B=32, k=200, T=2, P=5, n_heavy=32, ragged_min=40, page_size=64, seed=5)
    batch = W.make_batch(w, device="cuda")
    batch["seq_lens"][1] = 0                                         # one empty prefix in the batch
    for paged in (False, True):
        res = H.run_gpu_block(batch, w, flags=flags, paged=paged)
        for p in range(w.P):
            H.check_problem(oracle_mod, batch, res, w, p)


@pytest.mark.parametrize("flags", IMPLS)
def test_strided_cache_view(oracle_mod, flags):
    """The contiguous layout takes arbitrary (8-element aligned) strides: a [P, N, H_kv, d] buffer viewed as [P, H_kv, N, d]."""
    w = W.Workload("strided", H_q=8, H_kv=2, N=900, B=16, k=100, T=2, P=2, n_heavy=16, seed=9)
    batch = W.make_batch(w, device="cuda")
    kc_t = batch["kc"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    vc_t = batch["vc"].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert not kc_t.is_contiguous()
    b2 = dict(batch, kc=kc_t, vc=vc_t)
    res = H.run_gpu_block(b2, w, flags=flags)
    for p in range(w.P):
        H.check_problem(oracle_mod, batch, res, w, p)


def test_padded_row_pitch(oracle_mod):
    """Rows of 136 elements of which 128 are used: one row pitch for the whole cache (the reuse step's TMA row gather
    and the dense tensor maps both take the pitch from the strides)."""
    w = W.Workload("pitch", H_q=8, H_kv=2, N=1500, B=32, k=200, T=2, P=2, n_heavy=16, seed=10)
    batch = W.make_batch(w, device="cuda")
    def padded(x):
        buf = torch.full(x.shape[:-1] + (136,), 7.0, dtype=x.dtype, device=x.device)
        buf[..., :128] = x
        return buf[..., :128]
    b2 = dict(batch, kc=padded(batch["kc"]), vc=padded(batch["vc"]))
    assert b2["kc"].stride(2) == 136 and not b2["kc"].is_contiguous()
    res = H.run_gpu_block(b2, w)
    assert res["status"] == 0
    for p in range(w.P):
        H.check_problem(oracle_mod, batch, res, w, p)


@pytest.mark.parametrize("flags", IMPLS)
def test_runs_are_bitwise_reproducible(flags):
    w = dataclasses.replace(W.CONFIGS["cfg1_small"], N=5000, T=2)
    batch = W.make_batch(w, device="cuda")
    a = H.run_gpu_block(batch, w, flags=flags)
    b = H.run_gpu_block(batch, w, flags=flags)
    for x, y in zip(a["outs"], b["outs"]):
        assert np.array_equal(x, y)
    assert np.array_equal(a["scores"], b["scores"]) and np.array_equal(a["indices"], b["indices"])


def test_topk_edge_cases_against_full_sort():
    """mage_topk alone on crafted score rows: ties, zeros, k = N, k > N, N = 1, ragged lengths."""
    torch.manual_seed(0)
    P, H_kv, N_max, k = 3, 2, 5000, 37
    sc = torch.rand(P, H_kv, N_max, device="cuda")
    sc[0, 0, ::3] = 0.25                       # many exact ties around the threshold region
    sc[0, 1] = 0.0                             # all equal: the first k positions win
    sc[1, 0, :100] = torch.linspace(1, 2, 100, device="cuda")
    sc[2, 1, 4000:] = 1e-30                    # tiny values
    lens = torch.tensor([5000, 20, 4999], dtype=torch.int32, device="cuda")
    idx = torch.empty(P, H_kv, k, dtype=torch.int32, device="cuda")
    keff = torch.empty(P, dtype=torch.int32, device="cuda")
    mb.mage_topk(sc, lens, P, H_kv, N_max, k, idx, keff)
    torch.cuda.synchronize()
    from helpers import brute_force_topk
    for p in range(P):
        n = int(lens[p])
        assert int(keff[p]) == min(k, n)
        for h in range(H_kv):
            ref = brute_force_topk(sc[p, h, :n].double().cpu().numpy(), k)
            got = idx[p, h].cpu().numpy()
            assert np.array_equal(got[: len(ref)], ref), (p, h)
            assert (got[len(ref):] == -1).all()


def test_topk_long_rows_negative_values_and_quantised_ties():
    """Rows longer than one emit stretch (32 warps x 4096 entries), values of both signs, and a row quantised to 64 levels so
    that the threshold value has thousands of ties: positions come out ascending with ties to the smaller position."""
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    P, H_kv, N_max, k = 2, 2, 300001, 1000
    sc = torch.randn(P, H_kv, N_max, device="cuda", generator=g)
    sc[0, 1] = torch.round(sc[0, 1] * 8) / 8
    sc[1, 0] = -torch.rand(N_max, device="cuda", generator=g) - 1.0          # all negative
    lens = torch.tensor([300001, 140000], dtype=torch.int32, device="cuda")
    idx = torch.empty(P, H_kv, k, dtype=torch.int32, device="cuda")
    keff = torch.empty(P, dtype=torch.int32, device="cuda")
    mb.mage_topk(sc, lens, P, H_kv, N_max, k, idx, keff)
    torch.cuda.synchronize()
    from helpers import brute_force_topk
    for p in range(P):
        n = int(lens[p])
        for h in range(H_kv):
            ref = brute_force_topk(sc[p, h, :n].double().cpu().numpy(), k)
            assert np.array_equal(idx[p, h].cpu().numpy(), ref), (p, h)


@pytest.mark.parametrize("flags", IMPLS)
def test_bad_indices_and_pages_are_flagged_not_dereferenced(oracle_mod, flags):
    """Host-made faults: an out-of-range index / page id sets a status bit and the key is skipped -- it takes no part in
    the softmax, so the result is the oracle's on the inputs with that key removed, at the usual tolerances."""
    w = W.Workload("bad", H_q=8, H_kv=2, N=640, B=32, k=64, T=2, n_heavy=16, page_size=64, seed=2)
    batch = W.make_batch(w, device="cuda")
    f = lambda t: t.float().cpu().numpy()
    G = w.G
    for paged in (False, True):
        res = H.run_gpu_block(batch, w, paged=paged, flags=flags)
        ba = res["ba"]
        idx_good = ba.indices.cpu().numpy().copy()
        ba.indices[0, 0, 5] = 1 << 28
        ba.indices[0, 1, 0] = -7
        ba.status.zero_()
        out = ba.sparse_step(batch["q"][1], batch["kb"][1], batch["vb"][1])
        torch.cuda.synchronize()
        assert int(ba.status.item()) == mb.DEV_BAD_INDEX
        got = out.float().cpu().numpy()
        idx_left = np.stack([np.delete(idx_good[0, 0], 5), np.delete(idx_good[0, 1], 0)])       # one entry less per head
        O = oracle_mod.sparse_block_attn(f(batch["q"][1, 0]), f(batch["kc"][0]), f(batch["vc"][0]), f(batch["kb"][1, 0]),
                                         f(batch["vb"][1, 0]), idx_left, w.k - 1)
        err = np.abs(got[0] - O)
        assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (paged, err.max(), err.mean())
    # a page id out of range in Step 1: the 64 keys of that page are skipped by the attention and get score 0
    res = H.run_gpu_block(batch, w, paged=True, flags=flags)
    res["table"][0, 3] = 10 ** 6
    ba = res["ba"]
    ba.status.zero_()
    ba.scores.fill_(-1.0)
    ba.exact_select(batch["q"][0], batch["kb"][0], batch["vb"][0])
    torch.cuda.synchronize()
    assert int(ba.status.item()) == mb.DEV_BAD_PAGE
    keep = np.r_[0:192, 256:w.N]
    O = oracle_mod.exact_block_attn(f(batch["q"][0, 0]), f(batch["kc"][0])[:, keep], f(batch["vc"][0])[:, keep], f(batch["kb"][0, 0]),
                                    f(batch["vb"][0, 0]))
    err = np.abs(ba.out.float().cpu().numpy()[0] - O)
    assert err.max() <= H.O_MAX_ABS and err.mean() <= H.O_MEAN_ABS, (err.max(), err.mean())
    sc = oracle_mod.block_score(f(batch["q"][0, 0]), f(batch["kc"][0])[:, keep])
    got = ba.scores.cpu().numpy()[0].astype(np.float64)
    assert (got[:, 192:256] == 0.0).all()
    assert np.max(np.abs(got[:, keep] - sc) / sc) <= H.SCORE_REL


@pytest.mark.parametrize("flags", IMPLS)
@pytest.mark.parametrize("paged", [False, True], ids=["contiguous", "paged"])
def test_cache_rows_beyond_the_prefix_may_hold_anything(oracle_mod, flags, paged):
    """Cache rows at positions >= N_p are never used as data: they are filled with NaN bit patterns here (as an
    uninitialised or recycled cache would be) -- rows [N_p, N_max) of a contiguous cache, the tail of every last page and
    the spare pages of a pool -- with prefix lengths that are not multiples of 64 or 128.  Step 1, the select stream's
    scores alone, and the reuse step (single-CTA and split over CTAs) must all stay finite and match the oracle."""
    w = W.Workload("nan_tails", H_q=8, H_kv=2, N=3000, B=32, k=300, T=2, P=3, n_heavy=32, ragged_min=700, page_size=64, seed=31)
    batch = W.make_batch(w, device="cuda")
    lens = batch["seq_lens"].tolist()
    assert any(n % 64 for n in lens) and any(n % 128 for n in lens)
    nan = float("nan")
    clean = dict(batch, kc=batch["kc"].clone(), vc=batch["vc"].clone())
    for p, n in enumerate(lens):
        batch["kc"][p, :, n:] = nan
        batch["vc"][p, :, n:] = nan
    res = H.run_gpu_block(batch, w, paged=paged, flags=flags)
    if paged:
        # to_paged copies only rows < N_p; poison what it left: page tails and spare pages
        used = torch.zeros(res["k_pool"].shape[0], dtype=torch.bool, device="cuda")
        for p, n in enumerate(lens):
            pages = res["table"][p, : (n + 63) // 64].long()
            used[pages] = True
            if n % 64:
                res["k_pool"][pages[-1], :, n % 64:] = nan
                res["v_pool"][pages[-1], :, n % 64:] = nan
        res["k_pool"][~used] = nan
        res["v_pool"][~used] = nan
        res = dict(res, **_rerun(res["ba"], batch, w))
    for p in range(w.P):
        H.check_problem(oracle_mod, clean, res, w, p)
    ba = res["ba"]
    # the select stream's own pass (no values, no block keys)
    ba.scores.fill_(-1.0)
    mb.mage_select_scores(ba.kv, batch["q"][0], ba.sm_scale, ba.scores, ba.kv.new_workspace(w.k), ba.status)
    # the reuse step without a workspace: one CTA per (head, row group), no split
    out_ns = torch.empty_like(ba.out)
    mb.mage_sparse_block_attn(ba.kv, batch["q"][1], batch["kb"][1], batch["vb"][1], ba.indices, ba.k_eff, ba.k, ba.sm_scale, out_ns, None, ba.status)
    torch.cuda.synchronize()
    res2 = dict(res, scores=ba.scores.cpu().numpy(), outs=[res["outs"][0], out_ns.float().cpu().numpy()], status=int(ba.status.item()))
    for p in range(w.P):
        H.check_problem(oracle_mod, clean, res2, w, p)


def _rerun(ba, batch, w):
    """Run the block again on an existing BlockAttention (after its cache memory was modified in place)."""
    T = batch["q"].shape[0]
    outs = [torch.full_like(ba.out, float("nan")) for _ in range(T)]
    ba.scores.fill_(-1.0)
    ba.status.zero_()
    ba.run_block([batch["q"][t] for t in range(T)], [batch["kb"][t] for t in range(T)], [batch["vb"][t] for t in range(T)], outs)
    torch.cuda.synchronize()
    return {"outs": [o.float().cpu().numpy() for o in outs], "scores": ba.scores.cpu().numpy(), "indices": ba.indices.cpu().numpy(),
            "k_eff": ba.k_eff.cpu().numpy(), "status": int(ba.status.item())}


@pytest.mark.parametrize("flags", IMPLS)
def test_logit_jumps_beyond_the_lazy_rescale_range(oracle_mod, flags):
    """Keys whose logit exceeds everything seen before by far more than 2^100: the running reference of the online
    softmax has to move inside a tile (first half and second half) without losing the terms accumulated so far."""
    w = W.Workload("jumps", H_q=8, H_kv=2, N=1024, B=32, k=64, T=2, n_heavy=8, seed=12)
    batch = W.make_batch(w, device="cuda")
    batch["q"][..., 0] = 16.0
    batch["kc"][..., 0] = 0.0
    batch["kb"][..., 0] = 0.0
    for j, val in ((300, 64.0), (450, 144.0), (700, 256.0)):      # tile 2 first half, tile 3 second half, tile 5 first half
        batch["kc"][:, 0, j, 0] = val
    batch["kc"][:, 1, 20, 0] = 192.0                               # head 1: the big key sits in the very first tile
    batch["kc"][:, 1, 1000, 0] = 200.0                             # ... and a moderate rise (no overflow) near the end
    res = H.run_gpu_block(batch, w, flags=flags)
    # A row that one key dominates, met while the reference lags behind (rise between 2^8 and 2^100), carries that
    # key's bf16 rounding of P (relative 2^-9) into O, and |O| reaches 4 here (one bf16 ulp = 1.6e-2): the comparison is
    # against the oracle rounded to bf16, within two ulps.
    H.check_problem(oracle_mod, batch, res, w, 0, check_topk=False, o_rel_bf16=True)
    # the dominant key takes (almost) all of the probability mass of every row
    assert abs(res["scores"][0, 0, 700] - 1.0) < 1e-5 and res["scores"][0, 0, :700].max() < 1e-30


@pytest.mark.parametrize("H_q", [16, 28])
def test_logit_jumps_inside_multi_tile_ctas(oracle_mod, H_q):
    """The same jumps with enough (problem, head) pairs that a CTA of the exact pass walks several key tiles (a small
    batch gets one tile per CTA and never carries a reference from tile to tile): the jump then arrives in the single-sweep
    path, in the first half of a tile (redo on the careful path) and in the second half (the first half's PV has to be
    accumulated before the reference moves).  H_q = 16: one M-tile per head (two pipelines over alternating tiles);
    H_q = 28: two M-tiles."""
    w = W.Workload("jumps_multi", H_q=H_q, H_kv=4, N=2048, B=32, k=512, T=2, P=40, n_heavy=8, seed=13)
    batch = W.make_batch(w, device="cuda")
    batch["q"][..., 0] = 16.0
    batch["kc"][..., 0] = 0.0
    batch["kb"][..., 0] = 0.0
    # chunk 0 of a head is keys 0-1023: tile 2 first half, tile 3 second half, tile 5 first half, tile 6 second half
    for j, val in ((300, 64.0), (450, 144.0), (700, 256.0), (860, 400.0)):
        batch["kc"][:, 0, j, 0] = val
    batch["kc"][:, 1, 1100, 0] = 192.0                             # head 1: second chunk, first tile
    batch["kc"][:, 1, 1500, 0] = 200.0                             # ... and a moderate rise later in that chunk
    batch["kc"][:, 2, 1990, 0] = 300.0                             # head 2: second half of the ragged-free last tile
    res = H.run_gpu_block(batch, w)
    assert res["status"] == 0
    for p in (0, 39):
        H.check_problem(oracle_mod, batch, res, w, p, check_topk=False, o_rel_bf16=True)
    assert abs(res["scores"][0, 0, 860] - 1.0) < 1e-5 and res["scores"][0, 0, :860].max() < 1e-30


def test_layer_by_layer_runner_matches_batched_runner(oracle_mod):
    """pipeline.LayerwiseBlock (one launch per layer, P = 1 views of the same memory) against the batched call."""
    from paper_2602_14209_b200.pipeline import LayerwiseBlock
    w = W.Workload("layers", H_q=8, H_kv=2, N=3000, B=32, k=128, T=3, P=4, n_heavy=16, seed=17)
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w)
    lw = LayerwiseBlock(batch["kc"], batch["vc"], w.H_q, w.B, w.k, batch["seq_lens"])
    outs = [torch.full_like(lw.out, float("nan")) for _ in range(w.T)]
    lw.run_block([batch["q"][t] for t in range(w.T)], [batch["kb"][t] for t in range(w.T)], [batch["vb"][t] for t in range(w.T)], outs)
    torch.cuda.synchronize()
    assert int(lw.status.item()) == 0
    res_lw = {"outs": [o.float().cpu().numpy() for o in outs], "scores": lw.scores.cpu().numpy(), "indices": lw.indices.cpu().numpy(),
              "k_eff": lw.k_eff.cpu().numpy(), "status": 0, "k": w.k}
    res_lw["scores"][:, :, w.N:] = -1.0
    for p in range(w.P):
        H.check_problem(oracle_mod, batch, res_lw, w, p)
        assert np.abs(res_lw["outs"][0][p] - res["outs"][0][p]).max() < 1e-2


def test_sparse_step_without_workspace_and_events_variant(oracle_mod):
    """mage_sparse_block_attn accepts a null workspace (no split across CTAs); mage_exact_select_events records its events."""
    w = W.CONFIGS["cfg1_small"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w)
    ba = res["ba"]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    ba.exact_select(batch["q"][0], batch["kb"][0], batch["vb"][0], events=ev)
    out_a = ba.sparse_step(batch["q"][1], batch["kb"][1], batch["vb"][1]).clone()
    out_b = torch.empty_like(out_a)
    mb.mage_sparse_block_attn(ba.kv, batch["q"][1], batch["kb"][1], batch["vb"][1], ba.indices, ba.k_eff, ba.k, ba.sm_scale, out_b,
                              None, ba.status)
    torch.cuda.synchronize()
    assert ev[0].elapsed_time(ev[3]) > 0 and ev[0].elapsed_time(ev[1]) > 0
    assert (out_a.float() - out_b.float()).abs().max() < 5e-3
    assert np.abs(out_b.float().cpu().numpy() - res["outs"][1]).max() < 5e-3


def test_host_staged_blocks_match_the_resident_path(oracle_mod):
    """pipeline.HostStagedBlocks (pinned host inputs and outputs, two alternating sets of staging buffers) over four
    consecutive blocks with different inputs: every block's outputs on the host equal the resident-input run of that block."""
    from paper_2602_14209_b200.pipeline import HostStagedBlocks
    w = W.CONFIGS["cfg1_small"]
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w)
    ba, T = res["ba"], w.T
    staged = HostStagedBlocks(ba, T)
    host_out, expect = [], []
    for blk in range(4):
        scale = 1.0 + 0.25 * blk                                   # a different block each time
        q = [(batch["q"][t].float() * scale).to(torch.bfloat16) for t in range(T)]
        kb, vb = [batch["kb"][t] for t in range(T)], [batch["vb"][t] for t in range(T)]
        direct = [torch.empty_like(ba.out) for _ in range(T)]
        ba.run_block(q, kb, vb, direct)
        torch.cuda.synchronize()
        expect.append([o.cpu() for o in direct])
        out_h = [torch.empty(ba.out.shape, dtype=torch.bfloat16).pin_memory() for _ in range(T)]
        host_out.append(out_h)
        staged.submit([t.cpu().pin_memory() for t in q], [t.cpu().pin_memory() for t in kb], [t.cpu().pin_memory() for t in vb], out_h)
    staged.finish()
    assert int(ba.status.item()) == 0
    for blk in range(4):
        for t in range(T):
            assert torch.equal(host_out[blk][t], expect[blk][t]), (blk, t)
    assert np.abs(expect[0][0].float().numpy() - res["outs"][0]).max() == 0.0


def test_layouts_outside_the_tensor_core_kernels_are_refused_not_rerouted(oracle_mod):
    """16-token pages: the tensor-core kernels do not take them (a 64-key TMA box must lie inside one page).  The call is
    refused with MAGE_ERR_UNSUPPORTED and nothing runs -- no silent switch to the slow kernels; with MAGE_FLAG_SIMT_KERNELS
    the caller gets the portable kernels and the oracle's result."""
    w = W.Workload("small_pages", H_q=8, H_kv=2, N=700, B=32, k=100, T=2, P=2, n_heavy=16, ragged_min=200, page_size=16, seed=4)
    batch = W.make_batch(w, device="cuda")
    launches0 = mb.launch_count()
    with pytest.raises(mb.MageError) as e:
        H.run_gpu_block(batch, w, paged=True)
    assert e.value.code == -2 and mb.launch_count() == launches0
    k_pool, v_pool, table, _ = W.to_paged(batch["kc"], batch["vc"], batch["seq_lens"].tolist(), 16, seed=w.seed)
    kv = mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"], block_table=table, N_max=batch["N_max"])
    out = torch.empty(w.P, w.H_q, w.B, w.d, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(mb.MageError) as e:
        mb.mage_exact_attn(kv, batch["q"][0], batch["kb"][0], batch["vb"][0], 0.088, out, kv.new_workspace(w.k))
    assert e.value.code == -2 and mb.launch_count() == launches0
    res = H.run_gpu_block(batch, w, paged=True, flags=mb.FLAG_SIMT_KERNELS)
    for p in range(w.P):
        H.check_problem(oracle_mod, batch, res, w, p)


def _random_shapes(n, seed):
    rng = np.random.RandomState(seed)
    shapes = []
    for _ in range(n):
        G, H_kv = int(rng.choice([1, 2, 4, 7, 8])), int(rng.choice([1, 2, 4]))
        B = int(rng.choice([1, 4, 16, 32, 64]))
        N = int(rng.choice([rng.randint(0, 200), rng.randint(200, 2000), rng.randint(2000, 9000)]))
        k = int(rng.choice([16, 100, 512, 1024]))
        P = int(rng.choice([1, 2, 3]))
        paged = bool(rng.randint(0, 2))
        ragged = bool(rng.randint(0, 2)) and N > 64
        shapes.append((G * H_kv, H_kv, B, N, k, P, paged, ragged))
    return shapes


@pytest.mark.parametrize("shape", _random_shapes(12, seed=20260214), ids=lambda s: "x".join(str(int(v)) for v in s))
def test_randomly_drawn_shapes(oracle_mod, shape):
    """Shapes drawn at random (fixed seed): group size, KV heads, block size, prefix length, budget, batch, paged or not,
    ragged or not -- every problem of each batch against the oracle."""
    H_q, H_kv, B, N, k, P, paged, ragged = shape
    w = W.Workload("drawn", H_q=H_q, H_kv=H_kv, N=N, B=B, k=k, T=2, P=P, n_heavy=min(32, N), seed=11,
                   ragged_min=(N // 8 + 1) if ragged else 0, page_size=64 if paged else 0)
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w, paged=paged)
    assert res["status"] == 0
    for p in range(P):
        H.check_problem(oracle_mod, batch, res, w, p)


@pytest.mark.parametrize("flags", IMPLS)
@pytest.mark.parametrize("shape", [(8, 2, 32, 5000, 2), (28, 4, 32, 9000, 3), (14, 2, 64, 700, 1)], ids=lambda s: "x".join(map(str, s)))
def test_select_stream_scores_alone(oracle_mod, flags, shape):
    """mage_select_scores (Algorithm 1's select stream on its own: scores from Q and the cached keys, no attention output)
    gives the scores of mage_exact_select bit for bit, with ragged lengths and pages, and the two-stream pipeline built on
    it selects the same sets."""
    H_q, H_kv, B, N, P = shape
    w = W.Workload("select_only", H_q=H_q, H_kv=H_kv, N=N, B=B, k=128, T=2, P=P, n_heavy=32, seed=21,
                   ragged_min=N // 4 if P > 1 else 0, page_size=64 if P == 3 else 0)
    batch = W.make_batch(w, device="cuda")
    res = H.run_gpu_block(batch, w, paged=(P == 3), flags=flags)
    ba = res["ba"]
    fused_scores, fused_idx = ba.scores.clone(), ba.indices.clone()
    ba.scores.fill_(-1.0)
    ws2 = ba.kv.new_workspace(w.k)
    mb.mage_select_scores(ba.kv, batch["q"][0], ba.sm_scale, ba.scores, ws2, ba.status)
    torch.cuda.synchronize()
    assert int(ba.status.item()) == 0
    lens = batch["seq_lens"].tolist()
    for p in range(P):
        assert torch.equal(ba.scores[p, :, :lens[p]], fused_scores[p, :, :lens[p]]), p
        assert (ba.scores[p, :, lens[p]:] == -1.0).all()
    # the paper's arrangement: attention on the main stream, scores + top-k on the select stream, one join
    ba.indices.fill_(-7)
    out = torch.empty_like(ba.out)
    ba.select_scores_async(batch["q"][0])
    ba.exact_attn(batch["q"][0], batch["kb"][0], batch["vb"][0], out)
    ba.join()
    torch.cuda.synchronize()
    assert torch.equal(ba.indices, fused_idx)
    assert np.array_equal(out.float().cpu().numpy(), res["outs"][0])
    # and against the oracle directly: the attention output of mage_exact_attn, the scores of mage_select_scores and
    # the sets selected from them (Algorithm 1, main stream and select stream), problem by problem
    res2 = {"outs": [out.float().cpu().numpy()], "scores": ba.scores.cpu().numpy(), "indices": ba.indices.cpu().numpy(),
            "k_eff": ba.k_eff.cpu().numpy(), "status": int(ba.status.item()), "k": w.k}
    for p in range(P):
        H.check_problem(oracle_mod, batch, res2, w, p)
