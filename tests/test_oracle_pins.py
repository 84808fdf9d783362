"""Pins for the CPU oracle: it is checked against things other than itself.

Brute force in NumPy on tiny inputs, library special cases (torch SDPA, torch.topk),
a hand-derived worked example, closed forms and invariants (Algorithm 1, Eq. 2-4).
"""
import os

import numpy as np
import pytest
import torch

from helpers import bf16_exact, brute_force_block, brute_force_sparse, brute_force_topk

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")


def _rand_problem(rng, H_q, H_kv, B, N, d):
    return (bf16_exact(rng, (H_q, B, d)), bf16_exact(rng, (H_kv, N, d)), bf16_exact(rng, (H_kv, N, d)),
            bf16_exact(rng, (H_kv, B, d)), bf16_exact(rng, (H_kv, B, d)))


@pytest.mark.parametrize("G", [1, 4, 7])
@pytest.mark.parametrize("B,N,d", [(1, 5, 8), (4, 64, 16), (3, 37, 128)])
def test_bruteforce_tiny(oracle_mod, G, B, N, d):
    rng = np.random.default_rng(100 * G + B)
    H_kv = 2
    Q, Kc, Vc, Kb, Vb = _rand_problem(rng, G * H_kv, H_kv, B, N, d)
    scale = 1.0 / np.sqrt(d)
    O_ref, sc_ref = brute_force_block(Q, Kc, Vc, Kb, Vb, scale)
    O = oracle_mod.exact_block_attn(Q, Kc, Vc, Kb, Vb)
    sc = oracle_mod.block_score(Q, Kc)
    np.testing.assert_allclose(O, O_ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(sc, sc_ref, rtol=1e-12, atol=1e-15)
    for k in (1, 3, N, N + 4):
        idx, k_eff = oracle_mod.topk(sc, k)
        assert k_eff == min(k, N)
        for h in range(H_kv):
            np.testing.assert_array_equal(idx[h, :k_eff], brute_force_topk(sc_ref[h], k))
            assert (idx[h, k_eff:] == -1).all()
        Os = oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx, k_eff)
        np.testing.assert_allclose(Os, brute_force_sparse(Q, Kc, Vc, Kb, Vb, idx, k_eff, scale), rtol=0, atol=1e-12)


def test_worked_example(oracle_mod):
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        key, *nums = line.split()
        vals[key] = np.array([float(x) for x in nums])
    ln = np.log
    Q = np.array([[[1.0, 0.0]], [[0.0, 1.0]]], dtype=np.float32)             # [H_q=2, B=1, d=2]
    Kc = np.array([[[ln(3), 0.0], [0.0, ln(5)]]], dtype=np.float32)          # [1, 2, 2]
    Kb = np.array([[[ln(2), ln(2)]]], dtype=np.float32)
    Vc = np.array([[[1.0, 0.0], [0.0, 1.0]]], dtype=np.float32)
    Vb = np.array([[[1.0, 1.0]]], dtype=np.float32)
    O = oracle_mod.exact_block_attn(Q, Kc, Vc, Kb, Vb, scale=1.0)
    np.testing.assert_allclose(O.ravel(), vals["O_exact"], atol=3e-7)           # fp32 rounding of ln(.) only
    sc = oracle_mod.block_score(Q, Kc, scale=1.0)
    np.testing.assert_allclose(sc.ravel(), vals["score"], atol=3e-7)
    idx, k_eff = oracle_mod.topk(sc, 1)
    assert idx[0, 0] == int(vals["top1"][0]) and k_eff == 1
    Os = oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx, k_eff, scale=1.0)
    np.testing.assert_allclose(Os.ravel(), vals["O_sparse"], atol=3e-7)


def test_matches_torch_sdpa_and_topk(oracle_mod):
    """Exact pass == SDPA over concat(cache, block) with KV heads repeated G times; sparse == SDPA on gathered rows."""
    rng = np.random.default_rng(7)
    H_q, H_kv, B, N, d = 8, 2, 8, 300, 64
    G = H_q // H_kv
    Q, Kc, Vc, Kb, Vb = _rand_problem(rng, H_q, H_kv, B, N, d)
    t = lambda a: torch.from_numpy(a).double()
    K_all = torch.cat([t(Kc), t(Kb)], dim=1).repeat_interleave(G, dim=0)
    V_all = torch.cat([t(Vc), t(Vb)], dim=1).repeat_interleave(G, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(t(Q), K_all, V_all).numpy()
    O, lse = oracle_mod.exact_block_attn(Q, Kc, Vc, Kb, Vb, return_lse=True)
    np.testing.assert_allclose(O, ref, atol=1e-12)
    S = torch.einsum("gqd,gnd->gqn", t(Q), t(Kc).repeat_interleave(G, dim=0)) / np.sqrt(d)
    np.testing.assert_allclose(lse, torch.logsumexp(S, dim=-1).numpy(), atol=1e-12)
    sc = oracle_mod.block_score(Q, Kc)
    sc_ref = torch.softmax(S, dim=-1).reshape(H_kv, G * B, N).mean(dim=1).numpy()
    np.testing.assert_allclose(sc, sc_ref, rtol=1e-12)
    k = 40
    idx, k_eff = oracle_mod.topk(sc, k)
    for h in range(H_kv):
        assert set(idx[h].tolist()) == set(torch.topk(torch.from_numpy(sc[h]), k).indices.tolist())
        assert (np.diff(idx[h]) > 0).all()
    Kg = torch.stack([t(Kc)[h][idx[h]] for h in range(H_kv)])
    Vg = torch.stack([t(Vc)[h][idx[h]] for h in range(H_kv)])
    ref_s = torch.nn.functional.scaled_dot_product_attention(
        t(Q), torch.cat([Kg, t(Kb)], 1).repeat_interleave(G, 0), torch.cat([Vg, t(Vb)], 1).repeat_interleave(G, 0)).numpy()
    np.testing.assert_allclose(oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx, k_eff), ref_s, atol=1e-12)


def test_invariants(oracle_mod):
    rng = np.random.default_rng(11)
    H_q, H_kv, B, N, d = 14, 2, 5, 193, 32
    Q, Kc, Vc, Kb, Vb = _rand_problem(rng, H_q, H_kv, B, N, d)
    sc = oracle_mod.block_score(Q, Kc)
    # every softmax row sums to one, so the mean over rows does too (pins the prefix-only domain and the 1/(GB))
    np.testing.assert_allclose(sc.sum(axis=1), 1.0, rtol=1e-13)
    assert (sc > 0).all()
    # k = N: the sparse step is the exact pass
    idx, k_eff = oracle_mod.topk(sc, N)
    assert k_eff == N and (idx == np.arange(N)).all()
    O = oracle_mod.exact_block_attn(Q, Kc, Vc, Kb, Vb)
    np.testing.assert_allclose(oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx, N), O, atol=1e-13)
    # k > N behaves as k = N, padded with -1
    idx2, k_eff2 = oracle_mod.topk(sc, N + 7)
    assert k_eff2 == N and (idx2[:, N:] == -1).all()
    # permuting cache positions permutes the score, maps the top-k set, leaves O unchanged
    perm = rng.permutation(N)
    sc_p = oracle_mod.block_score(Q, Kc[:, perm])
    np.testing.assert_allclose(sc_p, sc[:, perm], rtol=1e-12)
    np.testing.assert_allclose(oracle_mod.exact_block_attn(Q, Kc[:, perm], Vc[:, perm], Kb, Vb), O, atol=1e-12)
    k = 17
    idx_k, _ = oracle_mod.topk(sc, k)
    idx_kp, _ = oracle_mod.topk(sc_p, k)
    for h in range(H_kv):
        assert set(perm[idx_kp[h]].tolist()) == set(idx_k[h].tolist())
    # the sparse step does not depend on the order of the index list
    Os = oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx_k, k)
    shuffled = np.stack([rng.permutation(row) for row in idx_k]).astype(np.int32)
    np.testing.assert_allclose(oracle_mod.sparse_block_attn(Q, Kc, Vc, Kb, Vb, shuffled, k), Os, atol=1e-13)
    # top-k set is a prefix of the full sort and holds at least as much mass as any other k-set
    for h in range(H_kv):
        np.testing.assert_array_equal(idx_k[h], brute_force_topk(sc[h], k))
        other = rng.choice(N, size=k, replace=False)
        assert sc[h][idx_k[h]].sum() >= sc[h][other].sum()
    # splitting the prefix in chunks and merging (m, L, O) by log-sum-exp reproduces the one-shot result
    cut = 80
    _, lse_a = oracle_mod.exact_block_attn(Q, Kc[:, :cut], Vc[:, :cut], Kb, Vb, return_lse=True)
    _, lse_b = oracle_mod.exact_block_attn(Q, Kc[:, cut:], Vc[:, cut:], Kb, Vb, return_lse=True)
    _, lse = oracle_mod.exact_block_attn(Q, Kc, Vc, Kb, Vb, return_lse=True)
    np.testing.assert_allclose(np.logaddexp(lse_a, lse_b), lse, rtol=1e-13)


def test_closed_forms(oracle_mod):
    rng = np.random.default_rng(3)
    H_q, H_kv, B, N, d = 4, 2, 3, 50, 16
    Q, Kc, Vc, Kb, Vb = _rand_problem(rng, H_q, H_kv, B, N, d)
    # all prefix keys equal: score is 1/N everywhere; with equal block keys too, O is the plain mean of all values
    Kc_eq = np.broadcast_to(Kc[:, :1], Kc.shape).copy()
    np.testing.assert_allclose(oracle_mod.block_score(Q, Kc_eq), 1.0 / N, rtol=1e-13)
    Kb_eq = np.broadcast_to(Kc[:, :1], Kb.shape).copy()
    O = oracle_mod.exact_block_attn(Q, Kc_eq, Vc, Kb_eq, Vb)
    mean_v = np.concatenate([Vc, Vb], axis=1).astype(np.float64).mean(axis=1)       # [H_kv, d]
    np.testing.assert_allclose(O, np.repeat(mean_v, H_q // H_kv, axis=0)[:, None, :].repeat(B, 1), atol=1e-13)
    # zero queries: uniform attention
    np.testing.assert_allclose(oracle_mod.block_score(np.zeros_like(Q), Kc), 1.0 / N, rtol=1e-13)
    # one key far above the rest: its score tends to 1 and O to its value row
    Qd = np.zeros_like(Q); Qd[..., 0] = 8.0
    Kd = np.zeros_like(Kc); Kd[:, 7, 0] = 32.0                                      # logit 8*32/4 = 64 above the others
    sc = oracle_mod.block_score(Qd, Kd)
    assert np.all(sc[:, 7] >= 1 - 1e-15) and np.all(np.delete(sc, 7, axis=1) < 1e-25)
    O = oracle_mod.exact_block_attn(Qd, Kd, Vc, np.zeros_like(Kb), Vb)
    np.testing.assert_allclose(O, np.repeat(Vc[:, 7], H_q // H_kv, axis=0)[:, None, :].repeat(B, 1), atol=1e-20)
    # B = G = 1: single-query decode attention; the score is the softmax row itself
    q1, k1 = Q[:1, :1], Kc[:1]
    s = (k1[0].astype(np.float64) @ q1[0, 0].astype(np.float64)) / np.sqrt(d)
    p = np.exp(s - s.max()); p /= p.sum()
    np.testing.assert_allclose(oracle_mod.block_score(q1, k1)[0], p, rtol=1e-13)
    # N = 0: attention inside the block only
    O0 = oracle_mod.exact_block_attn(Q, Kc[:, :0], Vc[:, :0], Kb, Vb)
    ref0, _ = brute_force_block(Q, Kc[:, :0], Vc[:, :0], Kb, Vb, 1 / np.sqrt(d))
    np.testing.assert_allclose(O0, ref0, atol=1e-13)
    idx0, k0 = oracle_mod.topk(np.zeros((H_kv, 0)), 4)
    assert k0 == 0 and (idx0 == -1).all()


def test_ties_prefer_smaller_position(oracle_mod):
    sc = np.array([[0.1, 0.3, 0.3, 0.1, 0.3, 0.05]])
    idx, _ = oracle_mod.topk(sc, 2)
    assert idx.tolist() == [[1, 2]]
    idx, _ = oracle_mod.topk(sc, 4)
    assert idx.tolist() == [[0, 1, 2, 4]]


def test_recall_and_planted_structure(oracle_mod):
    """Eq. 3 on the synthetic recipe: heavy positions are over-represented in the Step-1 set, drift keeps recall high."""
    import dataclasses
    from paper_2602_14209_b200 import workloads as W
    w = dataclasses.replace(W.CONFIGS["cfg1_small"], N=1024, T=3)
    pr = W.make_problem(w, 0)
    f = lambda a: a.float().numpy()
    sc1 = oracle_mod.block_score(f(pr["q"][0]), f(pr["kc"]))
    idx1, k_eff = oracle_mod.topk(sc1, w.k)
    for h in range(w.H_kv):
        frac = len(set(idx1[h].tolist()) & set(pr["heavy"][h].tolist())) / w.n_heavy
        assert frac > 0.9                          # chance level would be k/N = 0.25
    for t in (1, 2):
        idx_t, _ = oracle_mod.topk(oracle_mod.block_score(f(pr["q"][t]), f(pr["kc"])), w.k)
        r = oracle_mod.recall(idx1, idx_t, k_eff)
        assert ((r > 0.3) & (r <= 1.0)).all()
    assert (oracle_mod.recall(idx1, idx1, k_eff) == 1.0).all()


def test_recall_known_answers(oracle_mod):
    """Eq. 3 on hand-made index sets whose overlap is known: half, none, all, and a short prefix (k_eff < k, -1 padding),
    where the denominator is the number of entries a set actually holds."""
    a = np.array([[0, 1, 2, 3], [0, 1, 2, 3], [5, 6, 7, 8]], dtype=np.int32)
    b = np.array([[2, 3, 4, 5], [4, 5, 6, 7], [8, 7, 6, 5]], dtype=np.int32)
    assert oracle_mod.recall(a, b, 4).tolist() == [0.5, 0.0, 1.0]
    # N = 3 < k = 5: three entries per set, the rest is padding that must not count as a match
    a = np.array([[0, 1, 2, -1, -1]], dtype=np.int32)
    b = np.array([[1, 2, 9, -1, -1]], dtype=np.int32)
    np.testing.assert_allclose(oracle_mod.recall(a, b, 3), [2.0 / 3.0])
    # one shared entry of four, two KV heads with different answers
    a = np.array([[10, 20, 30, 40], [1, 2, 3, 4]], dtype=np.int32)
    b = np.array([[40, 50, 60, 70], [1, 2, 3, 9]], dtype=np.int32)
    assert oracle_mod.recall(a, b, 4).tolist() == [0.25, 0.75]


# ---- Quest-style page estimator (comparison system): pins for the oracle's restatement -----------------------------
def _quest_inputs(seed, H_q=4, H_kv=2, B=3, N=70, d=8):
    rng = np.random.default_rng(seed)
    from helpers import bf16_exact
    return bf16_exact(rng, (H_q, B, d)), bf16_exact(rng, (H_kv, N, d))


def test_quest_page_score_brute_force_loops(oracle_mod):
    """Pure-Python loops over pages, tokens, channels, rows on a tiny case (including a ragged tail that is no page)."""
    Q, Kc = _quest_inputs(1)
    H_q, B, d = Q.shape
    H_kv, N, _ = Kc.shape
    G, page = H_q // H_kv, 16
    kmin, kmax = oracle_mod.quest_page_summaries(Kc, page)
    sc = oracle_mod.quest_page_scores(Q, kmin, kmax)
    assert kmin.shape == (H_kv, N // page, d) and sc.shape == (H_kv, N // page)
    for h in range(H_kv):
        for pg in range(N // page):
            total = 0.0
            for g in range(h * G, (h + 1) * G):
                for qi in range(B):
                    for c in range(d):
                        lo = min(float(Kc[h, pg * page + t, c]) for t in range(page))
                        hi = max(float(Kc[h, pg * page + t, c]) for t in range(page))
                        total += max(float(Q[g, qi, c]) * hi, float(Q[g, qi, c]) * lo)
            np.testing.assert_allclose(sc[h, pg], total / (G * B), rtol=1e-12, atol=1e-12)


def test_quest_bound_dominates_every_key_of_its_page(oracle_mod):
    """The defining property (Section 2.2): per query, the page bound is an upper bound on q.k for every key of the page,
    so the per-block page score is at least the mean over rows of the page's best exact logit."""
    Q, Kc = _quest_inputs(2, H_q=6, H_kv=2, B=4, N=96, d=16)
    kmin, kmax = oracle_mod.quest_page_summaries(Kc)
    sc = oracle_mod.quest_page_scores(Q, kmin, kmax)
    G = 3
    for h in range(2):
        rows = Q[h * G:(h + 1) * G].reshape(-1, 16).astype(np.float64)
        logits = rows @ Kc[h].astype(np.float64).T                        # [M, N]
        best = logits.reshape(rows.shape[0], 6, 16).max(axis=2)            # per row and page
        assert (sc[h] >= best.mean(axis=0) - 1e-12).all()
        # and a transposed or sign-flipped bound would violate it somewhere: the bound is tight for single-key pages
    kmin1, kmax1 = oracle_mod.quest_page_summaries(Kc, page=1)
    sc1 = oracle_mod.quest_page_scores(Q, kmin1, kmax1)
    for h in range(2):
        rows = Q[h * G:(h + 1) * G].reshape(-1, 16).astype(np.float64)
        np.testing.assert_allclose(sc1[h], (rows @ Kc[h].astype(np.float64).T).mean(axis=0), rtol=1e-12, atol=1e-12)


def test_quest_closed_forms_and_selection(oracle_mod):
    """All keys of a page equal -> the bound is the exact logit; positive queries -> only Kmax matters; the selected
    tokens are whole pages, ascending, and the ragged tail is never selected."""
    rng = np.random.default_rng(3)
    from helpers import bf16_exact
    Q = np.abs(bf16_exact(rng, (2, 2, 8))) + 0.5
    Kc = bf16_exact(rng, (1, 52, 8))
    Kc[0, 16:32] = Kc[0, 16]                                               # page 1: sixteen copies of one key
    kmin, kmax = oracle_mod.quest_page_summaries(Kc)
    sc = oracle_mod.quest_page_scores(Q, kmin, kmax)
    rows = Q.reshape(-1, 8).astype(np.float64)
    np.testing.assert_allclose(sc[0, 1], (rows @ Kc[0, 16].astype(np.float64)).mean(), rtol=1e-12)
    np.testing.assert_allclose(sc[0], (rows @ kmax[0].T).mean(axis=0), rtol=1e-12)      # q > 0: the max keys alone
    idx, k_eff, _ = oracle_mod.quest_select(Q, Kc, 32)
    assert k_eff == 32 and (np.diff(idx[0]) > 0).all() and idx.max() < 48               # positions 48..51 are no page
    best2 = np.sort(np.argsort(-sc[0], kind="stable")[:2])
    assert idx[0].tolist() == [int(p) * 16 + t for p in best2 for t in range(16)]
    idx, k_eff, _ = oracle_mod.quest_select(Q, Kc, 64)                                   # more pages asked than exist
    assert k_eff == 48 and (idx[0, 48:] == -1).all() and idx[0, :48].tolist() == list(range(48))



# ---------------------------------------------------------------------------------------------------------------------
# 8-bit keys: the e4m3 rounding, the scales, and the wrappers that run the by-definition routines on the codes
# ---------------------------------------------------------------------------------------------------------------------
def _e4m3_grid():
    """The finite e4m3 values, written out from the format: sign, 4 exponent bits (bias 7), 3 mantissa bits, 0x7f/0xff = NaN."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            vals.append(m * 2.0 ** -9 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(sorted(set(vals)))


def test_e4m3_round_grid_and_ties(oracle_mod):
    o = oracle_mod
    grid = _e4m3_grid()
    assert grid.size == 127 and grid[-1] == 448.0 and grid[1] == 2.0 ** -9       # 126 positive values and zero
    # grid values are fixed points, both signs
    assert np.array_equal(o.e4m3_round(grid), grid) and np.array_equal(o.e4m3_round(-grid), -grid)
    # every value lands on the grid, on a nearest neighbour, and monotonically
    rng = np.random.default_rng(5)
    y = np.concatenate([rng.uniform(-460, 460, 20000), rng.normal(size=20000) * 0.05, rng.normal(size=20000) * 1e-3])
    r = o.e4m3_round(y)
    assert np.isin(np.abs(r), grid).all()
    clipped = np.clip(np.abs(y), 0, 448.0)
    nearest = np.abs(grid[None, :] - clipped[:, None]).min(axis=1)
    assert np.allclose(np.abs(np.abs(r) - clipped), nearest, rtol=0, atol=1e-15)
    ys = np.sort(y)
    assert (np.diff(o.e4m3_round(ys)) >= 0).all()
    # ties go to the even mantissa: midpoints between consecutive grid values
    mid = 0.5 * (grid[:-1] + grid[1:])
    want = np.where((np.arange(grid.size - 1) % 2) == 0, grid[:-1], grid[1:])     # grid index = mantissa parity (zero is even)
    assert np.array_equal(o.e4m3_round(mid), want)
    # clamping and specials
    assert np.array_equal(o.e4m3_round([464.0, 1e9, np.inf, -np.inf, -500.0]), [448.0, 448.0, 448.0, -448.0, -448.0])
    assert np.isnan(o.e4m3_round([np.nan]))[0]
    assert np.signbit(o.e4m3_round([-0.0]))[0] and o.e4m3_round([2.0 ** -11])[0] == 0.0 and o.e4m3_round([1.5 * 2.0 ** -10])[0] == 2.0 ** -9


def test_e4m3_round_matches_library_cast(oracle_mod):
    """torch's float -> float8_e4m3fn cast is round-to-nearest-even inside the finite range."""
    rng = np.random.default_rng(6)
    y = np.concatenate([rng.uniform(-448, 448, 50000), rng.normal(size=50000), rng.normal(size=50000) * 2.0 ** -7]).astype(np.float32)
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(oracle_mod.e4m3_round(y.astype(np.float64)), lib)


def test_k8_scale_codes_and_wrappers(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(7)
    H_kv, G, B, N, d = 2, 2, 3, 37, 16
    bf = lambda a: torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    Q = bf(rng.normal(size=(H_kv * G, B, d)).astype(np.float32)); Kc = bf(rng.normal(size=(H_kv, N, d)).astype(np.float32) * 3)
    Kb = bf(rng.normal(size=(H_kv, B, d)).astype(np.float32) * 6)                  # larger than the cache: some clamp
    Vc = bf(rng.normal(size=(H_kv, N, d)).astype(np.float32)); Vb = bf(rng.normal(size=(H_kv, B, d)).astype(np.float32))
    Qc, Kcc, Kbc, s_q, s_k = o.k8_quantize_block(Q, Kc, Kb)
    grid = _e4m3_grid()
    for h in range(H_kv):
        amax = np.abs(Kc[h]).max()
        assert s_k[h] == np.float32(amax / np.float32(448)) and s_k[h].dtype == np.float32
        assert np.abs(Kcc[h]).max() == 448.0                                        # the largest element gets the largest code
        assert np.abs(Qc[h * G:(h + 1) * G]).max() == 448.0
        # de-quantised keys are within half a grid step (2^-4 relative for normal codes) of the originals
        err = np.abs(Kcc[h] * float(s_k[h]) - Kc[h])
        assert (err <= np.maximum(np.abs(Kc[h]) * 2.0 ** -4, float(s_k[h]) * 2.0 ** -10) * 1.0001).all()
        assert np.abs(Kbc[h]).max() == 448.0 and (np.abs(Kb[h]) > amax * 1.1).any()   # block keys clamp at the cache's scale
    assert np.isin(np.abs(Qc), grid).all() and np.isin(np.abs(Kcc), grid).all() and np.isin(np.abs(Kbc), grid).all()
    assert o.k8_scale(np.zeros((3, 4), np.float32)) == np.float32(1) and o.k8_scale(np.zeros((0, 4), np.float32)) == np.float32(1)
    assert np.array_equal(o.k8_codes(np.array([0.5, -0.25], np.float32), np.float32(2.0 ** -9)), [256.0, -128.0])
    # the wrappers = the by-definition routines applied to the de-quantised tensors (written out here in float64 NumPy)
    Qd = np.concatenate([Qc[h * G:(h + 1) * G] * float(s_q[h]) for h in range(H_kv)], axis=0)
    Kd = Kcc * s_k.astype(np.float64)[:, None, None]; Kbd = Kbc * s_k.astype(np.float64)[:, None, None]
    scale = 1.0 / np.sqrt(d)
    O, lse = o.k8_exact_block_attn(Qc, Kcc, Vc, Kbc, Vb, s_q, s_k, return_lse=True)
    sc = o.k8_block_score(Qc, Kcc, s_q, s_k)
    for hq in range(H_kv * G):
        h = hq // G
        logits = np.concatenate([Qd[hq] @ Kd[h].T, Qd[hq] @ Kbd[h].T], axis=1) * scale     # [B, N + B]
        p = np.exp(logits - logits.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
        assert np.allclose(O[hq], p @ np.concatenate([Vc[h], Vb[h]], axis=0), rtol=1e-12, atol=1e-13)
    for h in range(H_kv):
        acc = np.zeros(N)
        for hq in range(h * G, (h + 1) * G):
            lg = (Qd[hq] @ Kd[h].T) * scale
            pp = np.exp(lg - lg.max(axis=1, keepdims=True)); pp /= pp.sum(axis=1, keepdims=True)
            acc += pp.sum(axis=0)
        assert np.allclose(sc[h], acc / (G * B), rtol=1e-12, atol=1e-15)
    idx, k_eff = o.topk(sc, 8)
    Os = o.k8_sparse_block_attn(Qc, Kcc, Vc, Kbc, Vb, idx, k_eff, s_q, s_k)
    for hq in range(H_kv * G):
        h = hq // G
        sel = idx[h, :k_eff]
        logits = np.concatenate([Qd[hq] @ Kd[h][sel].T, Qd[hq] @ Kbd[h].T], axis=1) * scale
        p = np.exp(logits - logits.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
        assert np.allclose(Os[hq], p @ np.concatenate([Vc[h][sel], Vb[h]], axis=0), rtol=1e-12, atol=1e-13)
