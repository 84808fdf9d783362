"""ctypes front end of ``mage_oracle.c`` (fp64, by-definition; see the C file).

TEST INFRASTRUCTURE ONLY: nothing in the product path may import this module.
Every function takes float32 NumPy arrays whose values are bf16-exact and
returns float64 / int32 NumPy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mage_oracle.c")
_LIB = os.path.join(_HERE, "libmage_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, so fp64 sums keep their written order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_topk.restype = ctypes.c_int
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.c_void_p)


def exact_block_attn(Q, Kc, Vc, Kb, Vb, scale=None, return_lse=False):
    """Exact attention of one block (Algorithm 1 main stream).  Q [H_q,B,d], Kc/Vc [H_kv,N,d], Kb/Vb [H_kv,B,d]."""
    Q, pq = _f32(Q); Kc, pk = _f32(Kc); Vc, pv = _f32(Vc); Kb, pkb = _f32(Kb); Vb, pvb = _f32(Vb)
    H_q, B, d = Q.shape
    H_kv, N, _ = Kc.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    O = np.empty((H_q, B, d), dtype=np.float64)
    lse = np.empty((H_q, B), dtype=np.float64)
    _load().oracle_exact_block_attn(pq, pk, pv, pkb, pvb, H_q, H_kv, B, d, ctypes.c_int64(N), ctypes.c_double(scale),
                                    O.ctypes.data_as(ctypes.c_void_p), lse.ctypes.data_as(ctypes.c_void_p))
    return (O, lse) if return_lse else O


def block_score(Q, Kc, H_kv=None, scale=None):
    """Per-block score of every prefix position (Eq. 4): [H_kv, N] float64, each row sums to 1."""
    Q, pq = _f32(Q); Kc, pk = _f32(Kc)
    H_q, B, d = Q.shape
    H_kv, N, _ = Kc.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    score = np.zeros((H_kv, N), dtype=np.float64)
    _load().oracle_block_score(pq, pk, H_q, H_kv, B, d, ctypes.c_int64(N), ctypes.c_double(scale),
                               score.ctypes.data_as(ctypes.c_void_p))
    return score


def topk(score, k):
    """Top-k positions per KV head by full sort.  Returns (idx [H_kv,k] int32 ascending, -1 padded; k_eff)."""
    score = np.ascontiguousarray(score, dtype=np.float64)
    H_kv, N = score.shape
    idx = np.empty((H_kv, k), dtype=np.int32)
    k_eff = min(k, N)
    for h in range(H_kv):
        k_eff = _load().oracle_topk(score[h].ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(N), int(k),
                                    idx[h].ctypes.data_as(ctypes.c_void_p))
    return idx, int(k_eff)


def sparse_block_attn(Q, Kc, Vc, Kb, Vb, idx, k_eff, scale=None):
    """Reuse step (Algorithm 1 Phase 2): attention over cache rows idx[h,:k_eff] plus the block's own keys."""
    Q, pq = _f32(Q); Kc, pk = _f32(Kc); Vc, pv = _f32(Vc); Kb, pkb = _f32(Kb); Vb, pvb = _f32(Vb)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    H_q, B, d = Q.shape
    H_kv, N, _ = Kc.shape
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    O = np.empty((H_q, B, d), dtype=np.float64)
    _load().oracle_sparse_block_attn(pq, pk, pv, pkb, pvb, idx.ctypes.data_as(ctypes.c_void_p), int(idx.shape[1]),
                                     int(k_eff), H_q, H_kv, B, d, ctypes.c_int64(N), ctypes.c_double(scale),
                                     O.ctypes.data_as(ctypes.c_void_p))
    return O


def recall(idx_ref, idx_other, k_eff):
    """Eq. 3: |S(1) ∩ S(tau)| / k per KV head, from two [H_kv, k] index arrays."""
    out = []
    for a, b in zip(np.asarray(idx_ref), np.asarray(idx_other)):
        out.append(len(set(a[:k_eff].tolist()) & set(b[:k_eff].tolist())) / max(1, k_eff))
    return np.array(out)


def run_block(q_steps, Kc, Vc, kb_steps, vb_steps, k, scale=None):
    """One block of Algorithm 1 on one problem: Step 1 exact + score + top-k, then T-1 reuse steps.

    q_steps [T,H_q,B,d], kb_steps/vb_steps [T,H_kv,B,d].  Returns dict with O_exact, score, idx, k_eff, O_sparse (list).
    """
    O1 = exact_block_attn(q_steps[0], Kc, Vc, kb_steps[0], vb_steps[0], scale)
    sc = block_score(q_steps[0], Kc, scale=scale)
    idx, k_eff = topk(sc, k)
    Os = [sparse_block_attn(q_steps[t], Kc, Vc, kb_steps[t], vb_steps[t], idx, k_eff, scale)
          for t in range(1, len(q_steps))]
    return {"O_exact": O1, "score": sc, "idx": idx, "k_eff": k_eff, "O_sparse": Os}


# ---------------------------------------------------------------------------------------------------------------------
# Quest-style page estimator in its per-block form (the paper's comparison system; Section 2.2 for the estimator,
# Section 3.1 / Eq. 2 for the per-block mean, Section 5 "Setup" for page size 16).  Plain NumPy in float64, written as
# the definitions read: per-channel extremes of each page, the sign-aware bound evaluated per query row with the max
# inside the sum over channels, then the mean over the block's G*B rows.
# ---------------------------------------------------------------------------------------------------------------------
def quest_page_summaries(Kc, page=16):
    """Per-channel min / max keys of each whole page (Section 2.2).  Kc [H_kv,N,d] -> (kmin, kmax) [H_kv, N // page, d]."""
    Kc = np.asarray(Kc, dtype=np.float64)
    H_kv, N, d = Kc.shape
    n_pages = N // page
    blocks = Kc[:, : n_pages * page].reshape(H_kv, n_pages, page, d)
    return blocks.min(axis=2), blocks.max(axis=2)


def quest_page_scores(Q, kmin, kmax):
    """Per-block page score: 1/(G B) * sum over g in group(h), q in block of sum_c max(Q[g,q,c] Kmax[c], Q[g,q,c] Kmin[c])
    (Section 2.2 for the inner bound; Eq. 2's per-block form with that bound as s).  Q [H_q,B,d] -> [H_kv, n_pages]."""
    Q = np.asarray(Q, dtype=np.float64)
    H_q, B, d = Q.shape
    H_kv, n_pages, _ = kmin.shape
    G = H_q // H_kv
    score = np.zeros((H_kv, n_pages))
    for h in range(H_kv):
        for g in range(h * G, (h + 1) * G):
            for qi in range(B):
                qv = Q[g, qi]                                             # [d]
                score[h] += np.maximum(qv[None, :] * kmax[h], qv[None, :] * kmin[h]).sum(axis=1)
    return score / (G * B)


def quest_select(Q, Kc, k, page=16):
    """The k/page best pages per KV head and their tokens.  Returns (idx [H_kv,k] int32 ascending, -1 padded; k_eff; page scores)."""
    kmin, kmax = quest_page_summaries(Kc, page)
    sc = quest_page_scores(Q, kmin, kmax)
    H_kv, n_pages = sc.shape
    k_pages = k // page
    idx = np.full((H_kv, k), -1, dtype=np.int32)
    n_sel = min(k_pages, n_pages)
    if n_pages > 0:
        pages, n_sel = topk(sc, k_pages)
        for h in range(H_kv):
            idx[h, : n_sel * page] = (pages[h, :n_sel, None].astype(np.int64) * page + np.arange(page)[None, :]).reshape(-1)
    return idx, n_sel * page, sc



# ---------------------------------------------------------------------------------------------------------------------
# Keys in 8 bits (the paper leaves cache compression to future work -- Limitations; this is this build's own definition
# of the variant, stated here in full because there is no passage to restate).
#
#   format     e4m3: 1 sign, 4 exponent bits (bias 7), 3 mantissa bits; no infinities, largest finite value 448,
#              smallest normal 2^-6, subnormals in steps of 2^-9
#   scale      one per (problem, KV head): s = fl32(amax / 448), amax = largest |x| of the head's rows (1 if amax = 0)
#   code       c = e4m3_rn_sat(fl32(x / s)): IEEE single division, then round to nearest even onto the e4m3 grid,
#              magnitudes beyond 448 (infinities included) clamp to 448, NaN stays NaN
#   keys       cache keys use the head's key scale s_k; the block's own keys use the same s_k (and so may clamp)
#   queries    the G*B query rows of a KV head share s_q, taken from those rows at every call
#   logits     s_q s_k * sum_c cq_c ck_c, everything after that as in the 16-bit path; values stay as they are
#
# So the variant is the unchanged method applied to the de-quantised queries and keys.  The functions below produce the
# codes (as float64 values on the e4m3 grid) and the scales; the k8_* wrappers run the by-definition routines above head
# by head on the codes with the head's s_q s_k folded into the softmax scale, so no value is rounded on the way in.
# ---------------------------------------------------------------------------------------------------------------------
E4M3_MAX = 448.0


def e4m3_round(y):
    """Nearest e4m3 value (ties to even, clamped to +-448, NaN kept) of each element; float64 in, float64 out."""
    y = np.asarray(y, dtype=np.float64)
    a = np.abs(y)
    with np.errstate(invalid="ignore", divide="ignore"):
        e = np.floor(np.log2(np.where((a > 0) & np.isfinite(a), a, 1.0)))
    e = np.maximum(e, -6.0)                      # below 2^-6 the grid is the subnormal one: step 2^-9
    step = np.exp2(e - 3.0)                      # 3 mantissa bits: 8 steps per binade
    q = np.rint(a / step) * step                 # np.rint rounds half to even
    q = np.where(np.isinf(a), E4M3_MAX, q)
    q = np.minimum(q, E4M3_MAX)
    return np.where(np.isnan(y), np.nan, np.copysign(q, y))


def k8_scale(x):
    """fl32(amax / 448) of an array (float32 arithmetic: the decision which code a value gets is taken in single precision)."""
    x = np.asarray(x, dtype=np.float32)
    amax = np.float32(np.nanmax(np.abs(x))) if x.size else np.float32(0)
    return np.float32(1) if not amax > 0 else np.float32(amax / np.float32(448))


def k8_codes(x, s):
    """e4m3 codes (as float64 grid values) of x under scale s: e4m3_rn_sat(fl32(x / s))."""
    x = np.asarray(x, dtype=np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        y = (x / np.float32(s)).astype(np.float32)
    return e4m3_round(y.astype(np.float64))


def k8_quantize_block(Q, Kc, Kb):
    """Codes and scales of one problem.  Q [H_q,B,d], Kc [H_kv,N,d], Kb [H_kv,B,d] ->
    (Q codes, Kc codes, Kb codes, s_q [H_kv], s_k [H_kv]); codes are float64 arrays of e4m3 grid values."""
    Q = np.asarray(Q, dtype=np.float32); Kc = np.asarray(Kc, dtype=np.float32); Kb = np.asarray(Kb, dtype=np.float32)
    H_q, H_kv = Q.shape[0], Kc.shape[0]
    G = H_q // H_kv
    s_q = np.array([k8_scale(Q[h * G:(h + 1) * G]) for h in range(H_kv)], dtype=np.float32)
    s_k = np.array([k8_scale(Kc[h]) for h in range(H_kv)], dtype=np.float32)
    Qc = np.concatenate([k8_codes(Q[h * G:(h + 1) * G], s_q[h]) for h in range(H_kv)], axis=0)
    Kcc = np.stack([k8_codes(Kc[h], s_k[h]) for h in range(H_kv)])
    Kbc = np.stack([k8_codes(Kb[h], s_k[h]) for h in range(H_kv)])
    return Qc, Kcc, Kbc, s_q, s_k


def _per_head(fn, Qc, s_q, s_k, scale, d, H_kv):
    G = Qc.shape[0] // H_kv
    scale = 1.0 / np.sqrt(d) if scale is None else scale
    return [fn(h, slice(h * G, (h + 1) * G), scale * float(s_q[h]) * float(s_k[h])) for h in range(H_kv)]


def k8_exact_block_attn(Qc, Kcc, Vc, Kbc, Vb, s_q, s_k, scale=None, return_lse=False):
    """exact_block_attn on 8-bit keys and queries: head by head on the codes, s_q s_k folded into the softmax scale."""
    H_kv = Kcc.shape[0]
    res = _per_head(lambda h, g, sc: exact_block_attn(Qc[g], Kcc[h:h + 1], Vc[h:h + 1], Kbc[h:h + 1], Vb[h:h + 1], sc, True),
                    Qc, s_q, s_k, scale, Qc.shape[-1], H_kv)
    O = np.concatenate([r[0] for r in res], axis=0)
    lse = np.concatenate([r[1] for r in res], axis=0)
    return (O, lse) if return_lse else O


def k8_block_score(Qc, Kcc, s_q, s_k, scale=None):
    """block_score (Eq. 4) on 8-bit keys and queries."""
    H_kv = Kcc.shape[0]
    res = _per_head(lambda h, g, sc: block_score(Qc[g], Kcc[h:h + 1], scale=sc), Qc, s_q, s_k, scale, Qc.shape[-1], H_kv)
    return np.concatenate(res, axis=0)


def k8_sparse_block_attn(Qc, Kcc, Vc, Kbc, Vb, idx, k_eff, s_q, s_k, scale=None):
    """sparse_block_attn on 8-bit keys and queries."""
    H_kv = Kcc.shape[0]
    res = _per_head(lambda h, g, sc: sparse_block_attn(Qc[g], Kcc[h:h + 1], Vc[h:h + 1], Kbc[h:h + 1], Vb[h:h + 1], idx[h:h + 1], k_eff, sc),
                    Qc, s_q, s_k, scale, Qc.shape[-1], H_kv)
    return np.concatenate(res, axis=0)
