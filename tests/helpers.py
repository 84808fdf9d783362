"""Shared test helpers: an independent NumPy brute force and bf16-exact random inputs."""
import numpy as np
import torch


def bf16_exact(rng, shape, scale=1.0):
    """float32 array whose values are exactly representable in bf16."""
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32) * scale)
    return x.to(torch.bfloat16).to(torch.float32).numpy()


def brute_force_block(Q, Kc, Vc, Kb, Vb, scale):
    """Explicit (N+B)-wide score matrices in float64; returns (O_exact, score).

    Written with whole-matrix NumPy expressions, independently of the C oracle's loops.
    """
    H_q, B, d = Q.shape
    H_kv, N, _ = Kc.shape
    G = H_q // H_kv
    Q, Kc, Vc, Kb, Vb = (a.astype(np.float64) for a in (Q, Kc, Vc, Kb, Vb))
    O = np.zeros((H_q, B, d))
    score = np.zeros((H_kv, N))
    for g in range(H_q):
        h = g // G
        K_all = np.concatenate([Kc[h], Kb[h]], axis=0)          # [N+B, d]
        V_all = np.concatenate([Vc[h], Vb[h]], axis=0)
        S = (Q[g] @ K_all.T) * scale                            # [B, N+B]
        Pm = np.exp(S - S.max(axis=1, keepdims=True))
        Pm /= Pm.sum(axis=1, keepdims=True)
        O[g] = Pm @ V_all
        if N:
            Sp = S[:, :N]
            A = np.exp(Sp - Sp.max(axis=1, keepdims=True))
            A /= A.sum(axis=1, keepdims=True)
            score[h] += A.sum(axis=0)
    return O, score / (G * B)


def brute_force_sparse(Q, Kc, Vc, Kb, Vb, idx, k_eff, scale):
    H_q, B, d = Q.shape
    H_kv = Kc.shape[0]
    G = H_q // H_kv
    Q, Kc, Vc, Kb, Vb = (a.astype(np.float64) for a in (Q, Kc, Vc, Kb, Vb))
    O = np.zeros((H_q, B, d))
    for g in range(H_q):
        h = g // G
        sel = idx[h, :k_eff]
        K_all = np.concatenate([Kc[h][sel], Kb[h]], axis=0)
        V_all = np.concatenate([Vc[h][sel], Vb[h]], axis=0)
        S = (Q[g] @ K_all.T) * scale
        Pm = np.exp(S - S.max(axis=1, keepdims=True))
        Pm /= Pm.sum(axis=1, keepdims=True)
        O[g] = Pm @ V_all
    return O


def brute_force_topk(score_row, k):
    """Positions of the k largest entries, ties to the smaller position, ascending output."""
    N = len(score_row)
    order = np.lexsort((np.arange(N), -score_row))             # primary: score desc, secondary: index asc
    return np.sort(order[: min(k, N)])
