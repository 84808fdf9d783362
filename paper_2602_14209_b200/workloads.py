"""Seeded synthetic inputs for the MAGE per-block attention path.

This module only draws random tensors and lays them out in memory (contiguous
or paged).  It contains none of the method's arithmetic (no attention, no
score, no selection), so both the CUDA path and the CPU oracle can be fed from
it without sharing any computation.

The inputs stand in for the long-context workloads the paper evaluates on
(Section 5: block size B = 32, budgets k in {256, 512, 1024}, contexts of
32K-128K tokens on Qwen2.5-7B / Llama-3-8B shaped attention layers).  The
recipe is the "planted heavy keys" construction:

* cache keys and values K, V ~ N(0, 1) per element;
* per KV head h a random unit direction u_h; ``n_heavy`` cache positions per
  head get the key 3 * u_h (their values stay N(0, 1));
* Step-1 queries  Q1[g, q] = 0.5 * u_{h(g)} + N(0, 1) / sqrt(d);
* Step-t queries  Qt = Q1 + N(0, 0.1^2), drawn independently for each step;
* block keys/values Kb1, Vb1 ~ N(0, 1); step t = step 1 + N(0, 0.1^2).

Everything is rounded to bf16 once, here, and the same bf16 bit patterns go to
both consumers.  Random streams are torch generators seeded per
(seed, problem, tensor); the bits depend on the generator's device, so one call
produces the data for both consumers of a test or benchmark.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and data recipe of one synthetic configuration."""

    name: str
    H_q: int
    H_kv: int
    N: int                      # prefix length (N_max when ragged)
    B: int = 32
    k: int = 512
    T: int = 8
    d: int = 128
    P: int = 1                  # independent problems (layers or sequences)
    n_heavy: int = 512
    cluster_frac: float = 0.0   # fraction of heavy positions in the last `cluster_window` tokens
    cluster_window: int = 4096
    ragged_min: int = 0         # >0: per-problem N log-uniform in [ragged_min, N]
    page_size: int = 0          # 0 = contiguous cache, else tokens per page
    seed: int = 0
    heavy_scale: float = 3.0    # planted heavy keys are heavy_scale * u_h
    q_align: float = 0.5        # Step-1 queries are q_align * u_h + N(0, 1) / sqrt(d)

    @property
    def G(self) -> int:
        return self.H_q // self.H_kv

    @property
    def M(self) -> int:
        return self.G * self.B


# The five configurations of the benchmark definition.
CONFIGS = {
    "cfg1_small": Workload("cfg1_small", H_q=8, H_kv=2, N=2048, B=32, k=256, T=4, n_heavy=64),
    "cfg2_qwen_32k": Workload("cfg2_qwen_32k", H_q=28, H_kv=4, N=32768, B=32, k=512, T=8),
    "cfg3_qwen_128k_x28": Workload("cfg3_qwen_128k_x28", H_q=28, H_kv=4, N=131072, B=32, k=512, T=8,
                                   P=28, cluster_frac=0.4),
    "cfg4_qwen_64k": Workload("cfg4_qwen_64k", H_q=28, H_kv=4, N=65536, B=32, k=512, T=8),
    "cfg5_llama_ragged_paged": Workload("cfg5_llama_ragged_paged", H_q=32, H_kv=8, N=131072, B=32, k=512,
                                        T=8, P=16, ragged_min=4096, page_size=64),
}
# Concentrated attention (an extra workload, not one of the five): the planted keys are far stronger (norm 45 against
# ~11 for an ordinary key) and the queries more aligned, so a planted key's softmax weight is ~e^8 times an ordinary key's
# and the 512 planted positions of a head hold ~90 % of the probability mass; 90 % of them lie in the last 4096 tokens.
# This is the regime the paper reports for trained models (a small set of positions carries the bulk of the mass), where
# the pruned selection has something to prune; on the flat recipe above nothing can be pruned.
CONFIGS["concentrated_qwen_128k_x28"] = dataclasses.replace(CONFIGS["cfg3_qwen_128k_x28"], name="concentrated_qwen_128k_x28",
                                                            heavy_scale=45.0, q_align=2.0, cluster_frac=0.9)
CFG4_K = (128, 256, 512, 1024, 2048)
CFG4_B = (4, 16, 32, 64)


def cfg4_variant(B: int, k: int) -> Workload:
    """One cell of the budget/block sweep: T = max(1, B / 4) steps."""
    return dataclasses.replace(CONFIGS["cfg4_qwen_64k"], name=f"cfg4_B{B}_k{k}", B=B, k=k, T=max(1, B // 4))


_TENSOR_IDS = {"kc": 1, "vc": 2, "u": 3, "heavy": 4, "q1": 5, "qdrift": 6, "kb1": 7, "vb1": 8,
               "kbdrift": 9, "vbdrift": 10, "seqlen": 11, "pages": 12}


def _gen(seed: int, problem: int, tensor: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + problem * 1009 + _TENSOR_IDS[tensor]) & 0x7FFFFFFFFFFF)
    return g


def seq_lens_for(w: Workload) -> List[int]:
    """Per-problem prefix lengths: N for all, or log-uniform in [ragged_min, N]."""
    if w.ragged_min <= 0:
        return [w.N] * w.P
    g = _gen(w.seed, 0, "seqlen", "cpu")
    u = torch.rand(w.P, generator=g, dtype=torch.float64)
    lo, hi = math.log(w.ragged_min), math.log(w.N)
    return [int(math.floor(math.exp(lo + (hi - lo) * float(x)))) for x in u]


def heavy_positions(w: Workload, problem: int, N: int) -> torch.Tensor:
    """[H_kv, n_heavy] distinct cache positions per head (CPU int64, sorted)."""
    g = _gen(w.seed, problem, "heavy", "cpu")
    n_heavy = min(w.n_heavy, N)
    out = []
    for _ in range(w.H_kv):
        n_cl = int(round(w.cluster_frac * n_heavy)) if N > w.cluster_window else 0
        chosen = torch.zeros(N, dtype=torch.bool)
        if n_cl > 0:
            tail = torch.randperm(w.cluster_window, generator=g)[:n_cl] + (N - w.cluster_window)
            chosen[tail] = True
        # the uniform part is drawn over all of N and skips positions already taken
        perm = torch.randperm(N, generator=g)
        perm = perm[~chosen[perm]][: n_heavy - n_cl]
        chosen[perm] = True
        out.append(torch.nonzero(chosen).flatten())
    return torch.stack(out)


def make_problem(w: Workload, problem: int = 0, N: Optional[int] = None, device="cpu", steps: Optional[int] = None):
    """Draw one problem (one layer / one sequence).

    Returns a dict of bf16 tensors on ``device``:
      kc, vc [H_kv, N, d];  q [T, H_q, B, d];  kb, vb [T, H_kv, B, d];
    plus ``heavy`` [H_kv, n_heavy] (CPU int64).  Index 0 of the T axis is Step 1.
    """
    N = w.N if N is None else N
    T = w.T if steps is None else steps
    d, dev = w.d, torch.device(device)
    f32 = dict(dtype=torch.float32, device=dev)
    kc = torch.randn(w.H_kv, N, d, generator=_gen(w.seed, problem, "kc", dev), **f32)
    vc = torch.randn(w.H_kv, N, d, generator=_gen(w.seed, problem, "vc", dev), **f32).to(torch.bfloat16)
    u = torch.randn(w.H_kv, d, generator=_gen(w.seed, problem, "u", "cpu"), dtype=torch.float32)
    u = (u / u.norm(dim=-1, keepdim=True)).to(dev)
    heavy = heavy_positions(w, problem, N) if N > 0 else torch.zeros(w.H_kv, 0, dtype=torch.int64)
    for h in range(w.H_kv):
        if heavy.shape[1]:
            kc[h, heavy[h].to(dev)] = w.heavy_scale * u[h]
    kc = kc.to(torch.bfloat16)
    u_q = u.repeat_interleave(w.G, dim=0)                       # [H_q, d]: head g uses u of KV head g // G
    q1 = w.q_align * u_q[:, None, :] + torch.randn(w.H_q, w.B, d, generator=_gen(w.seed, problem, "q1", dev), **f32) / math.sqrt(d)
    kb1 = torch.randn(w.H_kv, w.B, d, generator=_gen(w.seed, problem, "kb1", dev), **f32)
    vb1 = torch.randn(w.H_kv, w.B, d, generator=_gen(w.seed, problem, "vb1", dev), **f32)
    q, kb, vb = [q1], [kb1], [vb1]
    if T > 1:
        qd = torch.randn(T - 1, w.H_q, w.B, d, generator=_gen(w.seed, problem, "qdrift", dev), **f32) * 0.1
        kd = torch.randn(T - 1, w.H_kv, w.B, d, generator=_gen(w.seed, problem, "kbdrift", dev), **f32) * 0.1
        vd = torch.randn(T - 1, w.H_kv, w.B, d, generator=_gen(w.seed, problem, "vbdrift", dev), **f32) * 0.1
        for t in range(T - 1):
            q.append(q1 + qd[t]); kb.append(kb1 + kd[t]); vb.append(vb1 + vd[t])
    return {
        "kc": kc, "vc": vc,
        "q": torch.stack(q).to(torch.bfloat16), "kb": torch.stack(kb).to(torch.bfloat16),
        "vb": torch.stack(vb).to(torch.bfloat16), "heavy": heavy, "N": N,
    }


def make_batch(w: Workload, device="cpu", steps: Optional[int] = None, problems: Optional[List[int]] = None):
    """Draw all P problems of a workload into batched tensors.

    Returns a dict:
      kc, vc   [P, H_kv, N_max, d] bf16 (rows >= seq_lens[p] are zero), contiguous layout;
      q        [T, P, H_q, B, d];  kb, vb [T, P, H_kv, B, d];
      seq_lens [P] int32;  heavy: list of [H_kv, n_heavy] CPU tensors.
    ``problems`` restricts the batch to the listed problem ids (seeds stay those of the ids).
    """
    ids = list(range(w.P)) if problems is None else list(problems)
    lens_all = seq_lens_for(w)
    lens = [lens_all[i] for i in ids]
    T = w.T if steps is None else steps
    dev = torch.device(device)
    N_max = max(lens) if lens else 0
    kc = torch.zeros(len(ids), w.H_kv, N_max, w.d, dtype=torch.bfloat16, device=dev)
    vc = torch.zeros_like(kc)
    q = torch.empty(T, len(ids), w.H_q, w.B, w.d, dtype=torch.bfloat16, device=dev)
    kb = torch.empty(T, len(ids), w.H_kv, w.B, w.d, dtype=torch.bfloat16, device=dev)
    vb = torch.empty_like(kb)
    heavy = []
    for slot, (pid, n) in enumerate(zip(ids, lens)):
        pr = make_problem(w, pid, N=n, device=dev, steps=T)
        kc[slot, :, :n] = pr["kc"]; vc[slot, :, :n] = pr["vc"]
        q[:, slot] = pr["q"]; kb[:, slot] = pr["kb"]; vb[:, slot] = pr["vb"]
        heavy.append(pr["heavy"])
        del pr
    return {"kc": kc, "vc": vc, "q": q, "kb": kb, "vb": vb,
            "seq_lens": torch.tensor(lens, dtype=torch.int32, device=dev), "heavy": heavy, "N_max": N_max}


def to_paged(kc: torch.Tensor, vc: torch.Tensor, seq_lens, page_size: int, seed: int = 0, spare_pages: int = 3):
    """Scatter a contiguous [P, H_kv, N_max, d] cache into a page pool.

    Returns (k_pool, v_pool, block_table, max_pages): pools are
    [num_pages, H_kv, page_size, d] bf16, block_table is [P, max_pages] int32
    (logical page -> pool page; unused slots hold -1).  Pool pages are assigned
    by a seeded random permutation, so logical neighbours are not physical
    neighbours; the tail of each sequence's last page and a few spare pages are
    left filled with a non-zero pattern to show that they are never read.
    """
    P, H_kv, N_max, d = kc.shape
    lens = [int(x) for x in seq_lens]
    pages_per = [(n + page_size - 1) // page_size for n in lens]
    max_pages = max(1, max(pages_per) if pages_per else 1)
    total = sum(pages_per)
    num_pages = total + spare_pages
    g = _gen(seed, 0, "pages", "cpu")
    perm = torch.randperm(num_pages, generator=g)
    dev = kc.device
    k_pool = torch.full((num_pages, H_kv, page_size, d), 7.0, dtype=torch.bfloat16, device=dev)
    v_pool = torch.full((num_pages, H_kv, page_size, d), -7.0, dtype=torch.bfloat16, device=dev)
    table = torch.full((P, max_pages), -1, dtype=torch.int32)
    nxt = 0
    for p in range(P):
        n = lens[p]
        if pages_per[p] == 0:
            continue
        ids = perm[nxt: nxt + pages_per[p]]
        nxt += pages_per[p]
        table[p, : pages_per[p]] = ids.to(torch.int32)
        full = n // page_size
        ids_dev = ids.to(dev)
        if full:
            src_k = kc[p, :, : full * page_size].reshape(H_kv, full, page_size, d).permute(1, 0, 2, 3)
            src_v = vc[p, :, : full * page_size].reshape(H_kv, full, page_size, d).permute(1, 0, 2, 3)
            k_pool[ids_dev[:full]] = src_k
            v_pool[ids_dev[:full]] = src_v
        rem = n - full * page_size
        if rem:
            k_pool[ids_dev[full], :, :rem] = kc[p, :, full * page_size: n]
            v_pool[ids_dev[full], :, :rem] = vc[p, :, full * page_size: n]
    return k_pool, v_pool, table.to(dev), max_pages


def shard_by_kv_head(H_q: int, H_kv: int, world_size: int, rank: int):
    """KV-head sharding of one layer across ranks (no data-path collective).

    Returns (kv_head_slice, q_head_slice).  Every stage of the path is
    independent per KV head (the block score only sums inside a GQA group),
    so a rank that owns KV heads [a, b) needs query heads [a*G, b*G) and
    nothing from its peers.
    """
    if H_kv % world_size != 0:
        raise ValueError(f"H_kv={H_kv} is not divisible by world_size={world_size}")
    G = H_q // H_kv
    per = H_kv // world_size
    return slice(rank * per, (rank + 1) * per), slice(rank * per * G, (rank + 1) * per * G)


def shard_problems(P: int, world_size: int, rank: int) -> List[int]:
    """Round-robin split of independent problems (layers / sequences) across ranks."""
    return list(range(rank, P, world_size))


def shard_batch_by_kv_head(batch: dict, w: Workload, world_size: int, rank: int):
    """The slice of a `make_batch` result that rank `rank` of `world_size` owns under KV-head sharding.

    Returns (local_workload, local_batch).  The cache tensors are strided VIEWS of the full ones (head stride and problem
    stride unchanged: the library takes them as they are); queries, block keys and block values are small and are
    copied into the contiguous [.., H_local, B, d] layout the library expects.  Nothing here needs another rank's data.
    """
    hs, qs = shard_by_kv_head(w.H_q, w.H_kv, world_size, rank)
    local = dataclasses.replace(w, name=f"{w.name}[kv_heads {hs.start}:{hs.stop}]", H_q=qs.stop - qs.start, H_kv=hs.stop - hs.start)
    out = dict(batch)
    out["kc"], out["vc"] = batch["kc"][:, hs], batch["vc"][:, hs]
    out["q"] = batch["q"][:, :, qs].contiguous()
    out["kb"], out["vb"] = batch["kb"][:, :, hs].contiguous(), batch["vb"][:, :, hs].contiguous()
    out["heavy"] = [h[hs] for h in batch["heavy"]]
    return local, out

