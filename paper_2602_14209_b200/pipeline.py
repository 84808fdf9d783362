"""Per-block call sequence of Algorithm 1 on two CUDA streams (buffers, streams, events; no arithmetic).

Step 1 runs ``mage_exact_select`` on the main stream; ``mage_topk`` is enqueued on a
dedicated select stream behind an event, so whatever the caller puts on the main
stream next (the FFN in a model, other sequences' sparse steps in a serving
batch) overlaps it; the main stream joins once before the first reuse step.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch

from . import binding as mb


class BlockAttention:
    """Owns the outputs and scratch of one batch of problems and issues the three library calls."""

    def __init__(self, kv: mb.KVCache, k: int, sm_scale: Optional[float] = None, select_stream: Optional[torch.cuda.Stream] = None,
                 buffers: Optional[dict] = None, k8: Optional[mb.K8Keys] = None):
        """``buffers`` lets several instances (e.g. one per layer) live in slices of shared tensors: keys out, scores,
        indices, k_eff, status, workspace; anything missing is allocated here.  ``k8``: the cache's keys as 8-bit codes
        (already quantised); Step 1 and the reuse steps then go through the ``*_k8`` calls."""
        self.kv, self.k, self.k8 = kv, int(k), k8
        self.sm_scale = float(kv.d) ** -0.5 if sm_scale is None else float(sm_scale)
        dev = kv.device
        b = buffers or {}
        self.out = b["out"] if "out" in b else torch.empty(kv.P, kv.H_q, kv.B, kv.d, dtype=torch.bfloat16, device=dev)
        self.scores = b["scores"] if "scores" in b else torch.zeros(kv.P, kv.H_kv, max(kv.N_max, 1), dtype=torch.float32, device=dev)
        self.indices = b["indices"] if "indices" in b else torch.full((kv.P, kv.H_kv, self.k), -1, dtype=torch.int32, device=dev)
        self.k_eff = b["k_eff"] if "k_eff" in b else torch.zeros(kv.P, dtype=torch.int32, device=dev)
        self.status = b["status"] if "status" in b else torch.zeros(1, dtype=torch.int32, device=dev)
        self.workspace = b["workspace"] if "workspace" in b else kv.new_workspace(self.k)
        self.select_stream = select_stream if select_stream is not None else torch.cuda.Stream(device=dev)
        self._scores_ready = torch.cuda.Event()
        self._indices_ready = torch.cuda.Event()

    def exact_select(self, q, k_blk, v_blk, out=None, stream=None, events=None):
        """Step 1 on ``stream`` (default: current): exact attention -> out, block scores -> self.scores."""
        out = self.out if out is None else out
        if self.k8 is not None:
            mb.mage_exact_select_k8(self.kv, self.k8, q, k_blk, v_blk, self.sm_scale, out, self.scores, self.workspace, self.status,
                                    stream, events)
            return out
        mb.mage_exact_select(self.kv, q, k_blk, v_blk, self.sm_scale, out, self.scores, self.workspace, self.status, stream,
                             events)
        return out

    def exact_attn(self, q, k_blk, v_blk, out=None, stream=None):
        """Step 1's attention alone on ``stream`` (default: current); pair it with ``select_scores_async``."""
        out = self.out if out is None else out
        if self.k8 is not None:
            raise NotImplementedError("the two halves of Step 1 on their own exist for 16-bit keys only")
        mb.mage_exact_attn(self.kv, q, k_blk, v_blk, self.sm_scale, out, self.workspace, self.status, stream)
        return out

    def select_workspace(self) -> torch.Tensor:
        """The workspace the select stream's own score pass uses (allocated on first use): it may run while the main
        stream's Step 1 is using ``self.workspace``."""
        if getattr(self, "_select_workspace", None) is None:
            self._select_workspace = self.kv.new_workspace(self.k)
        return self._select_workspace

    def select_scores_async(self, q, workspace: Optional[torch.Tensor] = None, main_stream=None):
        """The paper's two-stream Phase 1: block scores and top-k on the select stream from the queries alone, beside
        whatever the main stream does (its attention, then the FFN).  Uses a workspace of its own (allocated on first use),
        since the main stream's Step 1 may be using ``self.workspace`` at the same time.  Follow with ``join()``."""
        if self.k8 is not None:
            raise NotImplementedError("the two halves of Step 1 on their own exist for 16-bit keys only")
        main = torch.cuda.current_stream() if main_stream is None else main_stream
        if workspace is None:
            workspace = self.select_workspace()
        self._scores_ready.record(main)                   # q is ready on the main stream
        self.select_stream.wait_event(self._scores_ready)
        mb.mage_select_scores(self.kv, q, self.sm_scale, self.scores, workspace, self.status, self.select_stream)
        mb.mage_topk(self.scores, self.kv.seq_lens, self.kv.P, self.kv.H_kv, max(self.kv.N_max, 0), self.k, self.indices,
                     self.k_eff, stream=self.select_stream)
        self._indices_ready.record(self.select_stream)

    def select_async(self, main_stream=None):
        """Top-k on the select stream, ordered after the scores written on ``main_stream``; does not block it."""
        main = torch.cuda.current_stream() if main_stream is None else main_stream
        self._scores_ready.record(main)
        self.select_stream.wait_event(self._scores_ready)
        mb.mage_topk(self.scores, self.kv.seq_lens, self.kv.P, self.kv.H_kv, max(self.kv.N_max, 0), self.k, self.indices,
                     self.k_eff, stream=self.select_stream)
        self._indices_ready.record(self.select_stream)

    def join(self, main_stream=None):
        """The single synchronisation at the end of Phase 1: the main stream waits for the index sets."""
        main = torch.cuda.current_stream() if main_stream is None else main_stream
        main.wait_event(self._indices_ready)

    def sparse_step(self, q, k_blk, v_blk, out=None, stream=None):
        """One reuse step (Phase 2) with the index sets fixed at Step 1."""
        out = self.out if out is None else out
        if self.k8 is not None:
            mb.mage_sparse_block_attn_k8(self.kv, self.k8, q, k_blk, v_blk, self.indices, self.k_eff, self.k, self.sm_scale, out,
                                         self.workspace, self.status, stream)
            return out
        mb.mage_sparse_block_attn(self.kv, q, k_blk, v_blk, self.indices, self.k_eff, self.k, self.sm_scale, out,
                                  self.workspace, self.status, stream)
        return out

    def run_block(self, q_steps: Sequence[torch.Tensor], kb_steps, vb_steps, outs: Optional[Sequence[torch.Tensor]] = None,
                  events=None):
        """One block: Step 1, asynchronous selection, join, then len(q_steps)-1 reuse steps.  Returns the outputs."""
        T = len(q_steps)
        res = []
        o = self.exact_select(q_steps[0], kb_steps[0], vb_steps[0], None if outs is None else outs[0], events=events)
        res.append(o)
        self.select_async()
        # joined even when no reuse step follows (T = 1): the index sets and k_eff are then ordered with respect to the main
        # stream for the caller, and the next block's Step 1 cannot overwrite the scores while top-k still reads them
        self.join()
        for t in range(1, T):
            res.append(self.sparse_step(q_steps[t], kb_steps[t], vb_steps[t], None if outs is None else outs[t]))
        return res


class HostStagedBlocks:
    """Blocks whose per-step inputs live in pinned host memory and whose outputs go back to pinned host memory.

    Two sets of device staging buffers alternate between consecutive blocks: the inputs of block n+1 cross PCIe while
    block n computes, and the outputs of block n leave while block n+1 computes.  Nothing here waits on the host;
    ``finish()`` does.  The prefix cache stays resident on the device (it is the state that block-level caching keeps).
    """

    def __init__(self, ba: BlockAttention, T: int, depth: int = 2):
        kv, dev = ba.kv, ba.kv.device
        self.ba, self.T, self.depth, self.n = ba, int(T), int(depth), 0
        mk = lambda *shape: torch.empty(*shape, dtype=torch.bfloat16, device=dev)
        self.q_s = [[mk(kv.P, kv.H_q, kv.B, kv.d) for _ in range(T)] for _ in range(depth)]
        self.kb_s = [[mk(kv.P, kv.H_kv, kv.B, kv.d) for _ in range(T)] for _ in range(depth)]
        self.vb_s = [[mk(kv.P, kv.H_kv, kv.B, kv.d) for _ in range(T)] for _ in range(depth)]
        self.out_s = [[mk(kv.P, kv.H_q, kv.B, kv.d) for _ in range(T)] for _ in range(depth)]
        self.h2d_stream, self.d2h_stream = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        self.ev_in = [[torch.cuda.Event() for _ in range(T)] for _ in range(depth)]
        self.ev_out = [[torch.cuda.Event() for _ in range(T)] for _ in range(depth)]
        self.ev_computed = [torch.cuda.Event() for _ in range(depth)]     # staging inputs of this set are no longer read
        self.ev_drained = [torch.cuda.Event() for _ in range(depth)]      # staging outputs of this set are on the host

    def h2d_bytes(self) -> int:
        return sum(t.numel() * 2 for t in self.q_s[0] + self.kb_s[0] + self.vb_s[0])

    def d2h_bytes(self) -> int:
        return sum(t.numel() * 2 for t in self.out_s[0])

    def submit(self, q_h: Sequence[torch.Tensor], kb_h, vb_h, out_h, main_stream=None):
        """Enqueue one block; returns immediately.  ``out_h[t]`` is valid after ``finish()`` (or a sync on d2h_stream)."""
        main = torch.cuda.current_stream() if main_stream is None else main_stream
        b, T, ba = self.n % self.depth, self.T, self.ba
        used_before = self.n >= self.depth
        self.n += 1
        if used_before:
            self.h2d_stream.wait_event(self.ev_computed[b])
        with torch.cuda.stream(self.h2d_stream):
            for t in range(T):
                self.q_s[b][t].copy_(q_h[t], non_blocking=True)
                self.kb_s[b][t].copy_(kb_h[t], non_blocking=True)
                self.vb_s[b][t].copy_(vb_h[t], non_blocking=True)
                self.ev_in[b][t].record(self.h2d_stream)
        if used_before:
            main.wait_event(self.ev_drained[b])
        with torch.cuda.stream(main):
            main.wait_event(self.ev_in[b][0])
            ba.exact_select(self.q_s[b][0], self.kb_s[b][0], self.vb_s[b][0], self.out_s[b][0])
            ba.select_async(main)
            self.ev_out[b][0].record(main)
            ba.join(main)
            for t in range(1, T):
                main.wait_event(self.ev_in[b][t])
                ba.sparse_step(self.q_s[b][t], self.kb_s[b][t], self.vb_s[b][t], self.out_s[b][t])
                self.ev_out[b][t].record(main)
            self.ev_computed[b].record(main)
        with torch.cuda.stream(self.d2h_stream):
            for t in range(T):
                self.d2h_stream.wait_event(self.ev_out[b][t])
                out_h[t].copy_(self.out_s[b][t], non_blocking=True)
            self.ev_drained[b].record(self.d2h_stream)

    def finish(self, main_stream=None):
        main = torch.cuda.current_stream() if main_stream is None else main_stream
        main.wait_stream(self.d2h_stream)
        main.wait_stream(self.ba.select_stream)
        main.synchronize()


class LayerwiseBlock:
    """One block of Algorithm 1 issued the way a model runs it: layer after layer.

    Step 1 walks the layers on the main stream (``mage_exact_select`` per layer) while each layer's ``mage_topk`` runs
    on the select stream behind it; one join; then every reuse step walks the layers again with one
    ``mage_sparse_block_attn`` per layer.  The batched tensors of a multi-layer workload are sliced per layer, so the
    per-layer calls see P = 1 descriptions of the same memory.
    """

    def __init__(self, k_cache: torch.Tensor, v_cache: torch.Tensor, H_q: int, B: int, k: int, seq_lens: torch.Tensor):
        P = k_cache.shape[0]
        dev = k_cache.device
        self.select_stream = torch.cuda.Stream(device=dev)
        self.P, self.k = P, k
        H_kv, N_max, d = k_cache.shape[1], k_cache.shape[2], k_cache.shape[3]
        self.out = torch.empty(P, H_q, B, d, dtype=torch.bfloat16, device=dev)
        self.scores = torch.zeros(P, H_kv, max(N_max, 1), dtype=torch.float32, device=dev)
        self.indices = torch.full((P, H_kv, k), -1, dtype=torch.int32, device=dev)
        self.k_eff = torch.zeros(P, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.layers = []
        workspace = None
        for l in range(P):
            kv = mb.KVCache(k_cache[l:l + 1], v_cache[l:l + 1], H_q, B, seq_lens=seq_lens[l:l + 1])
            if workspace is None:
                workspace = kv.new_workspace(k)          # the layers run one after another and share it
            self.layers.append(BlockAttention(kv, k, select_stream=self.select_stream, buffers={
                "out": self.out[l:l + 1], "scores": self.scores[l:l + 1], "indices": self.indices[l:l + 1],
                "k_eff": self.k_eff[l:l + 1], "status": self.status, "workspace": workspace}))

    def run_block(self, q_steps: Sequence[torch.Tensor], kb_steps, vb_steps, outs: Sequence[torch.Tensor]):
        """q_steps[t] is [P, H_q, B, d] (one slice per layer), likewise the block K/V and the outputs."""
        T = len(q_steps)
        for l, ba in enumerate(self.layers):
            ba.exact_select(q_steps[0][l:l + 1], kb_steps[0][l:l + 1], vb_steps[0][l:l + 1], outs[0][l:l + 1])
            ba.select_async()
        self.layers[-1].join()                           # the select stream is in order: its last event covers all layers
        for t in range(1, T):
            for l, ba in enumerate(self.layers):
                ba.sparse_step(q_steps[t][l:l + 1], kb_steps[t][l:l + 1], vb_steps[t][l:l + 1], outs[t][l:l + 1])
        return outs
