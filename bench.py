#!/usr/bin/env python
"""Benchmark of the MAGE per-block attention path: one "step" = one block of Algorithm 1
(Step-1 exact attention + block score, top-k on the select stream, T-1 sparse reuse steps)
over the 28-layer, 128K-context Qwen2.5-7B-shaped workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mage|reference] [--workload NAME] [--simt]

Prints one JSON line (rank 0).  With --impl reference the CPU oracle is timed on the host
cores on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "per_block_attention_latency"
UNIT = "ms/block"
SM_COUNT, FP32_LANES_PER_SM = 148, 128


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"], "bf16_tflops_sustained": p["bf16_tflops_sustained"],
                "sm_max_mhz": p.get("sm_max_mhz", 1965.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event (throttle) reasons through NVML every few ms while the timed region runs.

    Read-only queries; nothing on the GPU is changed.  Falls back to one `nvidia-smi` query if NVML is unavailable.
    """
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self._stop_evt = index, period_s, [], threading.Event()
        self.max_mhz, self.nvml = None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nvml = pynvml
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nvml = None

    def run(self):
        if self.nvml is None:
            return
        n = self.nvml
        while not self._stop_evt.is_set():
            try:
                mhz = n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)
                try:
                    mask = n.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
                except Exception:
                    mask = n.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
                try:
                    watts = n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0
                except Exception:
                    watts = 0.0
                self.samples.append((float(mhz), int(mask), watts))
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.nvml is not None:
            self.join(timeout=1.0)
        if not self.samples:
            try:
                out = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits", "-i",
                                      str(self.index)], capture_output=True, text=True, timeout=10).stdout.split(",")
                return {"sm_mhz": float(out[0]), "sm_max_mhz": float(out[1]), "reasons": [], "samples": 1, "source": "nvidia-smi after the run"}
            except Exception:
                return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm = sorted(x[0] for x in self.samples)
        reasons = [name for name, bit in self.REASONS if any(x[1] & bit for x in self.samples)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples), "power_w_max": max(x[2] for x in self.samples), "source": "nvml"}


def stage_bytes_flops(w, lens, key_bytes=2):
    """Algorithmic traffic and work of each stage for one block (all problems).

    Stage 1 must read every cached K and V row once (512 B per cached token per KV head), Q and the block's K/V,
    and write O and one fp32 score per cached token per KV head.  Its work is a dense (G*B) x N x d contraction
    done for the attention (QK^T and PV: 4*M*d flops per cached token per KV head) and once more for the score's
    QK^T (2*M*d).  Stage 3 gathers k rows of K and V per KV head and reads/writes Q, O, the block's K/V and indices.
    """
    d, M = w.d, w.M
    tok = sum(lens)
    qo = len(lens) * w.H_q * w.B * d * 2
    kvb = len(lens) * w.H_kv * w.B * d * 2 * 2
    row = d * key_bytes + d * 2                                     # one cached token of one KV head: its key and its value
    s1_bytes = tok * w.H_kv * (row + 4) + 2 * qo + kvb
    s1_attn_bytes = tok * w.H_kv * row + qo + kvb                   # the attention kernel alone
    s1_flops_attn = sum(4 * M * (n + w.B) * d * w.H_kv for n in lens)
    s1_flops_score = sum(2 * M * n * d * w.H_kv for n in lens)
    keff = [min(w.k, n) for n in lens]
    s3_bytes = sum(ke * w.H_kv * (row + 4) for ke in keff) + 2 * qo + kvb
    s3_flops = sum(4 * M * (ke + w.B) * d * w.H_kv for ke in keff)
    return {"s1_bytes": s1_bytes, "s1_attn_bytes": s1_attn_bytes, "s1_flops_attn": s1_flops_attn,
            "s1_flops_score": s1_flops_score, "s3_bytes": s3_bytes, "s3_flops": s3_flops}


def config_of(w, lens, world, kernels, parallelism=None, key_bytes=2):
    """The `config` object of the JSON line; both arms print the same keys."""
    return {"workload": w.name, "H_q": w.H_q, "H_kv": w.H_kv, "d": w.d, "N": w.N, "B": w.B, "k": w.k, "T": w.T,
            "problems": w.P, "cached_tokens": sum(lens), "kv_bytes": sum(lens) * w.H_kv * (w.d * key_bytes + w.d * 2),
            "l2_policy": "inputs_larger_than_l2 (KV cache streamed every step evicts L2)",
            "parallelism": parallelism or f"replicas x{world} (independent blocks, no collective)", "kernels": kernels}


def spawn_ranks_if_needed(args):
    """`python bench.py --gpus N` (N > 1) outside torchrun: start the N ranks here, one per GPU, over 127.0.0.1."""
    if args.gpus <= 1 or "WORLD_SIZE" in os.environ or args.impl == "reference":
        return
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def bootstrap_only(args):
    """Rank bootstrap and the max-over-ranks reduction alone (no kernels): what the N-rank launch path does around the
    timed region.  Uses NCCL when every rank has a GPU, gloo otherwise, so it also runs on a CPU-only box."""
    import torch
    import torch.distributed as dist
    rank, world, local_rank = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))
    use_cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    if world > 1:
        if use_cuda:
            torch.cuda.set_device(local_rank)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group("gloo")
    dev = torch.device("cuda", local_rank) if use_cuda else torch.device("cpu")
    t = torch.tensor([float(rank + 1)], dtype=torch.float64, device=dev)      # stands in for this rank's elapsed time
    if world > 1:
        dist.barrier()
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        print(json.dumps({"bootstrap_only": True, "n_gpus": world, "max_over_ranks": float(t[0]),
                          "backend": ("nccl" if use_cuda else "gloo") if world > 1 else None}))
    if world > 1:
        dist.destroy_process_group()


def run_reference(args, w):
    """The CPU oracle, as it stands, on a bounded sample: one KV head of one layer per step, scaled to the whole block."""
    import numpy as np
    import oracle
    from paper_2602_14209_b200 import workloads as W
    oracle.build()
    lens = W.seq_lens_for(w)
    p = max(range(w.P), key=lambda i: lens[i]) if w.ragged_min else 0
    pr = W.make_problem(w, p, N=lens[p], device="cpu")
    f = lambda t: t.float().numpy()
    q = [f(pr["q"][t]) for t in range(w.T)]
    kb = [f(pr["kb"][t]) for t in range(w.T)]
    vb = [f(pr["vb"][t]) for t in range(w.T)]
    Kc, Vc = f(pr["kc"]), f(pr["vc"])
    head_tokens = lens[p]
    all_head_tokens = sum(lens)
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        oracle.run_block(q, Kc, Vc, kb, vb, w.k)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            times.append(dt)
    per_sample = sum(times) / len(times)
    # the exact pass dominates and is linear in cached tokens x KV heads: scale the sample to the whole block
    ms_block = per_sample * 1e3 * all_head_tokens / head_tokens
    cores = oracle.num_threads()
    sample = (f"problem {p} (one layer/sequence, all {w.H_kv} KV heads, N={head_tokens}) of {w.name}: exact + score + top-k + "
              f"{w.T - 1} sparse steps; scaled to the whole block by cached tokens ({all_head_tokens / head_tokens:.1f}x)")
    scale = all_head_tokens / head_tokens
    line = {"impl": "reference", "metric": METRIC, "value": ms_block, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_block, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "extrapolated": scale != 1.0, "scale": scale,
            "config": config_of(w, lens, 1, "cpu oracle"),
            "cpu_baseline": {"value": ms_block, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                             "sample_seconds": per_sample, "extrapolated": scale != 1.0, "scale": scale},
            "e2e": {"value": ms_block, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="mage", choices=["mage", "reference"])
    ap.add_argument("--workload", default="cfg3_qwen_128k_x28")
    ap.add_argument("--simt", action="store_true", help="force the portable CUDA-core kernels")
    ap.add_argument("--P", type=int, default=None, help="override the number of problems (layers/sequences) of the workload")
    ap.add_argument("--N", type=int, default=None, help="override the prefix length of the workload")
    ap.add_argument("--ragged-min", type=int, default=None,
                    help="override the lower bound of the per-sequence prefix lengths (0 = every sequence has N tokens)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "kv_head"],
                    help="N > 1: replicas = every rank runs its own block (weak scaling); kv_head = the ranks split the KV heads of ONE "
                         "block between them, no collective on the data path (strong scaling)")
    ap.add_argument("--keys", default="bf16", choices=["bf16", "e4m3"],
                    help="e4m3: the variant with keys and queries as 8-bit codes (values bf16), timed the same way; no stage breakdown, "
                         "no CPU leg; the default line and every number quoted for the metric are bf16")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stage-breakdown", action="store_true")
    ap.add_argument("--bootstrap-only", action="store_true", help="start the ranks, reduce a stand-in time over them and exit (no kernels)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    spawn_ranks_if_needed(args)
    if args.bootstrap_only:
        bootstrap_only(args)
        return

    from paper_2602_14209_b200 import workloads as W
    w = W.CONFIGS[args.workload]
    if args.P is not None or args.N is not None:
        import dataclasses as _dc
        w = _dc.replace(w, P=args.P or w.P, N=args.N or w.N, name=f"{w.name}[P={args.P or w.P},N={args.N or w.N}]")
    if args.ragged_min is not None:
        import dataclasses as _dc
        w = _dc.replace(w, ragged_min=args.ragged_min, name=f"{w.name}[ragged_min={args.ragged_min}]")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            args.steps, args.warmup = min(args.steps, 3), min(args.warmup, 1)
            run_reference(args, w)
        return

    import torch
    import torch.distributed as dist
    from paper_2602_14209_b200 import binding as mb
    from paper_2602_14209_b200.pipeline import BlockAttention
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "VERSION")      # the communicator's own line in the log says what carried the barrier
        dist.init_process_group("nccl", device_id=dev)
    mb.load()
    peaks = load_peaks()

    # weak scaling: every rank runs its own block of the same shape on its own seeded data (independent problems,
    # no data-path collective); rank r draws seed + r.
    import dataclasses
    kv_head_sharded = args.shard == "kv_head" and world > 1
    w_full = w
    if kv_head_sharded:
        # strong scaling: ONE block; rank r owns KV heads [r*H_kv/W, (r+1)*H_kv/W) of every layer and their G query heads.
        # Every stage is independent per KV head (Eq. 2 / Eq. 4 sum only inside group(h)): no data-path collective.
        if w.page_size:
            raise SystemExit("--shard kv_head is implemented for contiguous caches")
        batch = W.make_batch(w, device=dev)                                   # same seed on every rank: the same block
        w, batch = W.shard_batch_by_kv_head(batch, w, world, rank)             # strided views of the cache, no copy
    else:
        w_rank = dataclasses.replace(w, seed=w.seed + rank)
        batch = W.make_batch(w_rank, device=dev)
    lens = [int(x) for x in batch["seq_lens"].tolist()]
    flags = mb.FLAG_SIMT_KERNELS if args.simt else 0
    if w.page_size:
        k_pool, v_pool, table, _ = W.to_paged(batch["kc"], batch["vc"], lens, w.page_size, seed=w.seed)
        batch["kc"] = batch["vc"] = None
        kv = mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"], block_table=table, N_max=batch["N_max"], flags=flags)
    else:
        kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"], flags=flags)
    k8_keys = None
    if args.keys == "e4m3":
        if args.simt or kv_head_sharded:
            raise SystemExit("--keys e4m3 runs on the tensor-core kernels, unsharded")
        k8_keys = mb.K8Keys(kv).quantize()              # one-off coding of the cache, outside the timed regions
        args.no_stage_breakdown = args.no_cpu_baseline = True
    ba = BlockAttention(kv, w.k, k8=k8_keys)
    T = w.T
    q_d = [batch["q"][t] for t in range(T)]
    kb_d = [batch["kb"][t] for t in range(T)]
    vb_d = [batch["vb"][t] for t in range(T)]
    outs = [torch.empty_like(ba.out) for _ in range(T)]
    sf = stage_bytes_flops(w, lens, key_bytes=1 if k8_keys is not None else 2)
    main_stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region 1: inputs resident in HBM ---------------------------------------------------------------
    n_total = args.warmup + args.steps
    ev_sets = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(n_total)]
    for i in range(args.warmup):
        ba.run_block(q_d, kb_d, vb_d, outs, events=ev_sets[i])
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    launches0 = mb.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        ba.run_block(q_d, kb_d, vb_d, outs, events=ev_sets[args.warmup + i])
    e1.record()
    barrier()
    launches = mb.launch_count() - launches0
    clocks = sampler.stop()
    ms_total = e0.elapsed_time(e1)
    attn_ms = [s[0].elapsed_time(s[1]) for s in ev_sets[args.warmup:]]
    comb_ms = [s[1].elapsed_time(s[2]) for s in ev_sets[args.warmup:]]
    score_ms = [s[2].elapsed_time(s[3]) for s in ev_sets[args.warmup:]]
    status = int(ba.status.item())

    # ---- timed region 2: end to end through the public API with host buffers ------------------------------------
    # Per block the host hands over each step's Q and block K/V (pinned) and reads back each step's output;
    # the prefix KV cache is resident state of the serving process, as in the paper's exact block-level caching.
    q_h = [t.cpu().pin_memory() for t in q_d]
    kb_h = [t.cpu().pin_memory() for t in kb_d]
    vb_h = [t.cpu().pin_memory() for t in vb_d]
    out_h = [torch.empty_like(o, device="cpu").pin_memory() for o in outs]

    # pipeline.HostStagedBlocks: copies run on their own streams and two sets of staging buffers alternate, so block
    # n+1's inputs arrive, and block n's outputs leave, while the other block computes; every byte still crosses PCIe
    # inside the timed region and the region ends with all outputs on the host.
    from paper_2602_14209_b200.pipeline import HostStagedBlocks
    staged = HostStagedBlocks(ba, T)
    h2d, d2h = staged.h2d_bytes(), staged.d2h_bytes()

    def e2e_block():
        staged.submit(q_h, kb_h, vb_h, out_h, main_stream)

    e2e_steps = args.steps
    for _ in range(min(args.warmup, 2)):
        e2e_block()
    staged.finish(main_stream)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(e2e_steps):
        e2e_block()
    staged.finish(main_stream)                       # the last block's outputs are on the host before the clock stops
    f1.record()
    barrier()
    e2e_ms_total = f0.elapsed_time(f1)

    # ---- max over ranks ----------------------------------------------------------------------------------------
    if world > 1:
        tt = torch.tensor([ms_total, e2e_ms_total], device=dev, dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_total, e2e_ms_total = float(tt[0]), float(tt[1])
        lt = torch.tensor([launches], device=dev, dtype=torch.int64)
        dist.all_reduce(lt)
        launches = int(lt[0])
    ms_per_step = ms_total / args.steps
    if kv_head_sharded:
        value, e2e_value = ms_per_step, e2e_ms_total / e2e_steps          # one block per step for the whole job
    else:
        value = ms_per_step / world             # ms per block over the whole job: each of the N ranks finishes one block per step
        e2e_value = e2e_ms_total / e2e_steps / world

    # ---- per-stage numbers (rank 0, outside the headline region): sparse step cold/warm, top-k alone -------------
    stages = {}
    if rank == 0 and not args.no_stage_breakdown:
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

        def timed(fn, cold, reps=10):
            ts = []
            for _ in range(reps):
                if cold:
                    flush.fill_(1)
                a.record(); fn(); b.record(); torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            ts.sort()
            return ts[len(ts) // 2]

        sp = lambda: ba.sparse_step(q_d[1], kb_d[1], vb_d[1], outs[1])
        tk = lambda: mb.mage_topk(ba.scores, kv.seq_lens, kv.P, kv.H_kv, kv.N_max, w.k, ba.indices, ba.k_eff)
        sp(); tk(); torch.cuda.synchronize()
        sp_cold, sp_warm, tk_ms = timed(sp, True), timed(sp, False), timed(tk, False)
        s1_ms = (sum(attn_ms) + sum(comb_ms) + sum(score_ms)) / len(attn_ms)

        # Phase 1 as the paper arranges it (attention on the main stream; scores from Q and the cached keys plus top-k on the
        # select stream; one join) against the fused form timed above (one call shares the rows' log-sum-exp).
        def fused_phase1():
            ba.exact_select(q_d[0], kb_d[0], vb_d[0], outs[0]); ba.select_async(); ba.join()

        def two_stream_phase1():
            ba.select_scores_async(q_d[0]); ba.exact_attn(q_d[0], kb_d[0], vb_d[0], outs[0]); ba.join()

        sel_alone = lambda: mb.mage_select_scores(kv, q_d[0], ba.sm_scale, ba.scores, ba.select_workspace(), ba.status)
        two_stream_phase1(); torch.cuda.synchronize()
        p1_fused, p1_two, sel_ms = timed(fused_phase1, False, 5), timed(two_stream_phase1, False, 5), timed(sel_alone, False, 5)
        stages = {
            "phase1_fused_ms": p1_fused, "phase1_two_stream_ms": p1_two, "select_scores_ms_alone": sel_ms,
            "exact_select_ms": s1_ms, "attn_kernel_ms": sum(attn_ms) / len(attn_ms), "combine_kernel_ms": sum(comb_ms) / len(comb_ms),
            "score_kernel_ms": sum(score_ms) / len(score_ms),
            "exact_select_gbs": sf["s1_bytes"] / s1_ms / 1e6, "exact_select_frac_of_8tbs": sf["s1_bytes"] / s1_ms / 1e6 / 8000.0,
            "exact_select_frac_of_measured_hbm": sf["s1_bytes"] / s1_ms / 1e6 / peaks["hbm_gbs"],
            "exact_select_tflops": (sf["s1_flops_attn"] + sf["s1_flops_score"]) / s1_ms / 1e9,
            "topk_ms_alone": tk_ms, "sparse_step_ms_cold_l2": sp_cold, "sparse_step_ms_warm_l2": sp_warm,
            "sparse_step_gbs_cold": sf["s3_bytes"] / sp_cold / 1e6, "sparse_step_frac_of_8tbs_cold": sf["s3_bytes"] / sp_cold / 1e6 / 8000.0,
            "sparse_step_frac_of_measured_hbm_cold": sf["s3_bytes"] / sp_cold / 1e6 / peaks["hbm_gbs"],
            "sparse_step_tflops_cold": sf["s3_flops"] / sp_cold / 1e9,
            "hbm_roofline_ms_block_at_8tbs": (sf["s1_bytes"] + (T - 1) * sf["s3_bytes"]) / 8e9,
        }
        # Step 1 + selection with the score pass restricted to the tiles that can hold a selected key, beside the plain pair
        # (exact_select + top-k, same stream).  On flat attention nothing can be pruned and the call pays its bookkeeping.
        pw = mb.pruned_workspace(kv, w.k)
        p_idx, p_keff, p_tiles = torch.empty_like(ba.indices), torch.empty_like(ba.k_eff), torch.zeros(kv.P, kv.H_kv, dtype=torch.int32, device=dev)
        pruned = lambda: mb.mage_exact_select_pruned(kv, q_d[0], kb_d[0], vb_d[0], ba.sm_scale, w.k, outs[0], ba.scores, p_idx, p_keff, pw,
                                                     tiles_scored=p_tiles, dev_status=ba.status)
        plain = lambda: (ba.exact_select(q_d[0], kb_d[0], vb_d[0], outs[0]), tk())
        plain(); torch.cuda.synchronize()
        idx_plain = ba.indices.clone()
        pruned(); torch.cuda.synchronize()
        tiles_all = sum((n + 127) // 128 for n in lens) * w.H_kv
        stages["pruned_select_ms"], stages["plain_select_ms_same_stream"] = timed(pruned, False, 5), timed(plain, False, 5)
        stages["pruned_tiles_scored_frac"] = float(p_tiles.sum().item()) / max(1, tiles_all)
        stages["pruned_same_index_sets"] = bool(torch.equal(p_idx, idx_plain))
        del pw
        # The paper's comparison system on the same inputs: a Quest-style page estimator (16-token pages) re-estimated at
        # every step = page scores + page top-k + index expansion, then the same reuse-step kernel on its index set.
        if w.k % mb.QUEST_PAGE == 0 and kv.N_max >= mb.QUEST_PAGE:
            n_pg = (kv.N_max + mb.QUEST_PAGE - 1) // mb.QUEST_PAGE
            pmin = torch.empty(kv.P, kv.H_kv, n_pg, kv.d, dtype=torch.bfloat16, device=dev)
            pmax = torch.empty_like(pmin)
            psc = torch.empty(kv.P, kv.H_kv, n_pg, dtype=torch.float32, device=dev)
            q_idx, q_keff, q_ws = torch.empty_like(ba.indices), torch.empty_like(ba.k_eff), mb.quest_workspace(kv, w.k)
            qb = lambda: mb.mage_quest_build(kv, pmin, pmax, ba.status)
            qs = lambda: mb.mage_quest_select(kv, q_d[1], pmin, pmax, w.k, psc, q_idx, q_keff, q_ws)
            qb(); qs(); torch.cuda.synchronize()
            qsp = lambda: mb.mage_sparse_block_attn(kv, q_d[1], kb_d[1], vb_d[1], q_idx, q_keff, w.k, ba.sm_scale, outs[1], ba.workspace, ba.status)
            stages["quest_build_ms"] = timed(qb, True, 5)
            stages["quest_select_ms_cold_l2"] = timed(qs, True, 5)
            stages["quest_step_ms_cold_l2"] = stages["quest_select_ms_cold_l2"] + timed(qsp, True, 5)
            stages["quest_summary_bytes"] = 2 * pmin.numel() * 2
            del pmin, pmax, psc
        # Step 1 and the reuse step with the keys (and queries) in 8 bits, beside the 16-bit calls, alternating so that both see
        # the same clocks; agreement of the two selections (|S_8 & S_16| / k, mean over heads).  Not part of the headline.
        try:
            k8 = mb.K8Keys(kv)
            stages["k8_quantize_cache_ms"] = timed(lambda: k8.quantize(0, ba.status), False, 3)
            s16 = lambda: mb.mage_exact_select(kv, q_d[0], kb_d[0], vb_d[0], ba.sm_scale, outs[0], ba.scores, ba.workspace, ba.status)
            s8 = lambda: mb.mage_exact_select_k8(kv, k8, q_d[0], kb_d[0], vb_d[0], ba.sm_scale, outs[0], ba.scores, ba.workspace, ba.status)
            t16, t8 = [], []
            for _ in range(5):
                t16.append(timed(s16, False, 1)); t8.append(timed(s8, False, 1))
            stages["exact_select_ms_alternating"], stages["k8_exact_select_ms_alternating"] = sorted(t16)[2], sorted(t8)[2]
            s16(); tk(); torch.cuda.synchronize()
            idx16, out16 = ba.indices.clone(), outs[0].float()
            s8(); tk(); torch.cuda.synchronize()
            diff = (outs[0].float() - out16).abs()
            stages["k8_step1_output_vs_16bit_max_abs"], stages["k8_step1_output_vs_16bit_mean_abs"] = float(diff.max()), float(diff.mean())
            stages["k8_step1_output_rms_16bit"] = float(out16.pow(2).mean().sqrt())
            del out16, diff
            same = 0
            for p_ in range(kv.P):
                for h_ in range(kv.H_kv):
                    same += len(set(idx16[p_, h_].tolist()) & set(ba.indices[p_, h_].tolist()) - {-1})
            stages["k8_selection_overlap_with_16bit"] = same / max(1, int(ba.k_eff.sum().item()) * kv.H_kv)
            sp8 = lambda: mb.mage_sparse_block_attn_k8(kv, k8, q_d[1], kb_d[1], vb_d[1], ba.indices, ba.k_eff, w.k, ba.sm_scale, outs[1], ba.workspace, ba.status)
            sp8(); torch.cuda.synchronize()
            stages["k8_sparse_step_ms_cold_l2"] = timed(sp8, True)
            stages["k8_key_bytes_per_token_head"] = 128
            del k8
            s16(); tk(); torch.cuda.synchronize()          # leave the 16-bit selection in place for what follows
        except mb.MageError as e:                          # a description the 8-bit calls do not take
            stages["k8_unavailable"] = str(e)
        del flush
        # The same block issued layer by layer, as a model would (config 3 "timed back-to-back"): one exact_select, one
        # top-k (select stream) and T-1 sparse launches per layer; plain launches, and replayed from a CUDA graph.
        if not w.page_size and w.P > 1:
            from paper_2602_14209_b200.pipeline import LayerwiseBlock
            lw = LayerwiseBlock(batch["kc"], batch["vc"], w.H_q, w.B, w.k, batch["seq_lens"])
            for _ in range(2):
                lw.run_block(q_d, kb_d, vb_d, outs)
            torch.cuda.synchronize()
            reps = 5
            a.record()
            for _ in range(reps):
                lw.run_block(q_d, kb_d, vb_d, outs)
            b.record(); torch.cuda.synchronize()
            stages["layerwise_ms_per_block"] = a.elapsed_time(b) / reps
            try:
                g = torch.cuda.CUDAGraph()
                cap = torch.cuda.Stream()
                cap.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(cap):
                    with torch.cuda.graph(g, stream=cap):
                        lw.run_block(q_d, kb_d, vb_d, outs)
                torch.cuda.current_stream().wait_stream(cap)
                g.replay(); torch.cuda.synchronize()
                a.record()
                for _ in range(reps):
                    g.replay()
                b.record(); torch.cuda.synchronize()
                stages["layerwise_cuda_graph_ms_per_block"] = a.elapsed_time(b) / reps
            except Exception as e:      # capture is an optimisation of the launch path only
                stages["layerwise_cuda_graph_ms_per_block"] = None
                stages["layerwise_cuda_graph_error"] = str(e)[:200]
            stages["layerwise_dev_status"] = int(lw.status.item())

        # Serving batch (ragged, paged): one scheduler tick with the sequences staggered over the T steps of a block.
        # Two sequences are at Step 1 (exact_select on the main stream, their top-k on the select stream), the other
        # fourteen take a reuse step on the main stream meanwhile.  Reported with the top-k overlapped and, for
        # comparison, with everything serialised on the main stream.
        if w.page_size and w.P >= 4:
            n1 = max(1, w.P // T)
            idx1 = torch.arange(0, n1, device=dev)
            idx2 = torch.arange(n1, w.P, device=dev)
            sub = lambda idx: mb.KVCache(k_pool, v_pool, w.H_q, w.B, seq_lens=batch["seq_lens"][idx].contiguous(),
                                         block_table=table[idx].contiguous(), N_max=batch["N_max"], flags=flags)
            ba1, ba2 = BlockAttention(sub(idx1), w.k), BlockAttention(sub(idx2), w.k)
            q1, kb1, vb1 = q_d[0][:n1].contiguous(), kb_d[0][:n1].contiguous(), vb_d[0][:n1].contiguous()
            q2, kb2, vb2 = q_d[1][n1:].contiguous(), kb_d[1][n1:].contiguous(), vb_d[1][n1:].contiguous()
            ba2.run_block([q2, q2], [kb2, kb2], [vb2, vb2])          # gives group 2 a valid index set
            torch.cuda.synchronize()

            def tick(overlap):
                ba1.exact_select(q1, kb1, vb1)
                if overlap:
                    ba1.select_async()
                else:
                    mb.mage_topk(ba1.scores, ba1.kv.seq_lens, ba1.kv.P, ba1.kv.H_kv, ba1.kv.N_max, w.k, ba1.indices, ba1.k_eff)
                ba2.sparse_step(q2, kb2, vb2)
                if overlap:
                    ba1.join()

            for mode in (True, False):
                for _ in range(3):
                    tick(mode)
                torch.cuda.synchronize()
                a.record()
                for _ in range(20):
                    tick(mode)
                b.record(); torch.cuda.synchronize()
                stages["serving_tick_ms_topk_on_select_stream" if mode else "serving_tick_ms_serialised"] = a.elapsed_time(b) / 20
            stages["serving_tick_groups"] = f"{n1} sequences at Step 1 + {w.P - n1} at a reuse step"

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the Step-1 attention kernel) -------------------------------------------
    # Which measured bf16 peak applies depends on the regime the run was in: a short run at full clock with no power
    # cap sampled is the burst regime; under sw_power_cap (or with the SM clock well below its maximum) the sustained one.
    attn_avg_ms = sum(attn_ms) / len(attn_ms)
    burst_regime = (clocks.get("sm_mhz") or 0) >= 0.95 * (clocks.get("sm_max_mhz") or 1e9) and "sw_power_cap" not in clocks.get("reasons", [])
    if args.simt:
        peak = SM_COUNT * FP32_LANES_PER_SM * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12
        roofline = {"bound": "alu", "kernel": "simt::attn_kernel<kExactPartial>", "achieved": sf["s1_flops_attn"] / attn_avg_ms / 1e9,
                    "peak": peak, "unit": "TFLOP/s", "peak_source": "148 SMs x 128 fp32 lanes x 2 flop x 1965 MHz (derived)",
                    "traffic": None}
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
    else:
        achieved = sf["s1_flops_attn"] / attn_avg_ms / 1e9
        # 8-bit keys: half of the kernel's flops (Q K^T) run on the e4m3 path, whose peak is the measured bf16 peak times the
        # nominal ratio 2, the other half (P V) on bf16: the blended peak is total / (1/2 / 2P + 1/2 / P) = 4/3 P
        blend = 4.0 / 3.0 if k8_keys is not None else 1.0
        roofline = {"bound": "tensor", "kernel": "tc::attn_kernel<false> (Step-1 exact pass over prefix + block keys)"
                                                 + (", Q K^T in e4m3, P V in bf16" if k8_keys is not None else ""), "achieved": achieved,
                    "peak": blend * (peaks["bf16_tflops"] if burst_regime else peaks["bf16_tflops_sustained"]), "unit": "TFLOP/s",
                    "peak_source": f"bf16 cuBLAS {'burst' if burst_regime else 'sustained'}, {peaks['source']}: "
                                   + ("median SM clock >= 0.95 max and no sw_power_cap sample" if burst_regime else "sw_power_cap sampled or SM clock below 0.95 max")
                                   + ("; x 4/3: half of the flops at the nominal 2x e4m3 rate" if k8_keys is not None else ""),
                    "frac_burst": achieved / (blend * peaks["bf16_tflops"]), "frac_sustained": achieved / (blend * peaks["bf16_tflops_sustained"]),
                    "issued_over_useful_flops": float(-(-w.M // 128) * 128) / w.M, "traffic": None}
        roofline["frac"] = roofline["achieved"] / roofline["peak"]
    roofline["hbm_view"] = {"achieved_gbs": sf["s1_attn_bytes"] / attn_avg_ms / 1e6, "peak_gbs": peaks["hbm_gbs"],
                            "frac_of_measured": sf["s1_attn_bytes"] / attn_avg_ms / 1e6 / peaks["hbm_gbs"],
                            "frac_of_8tbs": sf["s1_attn_bytes"] / attn_avg_ms / 1e6 / 8000.0}
    prof = os.path.join(ROOT, "profiles", "traffic.txt")       # ncu-measured DRAM bytes per launch (see the file's header)
    if os.path.exists(prof):
        for ln in open(prof):
            f = ln.split(None, 3)
            if len(f) >= 3 and not ln.startswith("#") and f[0] == ("simt" if args.simt else "default") and f[1] == w.name and k8_keys is None:
                roofline["traffic"] = int(f[2])
                roofline["traffic_source"] = f[3].strip() if len(f) > 3 else "ncu capture, see profiles/traffic.txt"
    # the stages the benchmark spec names, each against the roof that binds it
    s1_ms_all = (sum(attn_ms) + sum(comb_ms) + sum(score_ms)) / len(attn_ms)
    s1_flops = sf["s1_flops_attn"] + sf["s1_flops_score"]
    tensor_peak = peaks["bf16_tflops"] if burst_regime else peaks["bf16_tflops_sustained"]
    if k8_keys is not None:      # Step 1 as a whole: two of its three contractions (both Q K^T) on the e4m3 path: 1 / (2/3 / 2 + 1/3) = 3/2
        tensor_peak *= 1.5
    roofline_stages = {
        "step1_exact_select": {"bound": "tensor", "achieved": s1_flops / s1_ms_all / 1e9, "peak": tensor_peak, "unit": "TFLOP/s",
                               "frac": s1_flops / s1_ms_all / 1e9 / tensor_peak, "flops": s1_flops, "ms": s1_ms_all,
                               "hbm_view": {"algorithmic_bytes": sf["s1_bytes"], "achieved_gbs": sf["s1_bytes"] / s1_ms_all / 1e6,
                                            "frac_of_measured": sf["s1_bytes"] / s1_ms_all / 1e6 / peaks["hbm_gbs"],
                                            "frac_of_8tbs": sf["s1_bytes"] / s1_ms_all / 1e6 / 8000.0}}}
    if stages.get("sparse_step_ms_cold_l2"):
        sp_ms = stages["sparse_step_ms_cold_l2"]
        roofline_stages["sparse_reuse_step"] = {"bound": "hbm", "achieved": sf["s3_bytes"] / sp_ms / 1e6, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                                "frac": sf["s3_bytes"] / sp_ms / 1e6 / peaks["hbm_gbs"], "frac_of_8tbs": sf["s3_bytes"] / sp_ms / 1e6 / 8000.0,
                                                "algorithmic_bytes": sf["s3_bytes"], "ms": sp_ms, "l2": "flushed before each launch"}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        out = subprocess.run([sys.executable, os.path.abspath(__file__), "--impl", "reference", "--steps", "1", "--warmup", "0",
                              "--workload", args.workload] + (["--P", str(args.P)] if args.P else []) + (["--N", str(args.N)] if args.N else []),
                             capture_output=True, text=True)
        try:
            cpu_baseline = json.loads(out.stdout.strip().splitlines()[-1])["cpu_baseline"]
        except Exception:
            cpu_baseline = {"value": None, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": "failed: " + out.stderr[-200:]}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "strong" if kv_head_sharded else "weak", "vs_baseline": None,
        "dtype": "bf16" if k8_keys is None else "e4m3 (Q K^T) + bf16 (P V)", "data": "synthetic",
        "config": config_of(w_full, lens, world, "simt" if args.simt else ("default" if k8_keys is None else "default, keys and queries e4m3"),
                            f"kv_head x{world} (each rank owns H_kv/{world} KV heads of every layer; no collective)" if kv_head_sharded else None, key_bytes=1 if k8_keys is not None else 2),
        "clocks": clocks, "gpu_launches": launches, "dev_status": status,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
        "roofline": roofline, "roofline_stages": roofline_stages, "cpu_baseline": cpu_baseline, "stages": stages,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
