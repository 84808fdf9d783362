"""The bounded waits inside the kernels: a wait that cannot be satisfied runs out, the call returns, the status says so,
and the context stays usable.

The failure is made without faulting anything: with MAGE_FLAG_TEST_STALL the exact pass never requests its first key tile
(so no copy is in flight) and its waits use a limit of about a millisecond.  No trap, no device assert, no endless loop.
"""
import time

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W
import gpu_harness as H


def test_a_wait_that_runs_out_sets_the_status_and_leaves_the_context_usable(oracle_mod):
    from paper_2602_14209_b200 import build
    build.build()
    w = W.CONFIGS["cfg1_small"]
    batch = W.make_batch(w, device="cuda")
    kv_stall = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"], flags=mb.FLAG_TEST_STALL)
    out = torch.zeros(1, w.H_q, w.B, w.d, dtype=torch.bfloat16, device="cuda")
    scores = torch.zeros(1, w.H_kv, w.N, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = kv_stall.new_workspace(w.k)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    mb.mage_exact_select(kv_stall, batch["q"][0], batch["kb"][0], batch["vb"][0], w.d ** -0.5, out, scores, ws, status)
    torch.cuda.synchronize()                                  # returns: every role of every CTA took the common exit
    elapsed = time.perf_counter() - t0
    assert int(status.item()) & mb.DEV_TIMEOUT
    assert elapsed < 5.0, elapsed                             # ~1 ms of waiting per CTA, not the 0.25 s production limit
    # the same context, the same workspace: an ordinary block right afterwards is correct
    res = H.run_gpu_block(batch, w)
    assert res["status"] == 0
    H.check_problem(oracle_mod, batch, res, w, 0)
    # and the select stream's own pass takes the same exit
    status.zero_()
    mb.mage_select_scores(kv_stall, batch["q"][0], w.d ** -0.5, scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) & mb.DEV_TIMEOUT
    res = H.run_gpu_block(batch, w)
    H.check_problem(oracle_mod, batch, res, w, 0)
