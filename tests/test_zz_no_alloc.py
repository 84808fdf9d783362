"""The workspace-free Step-1 entry point against the regular one (collected last on purpose).

`mage_exact_select_static` serves hosts that are not allowed to allocate device memory around the call; its
scratch is a fixed array inside the library.  It must give what `mage_exact_select` gives with a caller
workspace, call after call, whatever the shared array held before.
"""
import dataclasses

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

from paper_2602_14209_b200 import binding as mb
from paper_2602_14209_b200 import workloads as W


def _run(kv, batch, step, static):
    out = torch.full((kv.P, kv.H_q, kv.B, kv.d), float("nan"), dtype=torch.bfloat16, device="cuda")
    scores = torch.full((kv.P, kv.H_kv, kv.N_max), -1.0, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = kv.d ** -0.5
    if static:
        mb.mage_exact_select_static(kv, batch["q"][step], batch["kb"][step], batch["vb"][step], scale, out, scores, status)
    else:
        ws = kv.new_workspace()
        mb.mage_exact_select(kv, batch["q"][step], batch["kb"][step], batch["vb"][step], scale, out, scores, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out.float().cpu().numpy(), scores.cpu().numpy()


def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row(oracle_mod):
    from paper_2602_14209_b200 import build
    build.build()
    assert torch.cuda.is_available()
    w = dataclasses.replace(W.CONFIGS["cfg1_small"], N=3000, P=2, ragged_min=500, T=2, seed=21)
    batch = W.make_batch(w, device="cuda")
    kv = mb.KVCache(batch["kc"], batch["vc"], w.H_q, w.B, seq_lens=batch["seq_lens"])
    assert 0 < kv.workspace_bytes() <= mb.STATIC_SCRATCH_BYTES
    lens = batch["seq_lens"].tolist()
    f = lambda t: t.float().cpu().numpy()
    # two calls in a row on different inputs (step 0 then step 1 queries): the second call finds the first call's
    # leftovers in the shared array and must not be affected by them
    for step in (0, 1):
        o_ref, s_ref = _run(kv, batch, step, static=False)
        o_new, s_new = _run(kv, batch, step, static=True)
        # same kernels on the same plan, only the scratch address differs: the results are the same bits
        assert np.array_equal(o_new, o_ref)
        assert np.array_equal(s_new, s_ref)
        # ... and they are right: output and scores of the built-in-scratch call against the CPU oracle
        for p, n in enumerate(lens):
            O = oracle_mod.exact_block_attn(f(batch["q"][step, p]), f(batch["kc"][p, :, :n]), f(batch["vc"][p, :, :n]),
                                            f(batch["kb"][step, p]), f(batch["vb"][step, p]))
            err = np.abs(o_new[p] - O)
            assert err.max() <= 1e-2 and err.mean() <= 1e-3
            sc = oracle_mod.block_score(f(batch["q"][step, p]), f(batch["kc"][p, :, :n]))
            assert np.max(np.abs(s_new[p, :, :n] - sc) / sc) <= 1e-5
            assert (s_new[p, :, n:] == -1.0).all()


def test_static_scratch_variant_refuses_what_does_not_fit():
    """Pure host check (no launch): a description whose scratch need exceeds the built-in array is rejected."""
    from paper_2602_14209_b200 import build
    build.build()
    import ctypes
    lib = mb.load()
    c = mb.mage_kv_t()
    c.P, c.H_q, c.H_kv, c.d, c.B, c.page_size = 28, 28, 4, 128, 32, 0
    c.k_cache = c.v_cache = 4096
    c.stride_n, c.stride_h, c.stride_p, c.N_max = 128, 131072 * 128, 4 * 131072 * 128, 131072
    assert lib.mage_workspace_bytes(ctypes.byref(c), 1) > mb.STATIC_SCRATCH_BYTES
    p = ctypes.c_void_p(4096)
    assert lib.mage_exact_select_static(ctypes.byref(c), p, p, p, 0.088, p, p, None, None) == -3
