"""Host-side checks of the C ABI that need no GPU: the library loads, exports what mage.h declares, rejects bad arguments."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_14209_b200 import build, binding
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "mage.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mage_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert {"mage_exact_select", "mage_topk", "mage_sparse_block_attn", "mage_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    from paper_2602_14209_b200 import binding
    assert set(binding.EXPORTS) == set(names)


def _kv(**over):
    from paper_2602_14209_b200.binding import mage_kv_t
    c = mage_kv_t()
    c.P, c.H_q, c.H_kv, c.d, c.B, c.page_size = 1, 8, 2, 128, 32, 0
    c.k_cache = c.v_cache = 4096          # never dereferenced by the host code
    c.stride_n, c.stride_h, c.stride_p = 128, 2048 * 128, 2 * 2048 * 128
    c.N_max = 2048
    for k, v in over.items():
        setattr(c, k, v)
    return c


def test_status_strings(lib):
    from paper_2602_14209_b200 import binding
    assert binding.status_string(0) == "MAGE_OK"
    assert binding.status_string(-1) == "MAGE_ERR_INVALID_ARG"
    assert binding.status_string(-3) == "MAGE_ERR_WORKSPACE"
    assert binding.status_string(-99) == "MAGE_ERR_UNKNOWN"


def test_workspace_bytes_is_pure_host_arithmetic(lib):
    c = _kv()
    n = lib.mage_workspace_bytes(ctypes.byref(c), 256)
    assert n > 0 and n % 256 == 0
    assert lib.mage_workspace_bytes(ctypes.byref(c), 256) == n
    assert lib.mage_workspace_bytes(ctypes.byref(_kv(d=64)), 256) == 0
    assert lib.mage_workspace_bytes(ctypes.byref(_kv(H_q=7)), 256) == 0
    assert lib.mage_workspace_bytes(None, 256) == 0
    big = _kv(P=28, H_q=28, H_kv=4, N_max=131072, stride_h=131072 * 128, stride_p=4 * 131072 * 128)
    assert 0 < lib.mage_workspace_bytes(ctypes.byref(big), 512) < (1 << 30)


def test_workspace_plan_over_a_range_of_shapes(lib):
    """The chunk count behind the workspace size comes from a cost search; whatever it picks, the size stays bounded
    (at most 148 partial results per head plus the split region), grows with the budget, and one Qwen-shaped layer at
    32K fits the 32 MiB of the no-allocation entry point."""
    from paper_2602_14209_b200 import binding
    per_item = 256 * (128 + 2) * 4                       # one partial result of a 224-row head: O and (m, l), fp32
    for P in (1, 3, 28, 200):
        for N in (0, 100, 2048, 32768, 131072, 1000000):
            for page in (0, 64):
                c = _kv(P=P, H_q=28, H_kv=4, N_max=N, stride_h=max(N, 1) * 128, stride_p=4 * max(N, 1) * 128, page_size=page)
                if page:
                    c.block_table, c.max_pages, c.num_pages = 4096, (N + page - 1) // page, max(1, P * ((N + page - 1) // page))
                small, large = lib.mage_workspace_bytes(ctypes.byref(c), 64), lib.mage_workspace_bytes(ctypes.byref(c), 2048)
                heads = P * 4
                assert 0 < small <= large, (P, N, page)
                assert small <= heads * (149 + 33) * per_item + (1 << 20), (P, N, page, small)
    layer = _kv(P=1, H_q=28, H_kv=4, N_max=32768, stride_h=32768 * 128, stride_p=4 * 32768 * 128)
    assert lib.mage_workspace_bytes(ctypes.byref(layer), 512) <= binding.STATIC_SCRATCH_BYTES + (8 << 20)


@pytest.mark.parametrize("over,code", [
    (dict(d=64), -2), (dict(B=65), -2), (dict(B=0), -1), (dict(H_q=9), -1), (dict(P=0), -1),
    (dict(stride_n=100), -1), (dict(stride_h=12), -1), (dict(k_cache=0), -1), (dict(page_size=-1), -1),
    (dict(page_size=48), -2), (dict(page_size=64, block_table=0), -1),
    (dict(page_size=64, block_table=4096, num_pages=100, max_pages=3), -1),
])
def test_exact_select_rejects_bad_descriptions_before_any_launch(lib, over, code):
    c = _kv(**over)
    p = ctypes.c_void_p(4096)
    rc = lib.mage_exact_select(ctypes.byref(c), p, p, p, 0.088, p, p, p, 1 << 30, None, None)
    assert rc == code
    rc = lib.mage_sparse_block_attn(ctypes.byref(c), p, p, p, p, p, 16, 0.088, p, None, 0, None, None)
    assert rc == code


def test_rejects_null_pointers_small_workspace_and_bad_scalars(lib):
    c = _kv()
    p = ctypes.c_void_p(4096)
    need = lib.mage_workspace_bytes(ctypes.byref(c), 1)
    assert lib.mage_exact_select(ctypes.byref(c), None, p, p, 0.088, p, p, p, need, None, None) == -1
    assert lib.mage_exact_select(ctypes.byref(c), p, p, p, 0.088, p, None, p, need, None, None) == -1
    assert lib.mage_exact_select(ctypes.byref(c), p, p, p, 0.088, p, p, p, 4096, None, None) == -3
    assert lib.mage_exact_select(ctypes.byref(c), p, p, p, 0.0, p, p, p, need, None, None) == -1
    assert lib.mage_exact_select(ctypes.byref(c), p, p, p, 0.088, p, p, ctypes.c_void_p(4100), need, None, None) == -1
    assert lib.mage_exact_select(None, p, p, p, 0.088, p, p, p, need, None, None) == -1
    assert lib.mage_sparse_block_attn(ctypes.byref(c), p, p, p, None, p, 16, 0.088, p, None, 0, None, None) == -1
    assert lib.mage_sparse_block_attn(ctypes.byref(c), p, p, p, p, p, 0, 0.088, p, None, 0, None, None) == -1
    assert lib.mage_topk(p, None, 1, 2, 2048, 0, p, p, None, 0, None) == -1
    assert lib.mage_topk(p, None, 0, 2, 2048, 8, p, p, None, 0, None) == -1
    assert lib.mage_topk(p, None, 1, 2, 2048, 8, None, p, None, 0, None) == -1
    assert lib.mage_topk(None, None, 1, 2, 2048, 8, p, p, None, 0, None) == -1
    assert lib.mage_append_block(ctypes.byref(c), p, p, None, None, None) == -1
    assert lib.mage_append_block(ctypes.byref(c), None, p, p, None, None) == -1
    assert lib.mage_append_block(None, p, p, p, None, None) == -1


def test_binding_fails_loudly_without_library(monkeypatch, tmp_path):
    from paper_2602_14209_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "missing.so"))
    with pytest.raises(RuntimeError, match="not built"):
        binding.load()
