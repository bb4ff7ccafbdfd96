"""The C-ABI library loads, exports every entry point the header declares, and rejects bad
arguments on the host before anything is launched.  No GPU needed (no compute call is made)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2602_08722_b200 import build
    build.build()
    from paper_2602_08722_b200 import api
    return api.load()


def declared_entry_points():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(quoka_[a-z_0-9]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    from paper_2602_08722_b200 import api
    names = declared_entry_points()
    assert {"quoka_select_queries", "quoka_score_keys", "quoka_select_keys", "quoka_sparse_attn",
            "quoka_prefill_chunk", "quoka_dense_chunk_attn"} <= names
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/ but not exported"
    assert set(api.EXPORTS) <= names


def good_params():
    from paper_2602_08722_b200 import api
    p = api.QuokaParams()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim = 1, 8, 2, 128
    p.chunk_len, p.n_retain, p.kv_budget, p.budget_frac = 256, 32, 512, 0.0
    p.dtype, p.impl, p.softmax_scale, p.max_ctx_len = api.BF16, api.IMPL_AUTO, 0.0, 4096
    p.ctx_len = 0x1000
    p.q_stride_b, p.q_stride_h, p.q_stride_t = 8 * 256 * 128, 256 * 128, 128
    p.o_stride_b, p.o_stride_h, p.o_stride_t = 8 * 256 * 128, 256 * 128, 128
    p.page_size, p.max_pages_per_seq, p.block_table = 0, 0, None
    p.kv_stride_b, p.kv_stride_h, p.kv_stride_t = 2 * 4352 * 128, 4352 * 128, 128
    p.kv_rows = 4352
    return p


def test_workspace_size_and_budget_cap(lib):
    from paper_2602_08722_b200 import api
    p = good_params()
    assert api.quoka_kv_budget_cap(p) == 512
    n = api.quoka_workspace_size(p)
    assert n >= 256 + 8 * 32 * 4 + 2 * 32 * 128 * 2 + 2 * 4096 * 4 + 2 * 512 * 4
    p.kv_budget, p.budget_frac, p.max_ctx_len = 0, 0.12, 32768
    p.kv_rows = 32768 + 256
    assert api.quoka_kv_budget_cap(p) == 3932
    p.max_ctx_len, p.kv_rows = 131072, 131072 + 256
    assert api.quoka_kv_budget_cap(p) == 15729


@pytest.mark.parametrize("field,value,status", [
    ("head_dim", 96, 2), ("n_kv_heads", 3, 1), ("batch", 0, 1), ("page_size", 16, 2), ("dtype", 7, 1),
    ("q_stride_t", 100, 1), ("kv_rows", 100, 1), ("chunk_len", 0, 1), ("impl", 9, 1), ("kv_stride_h", 12, 1),
])
def test_bad_params_are_rejected_before_any_launch(lib, field, value, status):
    from paper_2602_08722_b200 import api
    p = good_params()
    setattr(p, field, value)
    before = api.quoka_launch_count()
    n = C.c_size_t(0)
    assert lib.quoka_workspace_size(C.byref(p), C.byref(n)) == status
    # a compute entry point with otherwise plausible pointers must refuse as well, launching nothing
    st = lib.quoka_select_queries(C.byref(p), 0x1000, 0x2000, 0x3000, 0x4000, 1 << 30, None)
    assert st == status
    assert api.quoka_launch_count() == before


def test_null_and_misaligned_pointers_and_small_workspace(lib):
    from paper_2602_08722_b200 import api
    p = good_params()
    before = api.quoka_launch_count()
    assert lib.quoka_select_queries(C.byref(p), None, 0x2000, 0x3000, 0x4000, 1 << 30, None) == api.ERR_INVALID_ARG
    assert lib.quoka_select_queries(C.byref(p), 0x1008, 0x2000, 0x3000, 0x4000, 1 << 30, None) == api.ERR_INVALID_ARG
    assert lib.quoka_select_queries(C.byref(p), 0x1000, 0x2000, 0x3000, None, 1 << 30, None) == api.ERR_WORKSPACE
    assert lib.quoka_select_queries(C.byref(p), 0x1000, 0x2000, 0x3000, 0x4010, 1 << 30, None) == api.ERR_WORKSPACE
    assert lib.quoka_select_queries(C.byref(p), 0x1000, 0x2000, 0x3000, 0x4000, 64, None) == api.ERR_WORKSPACE
    assert lib.quoka_sparse_attn(C.byref(p), 0x1000, 0x2000, 0x3000, None, 0x5000, 0x6000, None, 0x4000, 1 << 30,
                                 None) == api.ERR_INVALID_ARG
    assert api.quoka_launch_count() == before
    assert api.status_string(api.ERR_TIMEOUT)


def test_f32_on_tensor_path_is_unsupported(lib):
    from paper_2602_08722_b200 import api
    p = good_params()
    p.dtype, p.impl = api.F32, api.IMPL_TENSOR
    n = C.c_size_t(0)
    assert lib.quoka_workspace_size(C.byref(p), C.byref(n)) == api.ERR_UNSUPPORTED


def test_missing_library_is_an_error(monkeypatch, tmp_path):
    from paper_2602_08722_b200 import api
    monkeypatch.setattr(api, "_lib", None)
    monkeypatch.setattr(api, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        api.load()


def test_block_table_check_on_the_host(lib):
    """quoka_check_block_table: pages outside the pool and pages used twice are refused; nothing is launched."""
    import torch
    from paper_2602_08722_b200 import api, synth
    inp = synth.to_paged(synth.make_chunk_inputs(3, 2, 4, 2, 64, [200, 70], 60, "bf16"), 3)
    p = good_params()
    p.batch, p.n_q_heads, p.n_kv_heads, p.head_dim, p.chunk_len, p.max_ctx_len = 2, 4, 2, 64, 60, 200
    p.page_size, p.max_pages_per_seq, p.kv_rows = 64, inp.block_table.shape[1], inp.k_pages.shape[0]
    before = api.quoka_launch_count()
    table = inp.block_table.clone()
    assert api.quoka_check_block_table(p, inp.ctx_len, table) == api.OK
    bad = table.clone()
    bad[0, 1] = p.kv_rows                     # one past the pool
    assert api.quoka_check_block_table(p, inp.ctx_len, bad) == api.ERR_INVALID_ARG
    bad = table.clone()
    bad[1, 0] = table[0, 0]                   # two logical pages on one physical page
    assert api.quoka_check_block_table(p, inp.ctx_len, bad) == api.ERR_INVALID_ARG
    bad = table.clone()
    bad[1, 3] = -1                            # a page the sequence does not need may be anything
    assert api.quoka_check_block_table(p, inp.ctx_len, bad) == api.OK
    too_long = torch.tensor([201, 70], dtype=torch.int32)
    assert api.quoka_check_block_table(p, too_long, table) == api.ERR_INVALID_ARG
    assert api.quoka_launch_count() == before


def test_debug_library_builds_and_exports_the_same_entry_points():
    from paper_2602_08722_b200 import api, build
    build.build(debug=True)
    dbg = api.open_debug_library()
    for n in declared_entry_points():
        assert hasattr(dbg, n)


def test_launch_logging_is_off_by_default(lib, capfd):
    from paper_2602_08722_b200 import api
    p = good_params()
    lib.quoka_select_queries(C.byref(p), None, 0x2000, 0x3000, 0x4000, 1 << 30, None)
    assert "[quoka]" not in capfd.readouterr().err
