"""Algorithm 2 as a loop with a growing cache (append, select, attend, every chunk against the oracle), and the
library's diagnostics: the bounded device wait, the debug build's index checks, the host-side block-table check."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import quoka_oracle as O
from paper_2602_08722_b200 import api, build, synth
from tests.parity import GpuProblem, check_attention, check_chain, f64

pytestmark = pytest.mark.gpu


# ---------------------------------------------------------------- Algorithm 2: the whole loop on a growing cache
@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("C_,n_chunks,frac", [(256, 6, 0.25), (128, 9, 0.12)])
def test_chunked_prefill_loop_with_append_matches_oracle_every_chunk(C_, n_chunks, frac, paged):
    """The device cache starts EMPTY.  Chunk i appends its own K_i, V_i at rows [iC, (i+1)C) with quoka_append_kv,
    runs the loop body, and advances the cached length on the device.  Every chunk's ranks, Q-bar, scores, index
    set and attention output are checked against the oracle run on the same growing cache."""
    b, n_q, n_kv, d = 2, 8, 2, 128
    T_end = C_ * (n_chunks - 1)
    full = synth.make_chunk_inputs(31, b, n_q, n_kv, d, T_end, C_, "bf16")          # all rows the prompt will append
    if paged:
        full = synth.to_paged(full, 31)
    gp = GpuProblem(full, n_retain=32, kv_budget=0, budget_frac=frac, paged=paged, max_ctx_len=T_end)
    gp.k.zero_()
    gp.v.zero_()
    k_inv = torch.full(tuple(gp.k.shape[:3]), float("nan"), dtype=torch.float32, device="cuda")
    gp.ctx_len.zero_()
    g = torch.Generator().manual_seed(77)
    mu = torch.randn(b, n_q, 1, d, generator=g)
    for i in range(n_chunks):
        T = i * C_
        q_i = (mu + 0.7 * torch.randn(b, n_q, C_, d, generator=g)).to(torch.bfloat16)
        gp.inp.q = q_i
        gp.q.copy_(q_i)
        gp.inp.ctx_len = torch.full((b,), T, dtype=torch.int32)
        k_new = full.k[:, :, T:T + C_].contiguous().cuda()
        v_new = full.v[:, :, T:T + C_].contiguous().cuda()
        api.quoka_append_kv(gp.p, k_new, v_new, gp.k, gp.v, k_inv, gp.ws)
        gp.run_staged()
        stats = check_chain(gp)
        want_out, want_idx = gp.out.clone(), gp.k_idx.clone()
        gp.out.zero_()
        idx2, cnt2 = torch.full_like(gp.k_idx, -9), torch.full_like(gp.k_cnt, -9)
        api.quoka_prefill_chunk(gp.p, gp.q, gp.k, gp.v, gp.out, idx2, cnt2, gp.ws)
        gp.ctx_len.add_(C_)                                                          # Alg. 2: the cache grew by one chunk
        torch.cuda.synchronize()
        assert torch.equal(gp.out, want_out) and torch.equal(idx2, want_idx) and torch.equal(cnt2, gp.k_cnt), i
    # the cache the loop built is the cache the oracle saw, and the inverse norms were kept for every appended row
    if paged:
        assert torch.equal(gp.k.cpu(), full.k_pages) and torch.equal(gp.v.cpu(), full.v_pages)
    else:
        assert torch.equal(gp.k.cpu(), full.k) and torch.equal(gp.v.cpu(), full.v)
    for s in range(b):
        want = O.key_inv_norms(f64(full.k[s]))
        if paged:
            tbl = full.block_table[s]
            got = np.stack([f64(k_inv[int(tbl[t // 64]), :, t % 64]) for t in range(T_end + C_)], axis=1)
        else:
            got = f64(k_inv[s, :, :T_end + C_])
        np.testing.assert_allclose(got, want[:, :T_end + C_], rtol=2e-6)
    assert api.quoka_last_device_status(gp.ws) == 0


def test_append_kv_f32_contiguous():
    inp = synth.make_chunk_inputs(32, 2, 4, 2, 64, [300, 77], 50, "f32")
    gp = GpuProblem(inp, 8, kv_budget=32)
    want_k, want_v = gp.k.clone(), gp.v.clone()
    k_new = torch.stack([inp.k[s, :, int(inp.ctx_len[s]):int(inp.ctx_len[s]) + 50] for s in range(2)]).contiguous().cuda()
    v_new = torch.stack([inp.v[s, :, int(inp.ctx_len[s]):int(inp.ctx_len[s]) + 50] for s in range(2)]).contiguous().cuda()
    for s in range(2):
        T = int(inp.ctx_len[s])
        gp.k[s, :, T:T + 50] = 0
        gp.v[s, :, T:T + 50] = 0
    api.quoka_append_kv(gp.p, k_new, v_new, gp.k, gp.v, None, gp.ws)
    torch.cuda.synchronize()
    assert torch.equal(gp.k, want_k) and torch.equal(gp.v, want_v)


# ---------------------------------------------------------------- the bounded device wait
def test_a_wait_that_nobody_satisfies_gives_up_and_reports():
    inp = synth.make_chunk_inputs(33, 1, 4, 2, 128, 500, 130, "bf16")
    gp = GpuProblem(inp, 16, kv_budget=100)
    gave_up = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    api.quoka_selftest_wait_timeout(gp.ws, 200_000, gave_up)          # about 0.1 ms of SM cycles
    torch.cuda.synchronize()
    assert int(gave_up[0]) == 1
    assert api.quoka_last_device_status(gp.ws) == api.ERR_TIMEOUT
    assert api.quoka_last_device_status(gp.ws) == 0                   # reading clears it
    # the context is intact: the next call works and is correct
    gp.run_staged()
    check_chain(gp)


# ---------------------------------------------------------------- debug build: bad indices are caught, not read
def test_debug_build_catches_a_bad_list_entry_and_a_bad_page_id():
    build.build(debug=True)
    dbg = api.open_debug_library()
    T, C_ = 900, 140
    inp = synth.to_paged(synth.make_chunk_inputs(34, 1, 4, 2, 128, T, C_, "bf16"), 34)
    gp = GpuProblem(inp, 16, kv_budget=200, paged=True)
    gp.run_staged()                                                   # the release library: a valid list
    good = gp.out.clone()
    stream = torch.cuda.current_stream().cuda_stream

    def attend():
        st = dbg.quoka_sparse_attn(C.byref(gp.p), gp.q.data_ptr(), gp.k.data_ptr(), gp.v.data_ptr(),
                                   gp.k_idx.data_ptr(), gp.k_cnt.data_ptr(), gp.out.data_ptr(), None,
                                   gp.ws.data_ptr(), gp.ws.numel(), stream)
        assert st == api.OK
        torch.cuda.synchronize()

    attend()                                                          # same inputs through the debug library
    assert torch.equal(gp.out, good) and api.quoka_last_device_status(gp.ws) == 0
    # a list entry far outside the cache: recorded, the row counts as a zero key with a zero value
    idx = gp.k_idx.clone()
    victim = int(idx[0, 1, 5])
    gp.k_idx[0, 1, 5] = T + 10_000_000
    attend()
    assert api.quoka_last_device_status(gp.ws) == api.ERR_BAD_INDEX
    assert torch.isfinite(gp.out.float()).all()
    q, k, v, _ = gp.oracle_inputs(0)
    k0, v0 = k.copy(), v.copy()
    k0[1, victim] = 0.0
    v0[1, victim] = 0.0
    idx_list = [idx[0, kv, :200].cpu().numpy() for kv in range(gp.n_kv)]
    want, _ = O.sparse_attention(q, k0, v0, T, idx_list)
    check_attention(f64(gp.out[0]), want, "bf16")
    # a page id outside the pool
    gp.k_idx.copy_(idx)
    table = gp.block_table.clone()
    gp.block_table[0, 2] = 1 << 28
    attend()
    assert api.quoka_last_device_status(gp.ws) == api.ERR_BAD_INDEX
    assert torch.isfinite(gp.out.float()).all()
    gp.block_table.copy_(table)
    attend()
    assert torch.equal(gp.out, good) and api.quoka_last_device_status(gp.ws) == 0
