"""quoka_prefill_chunk_static: the fused call for callers that cannot allocate a workspace (their
serving process has already given all of HBM to its cache pool, or they sit in a loop where
cudaMalloc's device-wide synchronisation is not acceptable).  It must give exactly what
quoka_prefill_chunk gives with a caller-owned workspace, call after call, although every call reuses
the same built-in scratch array and inherits the previous call's leftovers.

This file sorts last on purpose, so a run that stops at the first failure has already run the rest."""
import ctypes as C

import pytest
import torch

from paper_2602_08722_b200 import api, synth
from tests.parity import GpuProblem


def _problem(seed, T, C_, n_retain, kv_budget):
    inp = synth.make_chunk_inputs(seed, 1, 8, 2, 128, T, C_, "bf16")
    return GpuProblem(inp, n_retain, kv_budget)


@pytest.mark.gpu
def test_static_scratch_call_matches_workspace_call_twice_in_a_row():
    # two different problems back to back: the second is smaller, so stale scores, indices and Qbar
    # from the first are still lying in the array when it runs
    for seed, T, C_, n_retain, kv_budget in [(21, 3000, 300, 32, 400), (22, 700, 130, 16, 90)]:
        gp = _problem(seed, T, C_, n_retain, kv_budget)
        api.quoka_prefill_chunk(gp.p, gp.q, gp.k, gp.v, gp.out, gp.k_idx, gp.k_cnt, gp.ws)
        torch.cuda.synchronize()
        want_out, want_idx, want_cnt = gp.out.clone(), gp.k_idx.clone(), gp.k_cnt.clone()
        for _ in range(2):
            gp.out.zero_()
            gp.k_idx.fill_(-5)
            gp.k_cnt.fill_(-5)
            before = torch.cuda.memory_allocated()
            api.quoka_prefill_chunk_static(gp.p, gp.q, gp.k, gp.v, gp.out, gp.k_idx, gp.k_cnt)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            # same kernels, same inputs: the tolerance of the fused-vs-staged tests is bit equality
            assert torch.equal(gp.k_idx, want_idx) and torch.equal(gp.k_cnt, want_cnt)
            assert torch.equal(gp.out, want_out)


@pytest.mark.gpu
def test_problem_larger_than_the_static_array_is_refused():
    gp = _problem(23, 600, 128, 16, 64)
    gp.p.max_ctx_len = 4 << 20          # scores alone would need 2 * 4 Mi * 4 bytes = 32 MiB
    gp.p.kv_rows = (4 << 20) + 128
    assert api.quoka_workspace_size(gp.p) > api.STATIC_SCRATCH_BYTES
    n0 = api.quoka_launch_count()
    with pytest.raises(api.QuokaError) as e:
        api.quoka_prefill_chunk_static(gp.p, gp.q, gp.k, gp.v, gp.out, None, None)
    assert e.value.status == api.ERR_STATIC_LIMIT
    assert api.quoka_launch_count() == n0


def test_static_entry_point_is_declared_and_exported():
    from paper_2602_08722_b200 import build
    build.build()
    lib = api.load()
    assert hasattr(lib, "quoka_prefill_chunk_static")
    assert "built-in" in api.status_string(api.ERR_STATIC_LIMIT)
    p = api.QuokaParams()          # all zero: refused on the host, nothing launched, nothing allocated
    assert lib.quoka_prefill_chunk_static(C.byref(p), None, None, None, None, None, None, None) == api.ERR_INVALID_ARG
