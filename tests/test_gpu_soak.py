"""A seeded sweep of irregular shapes through the whole path: every stage of the staged calls against the oracle
(chain validation, all attention rows), then the fused call bit for bit against the staged calls.  The shapes mix
batch sizes, GQA ratios, head dims, dtypes, chunk lengths on and off the 128-row tiles, empty / one-row / long caches,
key budgets as counts and as fractions, contiguous and paged caches.  The dense chunk attention of the same problem
(the speed-up denominator; with a long cache and few heads it runs split into parts) is checked on one sequence."""
import numpy as np
import pytest
import torch

from paper_2602_08722_b200 import api, synth
from oracle import quoka_oracle as O
from tests.parity import GpuProblem, check_attention, check_chain, f64

pytestmark = pytest.mark.gpu


def shape(seed):
    r = np.random.default_rng(seed)
    batch = int(r.integers(1, 4))
    n_kv = int(r.choice([1, 2, 4]))
    G = int(r.choice([1, 2, 4]))
    d = int(r.choice([64, 128]))
    dtype = "bf16" if r.random() < 0.8 else "f32"
    C = int(r.choice([1, 7, 64, 129, 200, 256, 300, 513, 700]))
    T = [int(r.choice([0, 1, 63, 128, 500, 1100, 2500, 4100])) for _ in range(batch)]
    n_retain = int(r.choice([1, 4, 16, 33, 64, 128, 200]))
    if r.random() < 0.5:
        kv_budget, frac = int(r.choice([1, 17, 128, 300, 1000])), 0.0
    else:
        kv_budget, frac = 0, float(r.choice([0.05, 0.12, 0.25, 0.9]))
    paged = bool(r.random() < 0.4)
    return dict(batch=batch, n_q=n_kv * G, n_kv=n_kv, d=d, dtype=dtype, C=C, T=T, n_retain=n_retain,
                kv_budget=kv_budget, frac=frac, paged=paged)


@pytest.mark.parametrize("seed", list(range(9000, 9036)))
def test_random_shape(seed):
    c = shape(seed)
    inp = synth.make_chunk_inputs(seed, c["batch"], c["n_q"], c["n_kv"], c["d"], c["T"] if c["batch"] > 1 else c["T"][0],
                                  c["C"], c["dtype"])
    if c["paged"]:
        inp = synth.to_paged(inp, seed)
    gp = GpuProblem(inp, c["n_retain"], c["kv_budget"], c["frac"], paged=c["paged"])
    gp.run_staged()
    check_chain(gp)
    staged_out, staged_idx, staged_cnt = gp.out.clone(), gp.k_idx.clone(), gp.k_cnt.clone()
    for _ in range(2):
        gp.out.zero_()
        idx2, cnt2 = torch.full_like(gp.k_idx, -9), torch.full_like(gp.k_cnt, -9)
        api.quoka_prefill_chunk(gp.p, gp.q, gp.k, gp.v, gp.out, idx2, cnt2, gp.ws)
        torch.cuda.synchronize()
        assert torch.equal(idx2, staged_idx) and torch.equal(cnt2, staged_cnt), c
        assert torch.equal(gp.out, staged_out), c
    s_chk = seed % c["batch"]
    gp.out.zero_()
    api.quoka_dense_chunk_attn(gp.p, gp.q, gp.k, gp.v, gp.out, gp.lse, gp.ws)
    torch.cuda.synchronize()
    q, k, v, T = gp.oracle_inputs(s_chk)
    want, lse = O.dense_chunk_attention(q, k, v, T)
    check_attention(f64(gp.out[s_chk]), want, c["dtype"])
    assert np.abs(f64(gp.lse[s_chk]) - lse).max() <= 2e-3, c
    assert api.quoka_last_device_status(gp.ws) == 0
