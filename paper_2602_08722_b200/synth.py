"""Seeded synthetic inputs for one prefill chunk of one attention layer.

This module only draws random tensors and lays them out (contiguous or paged).
It holds none of the method's arithmetic, so both the CUDA path's callers and
the CPU checker can be fed from it: the same seed gives the same bits to both.

Distributions (stand-ins for real long-context prefill activations): per query
head a mean direction mu ~ N(0, I_d); queries = mu + 0.7 * N(0, I_d); keys ~
N(0, I_d) where, independently per (KV head, position), 5 % of the keys are
scaled by 3; values ~ N(0, I_d).  In bf16 mode every tensor is rounded to bf16
(torch's round-to-nearest-even) and the rounded values are what everyone uses.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

PAGE_SIZE = 64


@dataclass
class ChunkInputs:
    q: torch.Tensor            # (b, n_Q, C, d)
    k: torch.Tensor            # (b, n_KV, capacity, d): rows [0,T_s) cache, [T_s,T_s+C) the chunk's own keys
    v: torch.Tensor            # same layout
    ctx_len: torch.Tensor      # (b,) int32, T_s
    chunk_len: int
    dtype: str                 # "bf16" | "f32"
    k_pages: torch.Tensor | None = None      # (n_pages, n_KV, 64, d) when paged
    v_pages: torch.Tensor | None = None
    block_table: torch.Tensor | None = None  # (b, max_pages) int32
    meta: dict = field(default_factory=dict)


def _torch_dtype(dtype: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]


def make_chunk_inputs(seed: int, batch: int, n_q: int, n_kv: int, d: int, ctx_lens, chunk_len: int,
                      dtype: str = "bf16", capacity: int | None = None) -> ChunkInputs:
    """Draw q, k, v for `batch` sequences with cached lengths `ctx_lens` (an int
    applies to all).  Rows of k, v at and beyond T_s + chunk_len are zero."""
    if isinstance(ctx_lens, int):
        ctx_lens = [ctx_lens] * batch
    ctx_lens = [int(t) for t in ctx_lens]
    assert len(ctx_lens) == batch
    C = int(chunk_len)
    cap = max(ctx_lens) + C if capacity is None else int(capacity)
    assert cap >= max(ctx_lens) + C
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed))
    td = _torch_dtype(dtype)

    mu = torch.randn(batch, n_q, 1, d, generator=g)
    q = (mu + 0.7 * torch.randn(batch, n_q, C, d, generator=g)).to(td)
    k = torch.zeros(batch, n_kv, cap, d, dtype=td)
    v = torch.zeros(batch, n_kv, cap, d, dtype=td)
    for s in range(batch):
        rows = ctx_lens[s] + C
        ks = torch.randn(n_kv, rows, d, generator=g)
        big = torch.rand(n_kv, rows, 1, generator=g) < 0.05
        ks = torch.where(big, ks * 3.0, ks)
        k[s, :, :rows] = ks.to(td)
        del ks
        v[s, :, :rows] = torch.randn(n_kv, rows, d, generator=g).to(td)
    return ChunkInputs(q=q, k=k, v=v, ctx_len=torch.tensor(ctx_lens, dtype=torch.int32),
                       chunk_len=C, dtype=dtype,
                       meta=dict(seed=seed, batch=batch, n_q=n_q, n_kv=n_kv, d=d, capacity=cap))


def to_paged(inp: ChunkInputs, seed: int = 0, page_size: int = PAGE_SIZE) -> ChunkInputs:
    """Scatter the contiguous caches into a page pool [page][n_KV][page_size][d]
    with a random global page permutation and build the block table."""
    b, n_kv, cap, d = inp.k.shape
    C = inp.chunk_len
    need = [math.ceil((int(t) + C) / page_size) for t in inp.ctx_len.tolist()]
    total = sum(need)
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) + 7919)
    perm = torch.randperm(total, generator=g)
    max_pages = max(need)
    table = torch.full((b, max_pages), -1, dtype=torch.int32)
    kp = torch.zeros(total, n_kv, page_size, d, dtype=inp.k.dtype)
    vp = torch.zeros(total, n_kv, page_size, d, dtype=inp.v.dtype)
    off = 0
    for s in range(b):
        for p in range(need[s]):
            pid = int(perm[off + p])
            table[s, p] = pid
            lo = p * page_size
            hi = min(lo + page_size, cap)
            kp[pid, :, : hi - lo] = inp.k[s, :, lo:hi]
            vp[pid, :, : hi - lo] = inp.v[s, :, lo:hi]
        off += need[s]
    out = ChunkInputs(q=inp.q, k=inp.k, v=inp.v, ctx_len=inp.ctx_len, chunk_len=C, dtype=inp.dtype,
                      k_pages=kp, v_pages=vp, block_table=table, meta=dict(inp.meta))
    out.meta.update(page_size=page_size, n_pages=total, max_pages=max_pages)
    return out


def serving_mix_ctx_lens(seed: int, batch: int = 8, lo: int = 8192, hi: int = 65536):
    """Cached lengths T_s ~ U{lo..hi} for the serving-mix workload."""
    g = torch.Generator(device="cpu")
    g.manual_seed(int(seed) + 104729)
    return torch.randint(lo, hi + 1, (batch,), generator=g).tolist()


# Named workloads (shapes of the five benchmark configurations).
WORKLOADS = {
    "tiny_bf16": dict(batch=1, n_q=8, n_kv=2, d=128, T=4096, C=256, n_retain=32, kv_budget=512, dtype="bf16"),
    "tiny_f32": dict(batch=1, n_q=8, n_kv=2, d=128, T=4096, C=256, n_retain=32, kv_budget=512, dtype="f32"),
    "llama8b_32k": dict(batch=1, n_q=32, n_kv=8, d=128, T=32768, C=2048, n_retain=128, kv_budget=3932, dtype="bf16"),
    "long_128k": dict(batch=1, n_q=32, n_kv=8, d=128, T=131072, C=4096, n_retain=256, kv_budget=15729, dtype="bf16"),
    # generation phase (one query per sequence, no query sub-selection), budget 256 keys
    "decode_32k": dict(batch=1, n_q=32, n_kv=8, d=128, T=32768, C=1, n_retain=16, kv_budget=256, dtype="bf16"),
    "decode_32k_b16": dict(batch=16, n_q=32, n_kv=8, d=128, T=32768, C=1, n_retain=16, kv_budget=256, dtype="bf16"),
    "serving_mix": dict(batch=8, n_q=32, n_kv=8, d=128, T=None, C=1024, n_retain=64, kv_budget=0,
                        budget_frac=0.12, paged=True, dtype="bf16"),
}
