"""The benchmark's work model (algorithmic bytes and flops per launch) against the figures the roofline fractions are
quoted on, and the whole-job arithmetic of the multi-rank bench line (CPU only)."""
import importlib.util
import os

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
spec = importlib.util.spec_from_file_location("bench", os.path.join(ROOT, "bench.py"))
bench = importlib.util.module_from_spec(spec)
spec.loader.exec_module(bench)

from paper_2602_08722_b200 import synth  # noqa: E402


def test_work_model_at_the_32k_and_128k_workloads():
    w = synth.WORKLOADS["llama8b_32k"]
    m = bench.sum_work(w, [w["T"]])
    assert abs(m["sparse_attn"]["flops"] - 4 * 32 * 2048 * 128 * (3932 + 2049 / 2)) < 1
    assert abs(m["sparse_attn"]["flops"] / 1e9 - 166.3) < 0.1
    assert abs(m["dense_attn"]["flops"] / 1e9 - 1133.9) < 0.1
    assert abs(m["score_keys"]["bytes"] / 1e6 - 68.2) < 0.3 and abs(m["score_keys"]["flops"] / 1e9 - 8.59) < 0.01
    assert abs(m["select_queries"]["bytes"] / 1e6 - 17.1) < 0.1      # Q once + Q-bar + the ranks
    assert abs(m["select_keys"]["bytes"] / 1e6 - 1.17) < 0.01
    w = synth.WORKLOADS["long_128k"]
    m = bench.sum_work(w, [w["T"]])
    assert abs(m["sparse_attn"]["flops"] / 1e9 - 1193) < 1
    assert abs(m["dense_attn"]["flops"] / 1e9 - 8933.6) < 1
    assert abs(m["score_keys"]["bytes"] / 1e6 - 272.6) < 0.6 and abs(m["score_keys"]["flops"] / 1e9 - 68.7) < 0.1


def test_budget_fraction_rounds_like_the_library():
    w = dict(synth.WORKLOADS["serving_mix"])
    lens = [8192, 10000, 65536]
    m = bench.sum_work(w, lens)
    want = sum(4 * 32 * 1024 * 128 * (int(0.12 * T + 0.5) + 1025 / 2) for T in lens)
    assert abs(m["sparse_attn"]["flops"] - want) < 1


def test_whole_job_value_counts_every_rank():
    assert bench.job_us_per_chunk(1000.0, 10, 1) == 100.0
    assert bench.job_us_per_chunk(1000.0, 10, 4) == 25.0
    assert bench.max_over_ranks(3.5, 1) == 3.5
