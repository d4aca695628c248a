"""The work-counting formulas reproduce the numbers the paper prints in its appendix tables."""
import os

import numpy as np
import pytest

from paper_2604_15464_b200 import metrics

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


def test_decode_table_reproduced():
    # latencies are printed to the microsecond, so allow the rounding of the shortest one (0.5/137)
    for ctx, us, gbs, mbu in _rows("paper_decode_d128.txt"):
        got = metrics.paper_decode_throughput(128, int(ctx), 32, 8, 128, us * 1e-6)
        assert got == pytest.approx(gbs, rel=0.5 / us + 1e-3)
        assert 100 * metrics.utilisation(got, 7380.0) == pytest.approx(mbu, rel=0.5 / us + 1e-3)


def test_noncausal_prefill_table_reproduced():
    for s, us, tf, mfu in _rows("paper_prefill_noncausal_d128.txt"):
        got = metrics.paper_prefill_speed(int(s), 32, 128, us * 1e-6, causal=False)
        assert got == pytest.approx(tf, rel=0.5 / us + 2e-3)
        assert 100 * metrics.utilisation(got, 2307.0 * 0.5) == pytest.approx(mfu, rel=0.5 / us + 2e-3)


def test_causal_prefill_table_consistent_with_one_block_size():
    # c_kv is not printed; the long rows must all be explained by one value near 1024
    solved = []
    for s, us, tf, _ in _rows("paper_prefill_causal_d128.txt"):
        if s >= 4096:
            solved.append(tf * 1e12 * us * 1e-6 / (2 * s * 32 * 128) - s)
    assert max(solved) - min(solved) < 64 and 960 < np.mean(solved) < 1090
    for s, us, tf, mfu in _rows("paper_prefill_causal_d128.txt"):
        if s >= 4096:
            got = metrics.paper_prefill_speed(int(s), 32, 128, us * 1e-6, causal=True, c_kv=1024)
            assert got == pytest.approx(tf, rel=5e-3)
            assert 100 * got / (2307.0 * 0.5) == pytest.approx(mfu, rel=5e-3)


def test_ragged_forms_reduce_to_the_uniform_ones():
    n, ctx = 128, 4096
    b = metrics.algorithmic_bytes([1] * n, [ctx] * n, 32, 8, 128)
    assert b / 1024 ** 3 / 1e-3 == pytest.approx(metrics.paper_decode_throughput(n, ctx, 32, 8, 128, 1e-3))
    s = 2048
    assert metrics.attention_flops([s], [s], 32, 128, causal=False) == 4 * s * s * 32 * 128
    assert metrics.attention_flops([s], [s], 32, 128, causal=True) == 4 * 32 * 128 * (s * (s + 1) // 2)
    # chunked prefill: 3 new tokens on 5 cached ones see 6 + 7 + 8 keys
    assert metrics.attention_flops([3], [8], 1, 1, causal=True) == 4 * (6 + 7 + 8)


def test_bench_cpu_baseline_leg_runs_on_bf16_and_fp8_caches():
    """bench.py's cpu_baseline leg (the oracle on a bounded sample) on a small batch, for both cache
    types: the sample must cover the batch and its units must be the batch's own."""
    import sys
    import os
    import torch

    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import bench
    from paper_2604_15464_b200 import workloads as wl

    for fp8 in (False, True):
        extra = dict(kv_fp8=True, k_scale=0.05, v_scale=0.05) if fp8 else {}
        meta = wl.build_meta("cpu_leg", [1, 5, 1], [40, 5, 130], num_q_heads=8, num_kv_heads=2, head_dim=64, page_size=16,
                             seed=3, **extra)
        batch = wl.materialize(meta, torch.device("cpu"))
        dt, units, what, cores, _ = bench.oracle_sample(meta, batch, budget_s=1.0)
        assert dt > 0 and cores >= 1 and what.startswith("3 of 3 requests")
        assert units["tokens"] == 7
        kv_bytes = 1 if fp8 else 2
        want = sum((L + q) * 2 * 2 * 64 * kv_bytes + q * 2 * 8 * 64 * 2 for q, L in zip([1, 5, 1], [40, 5, 130]))
        assert abs(units["GB"] * 1e9 - want) < 1
