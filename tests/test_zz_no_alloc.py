"""rpa_forward_static, the entry point for callers that cannot allocate device memory (a server
whose own pool already owns all of HBM, or a loop that cannot take cudaMalloc's synchronisation).

It must give what the handle-based entry points give, out of the library's built-in scratch array,
on consecutive calls that share that array; and, like them, it must match the fp64 oracle: every
output row within the tolerance, every cache byte exactly.  This file sorts last so that a run that
stops at the first failure has already run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import rpa_oracle as orc
from paper_2604_15464_b200 import binding, build
from paper_2604_15464_b200 import workloads as wl

import rpa_harness as hz

pytestmark = pytest.mark.gpu


def _config(meta):
    return binding.RpaConfig(meta.num_q_heads, meta.num_kv_heads, meta.head_dim, meta.page_size, meta.num_pages,
                             meta.max_pages_per_seq, max(meta.num_seqs, 1), max(meta.token_capacity, 1), meta.scale,
                             meta.causal, meta.kv_fp8, meta.k_scale, meta.v_scale, meta.q_scale)


def _run_static(meta, stream=None):
    """One batch through the static entry point; returns (output bits, cache bits after the call,
    the oracle's outputs, the oracle's cache)."""
    dev = torch.device("cuda", 0)
    b = wl.materialize(meta, dev)
    host = dict(q=wl.bf16_bits(b.q), new_k=wl.bf16_bits(b.new_k), new_v=wl.bf16_bits(b.new_v),
                kv_cache=wl.bf16_bits(b.kv_cache).copy(), page_table=meta.page_table, cu_q_lens=meta.cu_q_lens,
                kv_lens=meta.kv_lens)
    ref = orc.forward(hz.oracle_shape(meta), **host)  # updates host["kv_cache"] as the call must
    out = torch.full(b.q.shape, hz.SENTINEL, dtype=torch.int16, device=dev).view(torch.bfloat16)
    torch.cuda.synchronize()
    if stream is None:
        binding.rpa_forward_static(_config(meta), b.q, b.new_k, b.new_v, b.kv_cache, b.page_table, b.cu_q_lens,
                                   b.kv_lens, meta.cu_q_lens, meta.kv_lens, out)
    else:
        with torch.cuda.stream(stream):
            binding.rpa_forward_static(_config(meta), b.q, b.new_k, b.new_v, b.kv_cache, b.page_table, b.cu_q_lens,
                                       b.kv_lens, meta.cu_q_lens, meta.kv_lens, out, stream.cuda_stream)
    torch.cuda.synchronize()
    return wl.bf16_bits(out), wl.bf16_bits(b.kv_cache), ref, host["kv_cache"]


def _check_against_oracle(meta, stream=None):
    got, cache, ref, ref_cache = _run_static(meta, stream)
    T = meta.num_tokens
    hz.compare_outputs(got[:T], ref, meta.name)
    assert np.all(got[T:] == hz.SENTINEL), "rows past the last token were written"
    assert np.array_equal(cache, ref_cache), "cache differs from the oracle's (must be bit-exact)"
    return got, cache


def test_static_entry_point_matches_handle_and_oracle_on_two_calls_in_a_row():
    build.build()
    # few long requests: the planner splits their KV ranges, so the scratch partials are in play
    first = wl.build_meta("long_decode", [1, 1, 1, 1, 3], [3000, 4100, 5000, 6000, 2500], num_q_heads=32,
                          num_kv_heads=8, head_dim=128, page_size=16, seed=31, token_capacity=9)
    second = wl.build_meta("other_batch", [1, 2, 1], [7000, 900, 33], num_q_heads=32, num_kv_heads=8, head_dim=128,
                           page_size=16, seed=32, token_capacity=6)
    for meta in (first, second):  # the second call finds the first call's leftovers in the scratch
        got_static, cache_static = _check_against_oracle(meta)
        a = wl.materialize(meta, torch.device("cuda", 0))  # same seed: identical bits, separate cache
        got_handle, info = hz.run_gpu(a)
        assert info["num_combine_groups"] > 0
        T = meta.num_tokens
        x, y = hz.bf16_to_f64(got_handle[:T]), hz.bf16_to_f64(got_static[:T])
        err = np.abs(x - y)
        assert err.max() <= hz.MAX_ABS and err.mean() <= hz.MEAN_ABS
        assert np.array_equal(wl.bf16_bits(a.kv_cache), cache_static)


@pytest.mark.parametrize("shape", [
    dict(num_q_heads=16, num_kv_heads=1, head_dim=64, causal=True),    # d_k = 64, 16 grouped heads
    dict(num_q_heads=4, num_kv_heads=4, head_dim=64, causal=True),     # no grouping
    dict(num_q_heads=32, num_kv_heads=8, head_dim=128, causal=False),  # no causal mask
    dict(num_q_heads=16, num_kv_heads=2, head_dim=128, causal=True),   # 8 grouped heads
])
def test_static_entry_point_other_shapes_against_the_oracle(shape):
    build.build()
    meta = wl.build_meta("static_shape", [1, 5, 1, 20, 2], [2100, 300, 17, 20, 1500], page_size=32, seed=33, **shape)
    _check_against_oracle(meta)


def test_static_entry_point_on_a_side_stream():
    build.build()
    meta = wl.build_meta("static_side", [1, 1, 4], [5000, 640, 90], num_q_heads=32, num_kv_heads=8, head_dim=128,
                         page_size=16, seed=34)
    _check_against_oracle(meta, stream=torch.cuda.Stream())


def test_static_entry_point_rejects_batches_beyond_its_scratch():
    build.build()
    meta = wl.workload_meta(3)  # 4 x 8192-token prefill: far more work items than the scratch holds
    lib = binding.load_library()
    cfg = _config(meta)._c()
    cu = np.ascontiguousarray(meta.cu_q_lens, np.int32)
    kl = np.ascontiguousarray(meta.kv_lens, np.int32)
    st = lib.rpa_forward_static(ctypes.byref(cfg), 16, 16, 16, 16, 16, 16, 16, cu.ctypes.data, kl.ctypes.data, 4, 16, None)
    assert st == 3  # RPA_ERR_CAPACITY, before anything is launched


def test_static_entry_point_rejects_what_it_has_no_kernel_for():
    build.build()
    lib = binding.load_library()
    cu, kl = np.array([0, 1], np.int32), np.array([40], np.int32)
    for meta in (wl.build_meta("d256", [1], [40], num_q_heads=32, num_kv_heads=8, head_dim=256, page_size=16, seed=35),
                 wl.build_meta("fp8", [1], [40], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=36,
                               kv_fp8=True, k_scale=0.03, v_scale=0.03)):
        cfg = _config(meta)._c()
        st = lib.rpa_forward_static(ctypes.byref(cfg), 16, 16, 16, 16, 16, 16, 16, cu.ctypes.data, kl.ctypes.data, 1, 16, None)
        assert st == 2  # RPA_ERR_UNSUPPORTED, before any device work


def test_static_entry_point_refuses_a_capturing_stream():
    """Its work lists are copied from ordinary host memory that the next call overwrites; a captured
    copy would re-read that memory at every replay.  The call must refuse and leave no node behind."""
    build.build()
    meta = wl.build_meta("static_cap", [1, 1], [300, 40], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=37)
    dev = torch.device("cuda", 0)
    b = wl.materialize(meta, dev)
    out = torch.zeros_like(b.q)
    # (the first call on the device happened in the tests above or happens here, outside any capture)
    binding.rpa_forward_static(_config(meta), b.q, b.new_k, b.new_v, b.kv_cache, b.page_table, b.cu_q_lens, b.kv_lens,
                               meta.cu_q_lens, meta.kv_lens, out)
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    marker = torch.zeros(4, device=dev)
    with torch.cuda.graph(graph, stream=side):
        marker += 1  # so that the capture holds something
        with pytest.raises(binding.RpaError) as err:
            binding.rpa_forward_static(_config(meta), b.q, b.new_k, b.new_v, b.kv_cache, b.page_table, b.cu_q_lens,
                                       b.kv_lens, meta.cu_q_lens, meta.kv_lens, out, side.cuda_stream)
    assert err.value.status == 2
    graph.replay()
    torch.cuda.synchronize()
    assert float(marker[0]) >= 1.0  # the context is intact and the graph runs
