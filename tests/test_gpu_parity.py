"""GPU parity: the CUDA path, called through the C-ABI binding, against the fp64 CPU oracle on
the same seeded inputs.  Outputs within max-abs 1.5e-2 / mean-abs 2e-3 of the oracle; cache pages
bit-exact; rows and slots the call must not touch unchanged."""
import numpy as np
import pytest
import torch

from paper_2604_15464_b200 import binding, build
from paper_2604_15464_b200 import workloads as wl

import rpa_harness as hz

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _dev():
    return torch.device("cuda", 0)


def test_tiny_mixed_batch():
    batch = wl.materialize(wl.workload_meta(1), _dev())
    (mx, mean), info = hz.full_parity(batch)
    assert info["batch_case_name"] == "mixed" and info["gpu_launches"] >= 1


@pytest.mark.parametrize("chunk", [16, 32])
def test_tiny_mixed_batch_split_kv(chunk):
    batch = wl.materialize(wl.workload_meta(1), _dev())
    _, info = hz.full_parity(batch, kv_chunk=chunk)
    assert info["num_combine_groups"] > 0


def test_tiny_mixed_batch_nan_canaries():
    # unmapped pages and every slot at or past the cached context hold NaN before the call
    batch = wl.materialize(wl.workload_meta(1), _dev(), canaries=True)
    hz.full_parity(batch)
    batch = wl.materialize(wl.workload_meta(1), _dev(), canaries=True)
    hz.full_parity(batch, kv_chunk=16)


RAGGED = [
    # q_lens, kv_lens, h_q, h_kv, d, page_size
    ([1, 1, 1], [1, 16, 17], 32, 8, 128, 16),                 # single key; page-aligned; one past
    ([3, 0, 1, 40, 17], [3, 0, 130, 40, 100], 32, 8, 128, 16),  # empty request inside the batch
    ([7, 1, 33], [64, 1, 33], 8, 8, 128, 32),                 # MHA (h_g = 1)
    ([5, 9, 1], [21, 9, 300], 8, 1, 128, 16),                 # MQA (h_g = 8)
    ([2, 19], [50, 19], 16, 1, 64, 16),                       # h_g = 16: one token per item
    ([1, 6, 12], [200, 70, 12], 4, 2, 64, 64),                # d = 64, bigger pages
    ([1] * 9, [5, 31, 32, 33, 47, 48, 49, 255, 257], 32, 8, 128, 128),  # decode around tile/page edges
    ([1, 1, 9, 30], [700, 17, 40, 30], 32, 8, 256, 16),       # d = 256: every sequence on the row kernel
    ([1, 4], [300, 64], 8, 8, 256, 256),                      # d = 256, MHA, page 256
]


@pytest.mark.parametrize("case", RAGGED)
@pytest.mark.parametrize("chunk", [0, 32])
def test_ragged_cases(case, chunk):
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("ragged", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=7,
                         token_capacity=sum(ql) + 3)
    batch = wl.materialize(meta, _dev())
    hz.full_parity(batch, kv_chunk=chunk)


def test_noncausal():
    meta = wl.build_meta("nc", [4, 1, 20], [36, 90, 20], num_q_heads=8, num_kv_heads=2, head_dim=128, page_size=16,
                         seed=9, causal=False)
    hz.full_parity(wl.materialize(meta, _dev()))
    hz.full_parity(wl.materialize(meta, _dev()), kv_chunk=16)


def test_single_key_returns_new_v_exactly():
    meta = wl.build_meta("one", [1, 1, 1], [1, 1, 1], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=3)
    batch = wl.materialize(meta, _dev())
    got, _ = hz.run_gpu(batch)
    v = wl.bf16_bits(batch.new_v)
    for a in range(32):
        assert np.array_equal(got[:3, a], v[:3, a // 4])  # softmax over one key is exactly 1


def test_chunked_prefill_matches_single_prefill():
    hq, hkv, d, ps = 32, 8, 128, 16
    full = wl.materialize(wl.build_meta("full", [150], [150], num_q_heads=hq, num_kv_heads=hkv, head_dim=d,
                                        page_size=ps, seed=21, num_pages=16), _dev())
    got_full, _ = hz.run_gpu(full)
    cache_full = wl.bf16_bits(full.kv_cache)
    # same data, two calls: 90 tokens, then 60 more on the cache the first call produced
    two = wl.materialize(full.meta, _dev())
    rapi = binding.Rpa.for_meta(full.meta)
    out = torch.zeros_like(two.q)
    for (t0, t1) in [(0, 90), (90, 150)]:
        cu = np.array([0, t1 - t0], np.int32)
        kl = np.array([t1], np.int32)
        rapi.rpa_plan(cu, kl)
        rapi.rpa_forward(two.q[t0:t1], two.new_k[t0:t1], two.new_v[t0:t1], two.kv_cache, two.page_table,
                         torch.from_numpy(cu).cuda(), torch.from_numpy(kl).cuda(), out[t0:t1])
    torch.cuda.synchronize()
    assert np.array_equal(wl.bf16_bits(two.kv_cache), cache_full)
    a, b = hz.bf16_to_f64(wl.bf16_bits(out)[:150]), hz.bf16_to_f64(got_full[:150])
    assert np.abs(a - b).max() <= hz.MAX_ABS


def test_plan_mismatch_and_bad_pointers_are_rejected_before_launch():
    meta = wl.workload_meta(1)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    out = torch.zeros_like(batch.q)
    with pytest.raises(binding.RpaError) as e:  # no plan yet
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out)
    assert e.value.status == 4
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    with pytest.raises(binding.RpaError) as e:  # another num_seqs
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, num_seqs=3)
    assert e.value.status == 4
    with pytest.raises(binding.RpaError) as e:  # misaligned q
        rapi.rpa_forward(batch.q.view(-1)[1:], batch.new_k, batch.new_v, batch.kv_cache, batch.page_table,
                         batch.cu_q_lens, batch.kv_lens, out)
    assert e.value.status == 1
    with pytest.raises(binding.RpaError) as e:  # null output
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, None)
    assert e.value.status == 1
    before = wl.bf16_bits(batch.kv_cache).copy()
    torch.cuda.synchronize()
    assert np.array_equal(before, wl.bf16_bits(batch.kv_cache))  # nothing ran


def test_host_buffer_entry_point_matches_device_entry_point():
    meta = wl.workload_meta(1)
    a = wl.materialize(meta, _dev())
    b = wl.materialize(meta, _dev())
    got_dev, _ = hz.run_gpu(a)
    rapi = binding.Rpa.for_meta(meta)
    pin = lambda t: t.cpu().pin_memory()
    out_h = torch.zeros(b.q.shape, dtype=torch.bfloat16).pin_memory()
    rapi.rpa_forward_host(pin(b.q), pin(b.new_k), pin(b.new_v), b.kv_cache, pin(b.page_table), pin(b.cu_q_lens),
                          pin(b.kv_lens), out_h)
    T = meta.num_tokens
    assert np.array_equal(wl.bf16_bits(out_h)[:T], got_dev[:T])
    assert np.array_equal(wl.bf16_bits(a.kv_cache), wl.bf16_bits(b.kv_cache))


def test_ablation_switch_skips_the_cache_update():
    meta = wl.workload_meta(1)
    batch = wl.materialize(meta, _dev())
    before = wl.bf16_bits(batch.kv_cache).copy()
    rapi = binding.Rpa.for_meta(meta)
    rapi.rpa_set_ablation(binding.ABLATE_UPDATE)
    rapi.run_batch(batch)
    torch.cuda.synchronize()
    assert np.array_equal(before, wl.bf16_bits(batch.kv_cache))


# ---- the named Llama-3-8B-shaped workloads at full size, in the launch configuration bench.py times ----

def test_llama_decode_full_batch():
    batch = wl.materialize(wl.workload_meta(2), _dev())
    (mx, mean), info = hz.full_parity(batch)
    assert info["batch_case_name"] == "decode"


def test_llama_prefill_sampled_rows():
    batch = wl.materialize(wl.workload_meta(3), _dev())
    (mx, mean), info = hz.sampled_parity(batch, seqs=[0, 3], rows_per_seq=192, whole_cache=True)
    assert info["batch_case_name"] == "prefill"


def _mixed_sample(meta):
    prefill = [r for r in range(meta.num_seqs) if meta.q_lens[r] > 1]
    decode = [r for r in range(meta.num_seqs) if meta.q_lens[r] == 1]
    return prefill[:3] + decode[:12]


def test_llama_mixed_sampled_rows():
    meta = wl.workload_meta(4)
    batch = wl.materialize(meta, _dev())
    (mx, mean), info = hz.sampled_parity(batch, seqs=_mixed_sample(meta), rows_per_seq=128, whole_cache=True)
    assert info["batch_case_name"] == "mixed" and info["num_tokens"] == 4288


def test_llama_mixed_1000_token_chunks_fill_the_token_capacity():
    # 192 decode requests + 8 chunks of 1000 tokens = 8192 new tokens = the capacity of q / new_k / new_v / out;
    # 1000 is no multiple of a query tile (32 tokens) nor of an item (64)
    meta = wl.workload_meta("4b")
    assert meta.num_tokens == 8192 == meta.token_capacity
    batch = wl.materialize(meta, _dev())
    (mx, mean), info = hz.sampled_parity(batch, seqs=_mixed_sample(meta), rows_per_seq=160, whole_cache=True)
    assert info["batch_case_name"] == "mixed" and info["num_tokens"] == 8192


def _bench_pool_pages():
    """The pool bench.py gives the skewed workload: min(150 GB, 0.8 x free HBM) of 512-KB pages."""
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    return int(min(150e9, 0.8 * free) // (128 * 2 * 8 * 128 * 2))


@pytest.mark.parametrize("sigma", [1.5, 2.0])
def test_skewed_long_decode_sampled_requests(sigma):
    # the timed configuration: mapped pages drawn from the whole ~150 GB pool (only they hold random
    # values; the rest of the pool is a constant)
    meta = wl.workload_meta(5, num_pages=_bench_pool_pages(), sigma=sigma)
    assert meta.page_table.max() > 0.9 * meta.num_pages  # ids reach the far end of the pool
    batch = wl.materialize(meta, _dev())
    order = np.argsort(meta.kv_lens)
    seqs = [int(order[-1]), int(order[-2]), int(order[0]), int(order[len(order) // 2]), int(order[len(order) // 3])]
    (mx, mean), info = hz.sampled_parity(batch, seqs=seqs)
    assert info["num_combine_groups"] > 0  # the longest requests were split
    # slots the call must leave alone: every page of the pool that no request maps still holds the
    # fill constant (the sampled requests' pages were compared with the oracle's, bit for bit, above)
    mapped = torch.zeros(meta.num_pages, dtype=torch.bool, device=_dev())
    mapped[torch.from_numpy(meta.mapped_pages().astype(np.int64)).to(_dev())] = True
    raw = batch.kv_cache.view(torch.int16)
    step = 2048  # pages per pass (1 GB)
    for p0 in range(0, meta.num_pages, step):
        dirty = (raw[p0:p0 + step] != 0x3F00).flatten(1).any(1)
        assert not bool((dirty & ~mapped[p0:p0 + step]).any()), f"an unmapped page near {p0} was written"
    del batch
    torch.cuda.empty_cache()


# ---- edge cases ----

def test_empty_batch_launches_nothing():
    meta = wl.build_meta("empty", [0, 0], [0, 9], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=2,
                         token_capacity=4)
    batch = wl.materialize(meta, _dev())
    before = wl.bf16_bits(batch.kv_cache).copy()
    got, info = hz.run_gpu(batch)
    assert info["gpu_launches"] == 0 and info["batch_case_name"] == "empty"
    assert np.all(got == hz.SENTINEL) and np.array_equal(before, wl.bf16_bits(batch.kv_cache))


@pytest.mark.parametrize("tile_min_q", [None, 1, 10 ** 6])
def test_page_size_256_both_kernels(tile_min_q):
    meta = wl.build_meta("ps256", [1, 70, 1, 300], [700, 330, 256, 300], num_q_heads=32, num_kv_heads=8, head_dim=128,
                         page_size=256, seed=41)
    hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=tile_min_q)


def test_forward_twice_with_one_plan_is_idempotent():
    meta = wl.build_meta("twice", [1, 40, 3], [500, 90, 64], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=42)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    rapi.rpa_set_kv_chunk(64)  # split groups: their arrival tickets must be back at zero for the second call
    out1 = rapi.run_batch(batch).clone()
    cache1 = wl.bf16_bits(batch.kv_cache).copy()
    out2 = torch.zeros_like(batch.q)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, batch.kv_lens,
                     out2)
    torch.cuda.synchronize()
    assert np.array_equal(wl.bf16_bits(out1), wl.bf16_bits(out2))
    assert np.array_equal(cache1, wl.bf16_bits(batch.kv_cache))


def test_runs_on_a_side_stream_at_full_capacity():
    # num_seqs == max_num_seqs and T == max_num_tokens; the work is enqueued on a non-default stream
    meta = wl.build_meta("side", [1, 1, 65, 2], [100, 4096, 65, 18], num_q_heads=32, num_kv_heads=8, head_dim=128,
                         page_size=16, seed=43)
    batch = wl.materialize(meta, _dev())
    host = dict(q=wl.bf16_bits(batch.q), new_k=wl.bf16_bits(batch.new_k), new_v=wl.bf16_bits(batch.new_v),
                kv_cache=wl.bf16_bits(batch.kv_cache).copy(), page_table=meta.page_table, cu_q_lens=meta.cu_q_lens,
                kv_lens=meta.kv_lens)
    from oracle import rpa_oracle as orc
    ref = orc.forward(hz.oracle_shape(meta), **host)
    rapi = binding.Rpa.for_meta(meta)
    side = torch.cuda.Stream()
    out = torch.zeros_like(batch.q)
    torch.cuda.synchronize()
    with torch.cuda.stream(side):
        rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens, side.cuda_stream)
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, side.cuda_stream)
    side.synchronize()
    hz.compare_outputs(wl.bf16_bits(out)[: meta.num_tokens], ref, "side stream")
    assert np.array_equal(wl.bf16_bits(batch.kv_cache), host["kv_cache"])


def test_tile_path_query_lengths_around_the_item_size():
    # one tile item covers 64 tokens at h_g = 4: lengths just below, at and above one and two items
    for ql, ctx in [(63, 0), (64, 128), (65, 5), (128, 256), (129, 1)]:
        meta = wl.build_meta("edge", [ql], [ql + ctx], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=44)
        hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)


def test_bounded_wait_gives_up_and_reports_without_harming_the_context():
    # a wait nothing can satisfy expires after about a millisecond: status word set, kernel returns
    meta = wl.workload_meta(1)
    rapi = binding.Rpa.for_meta(meta)
    assert rapi.rpa_poll_status() == 0
    rapi.rpa_selftest_bounded_wait()
    word = rapi.rpa_poll_status()
    assert word == 0x1000007F
    assert rapi.rpa_poll_status() == 0  # reported once, then cleared
    # the handle and the context keep working
    hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi)


def test_validation_rejects_bad_page_ids_and_length_mismatch_without_touching_memory():
    import dataclasses

    tight = wl.build_meta("val", [1, 40, 3], [500, 90, 64], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                          seed=45, pool_slack=1.0)
    # the tensor holds 8 pages more than the handle is told about, so that an id in that tail is
    # out of range for the library while every address it could form stays inside the allocation
    meta = dataclasses.replace(tight, num_pages=tight.num_pages + 8)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(tight)
    rapi.rpa_set_validation(True)
    table = batch.page_table.clone()
    table[1, 2] = tight.num_pages + 5
    before_cache = wl.bf16_bits(batch.kv_cache).copy()
    out = torch.full(batch.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, table, batch.cu_q_lens, batch.kv_lens, out)
    torch.cuda.synchronize()
    word = rapi.rpa_poll_status()
    assert word & (1 << 29) and (word & 0xFFFFF) == 1  # sequence 1 named
    assert np.all(wl.bf16_bits(out) == hz.SENTINEL) and np.array_equal(before_cache, wl.bf16_bits(batch.kv_cache))
    # device lengths that differ from the planned ones are caught too
    wrong = batch.kv_lens.clone()
    wrong[0] -= 16
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, wrong, out)
    torch.cuda.synchronize()
    assert rapi.rpa_poll_status() & (1 << 29)
    assert np.all(wl.bf16_bits(out) == hz.SENTINEL) and np.array_equal(before_cache, wl.bf16_bits(batch.kv_cache))
    # with consistent inputs the same handle works, validation still on
    hz.full_parity(batch, rapi=rapi)


def test_ablation_switches_for_movement_only_and_arithmetic_only_runs_complete():
    """Bits 2 and 3 of the ablation mask (the paper's "w/o FA" and "w/o DMA" runs) leave the result
    undefined; the calls must complete without touching the status word, the cache update must still
    be exact, and the handle must give exact results again once the mask is cleared."""
    meta = wl.build_meta("abl", [1, 150, 12, 1, 40], [700, 406, 12, 33, 1300], seed=9, **wl.LLAMA3_8B, page_size=16)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    ref_cache = None
    for mask in (4, 8):
        fresh = wl.materialize(meta, _dev())
        rapi.rpa_set_ablation(mask)
        rapi.run_batch(fresh)
        torch.cuda.synchronize()
        assert rapi.rpa_poll_status() == 0
        bits = wl.bf16_bits(fresh.kv_cache)
        ref_cache = bits if ref_cache is None else ref_cache
        assert np.array_equal(bits, ref_cache)
    rapi.rpa_set_ablation(0)
    hz.full_parity(batch, rapi=rapi)
    assert np.array_equal(wl.bf16_bits(batch.kv_cache), ref_cache)


@pytest.mark.parametrize("kv_fp8", [False, True])
def test_very_long_contexts_sampled_rows(kv_fp8):
    # a quarter of a million cached tokens behind one decode row, a chunk of a prefill and a small-q step far
    # into their contexts: positions, page-table rows of 16K entries, split-KV groups of hundreds of
    # partials and tile items with thousands of key blocks
    q_lens = [1, 256, 8, 1]
    kv_lens = [262145, 180256, 150008, 3]
    extra = dict(kv_fp8=True, k_scale=0.03, v_scale=0.03) if kv_fp8 else {}
    meta = wl.build_meta("long", q_lens, kv_lens, page_size=16, seed=91, **wl.LLAMA3_8B, **extra)
    batch = wl.materialize(meta, _dev())
    (mx, mean), info = hz.sampled_parity(batch, seqs=[0, 1, 2, 3], rows_per_seq=48)
    assert info["num_tile_items"] > 0 and info["num_combine_groups"] > 0
