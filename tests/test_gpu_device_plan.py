"""The device-side planner: its lists against the host planner's (integer work: identical up to the
order of row items of equal length), GPU parity of steps planned on the device, replay of a captured
CUDA graph after the lengths changed in place, and detection of bad lengths on the device."""
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


def _lists_match(meta, kv_chunk=0):
    """Plan the same lengths on the host and on the device and compare the lists."""
    host = binding.Rpa.for_meta(meta, device=-1)
    host.rpa_set_kv_chunk(kv_chunk)
    host.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    info = host.rpa_plan_info()
    h_rows, h_tiles, h_groups = host.rpa_plan_dump()
    dev = binding.Rpa.for_meta(meta)
    dev.rpa_set_kv_chunk(kv_chunk)
    cu = torch.tensor(meta.cu_q_lens, dtype=torch.int32, device=_dev())
    kl = torch.tensor(meta.kv_lens, dtype=torch.int32, device=_dev())
    dev.rpa_plan_device(cu, kl)
    counts, d_rows, d_tiles, d_groups = dev.rpa_plan_device_dump(len(h_rows) + 8, len(h_tiles) + 8, len(h_groups) + 8)
    assert dev.rpa_poll_status() == 0 and counts[4] == 0
    assert (counts[0], counts[1], counts[2]) == (len(h_rows), len(h_tiles), len(h_groups))
    assert counts[6] == info["kv_chunk_tokens"]
    # (the host planner may order tile items heaviest first across heads; the device planner keeps head order)
    assert sorted(map(tuple, d_tiles)) == sorted(map(tuple, h_tiles)) and np.array_equal(d_groups, h_groups)
    assert sorted(map(tuple, d_rows)) == sorted(map(tuple, h_rows))
    lens = [-(-(r[5] - r[4]) // 16) for r in d_rows]
    assert lens == sorted(lens, reverse=True), "row items must come longest first"
    if len(h_rows) and len(h_tiles):
        assert 148 // 8 <= counts[3] <= 148 * 5 // 8 or counts[3] == len(h_tiles)
    return counts


def test_device_lists_equal_host_lists():
    _lists_match(wl.workload_meta(2))                      # decode: split groups for the longest requests
    _lists_match(wl.workload_meta(2), kv_chunk=2048)       # more groups
    c = _lists_match(wl.workload_meta(4))                  # mixed: rows and tiles, SM split
    assert c[0] > 0 and c[1] > 0
    _lists_match(wl.workload_meta(3))                      # prefill: tiles only
    meta = wl.build_meta("dp", [1, 5, 0, 40, 3, 1, 700], [33, 29, 0, 300, 3, 5000, 700], seed=2, **wl.LLAMA3_8B, page_size=16)
    _lists_match(meta, kv_chunk=32)
    for n_req, ctx in [(4, 4096), (8, 4096), (16, 2048), (40, 1000)]:  # small batches: the chunk is refined by waves
        small = wl.build_meta("dps", [1] * n_req, [ctx + 1] * n_req, seed=4, **wl.LLAMA3_8B, page_size=16)
        _lists_match(small)
    ql = [10, 20, 30, 40, 8, 5, 5, 300, 1, 1, 1]  # runs of short prompts without context: packed tile items
    packed = wl.build_meta("dpp", ql, [10, 20, 30, 40, 50, 5, 5, 300, 1, 1, 1], seed=6, **wl.LLAMA3_8B, page_size=16)
    _lists_match(packed)
    nc = wl.build_meta("dpn", [4, 1, 20], [36, 900, 20], num_q_heads=8, num_kv_heads=2, head_dim=64, page_size=16,
                       causal=False, seed=3)
    _lists_match(nc, kv_chunk=64)


@pytest.mark.parametrize("seed", range(16))
def test_device_lists_equal_host_lists_on_random_batches(seed):
    """The two planners are separate code (C++ on the host, one CUDA block on the device): seeded
    random batches over head shapes, page sizes, masks and lengths must give the same lists."""
    rng = np.random.default_rng(6000 + seed)
    d = int(rng.choice([64, 128, 256]))
    h_kv = int(rng.choice([1, 2, 8]))
    h_g = int(rng.choice([1, 2, 4, 8, 16]))
    ps = int(rng.choice([16, 32, 48, 64, 128, 256]))
    n = int(rng.integers(1, 40))
    q_lens, kv_lens = [], []
    for _ in range(n):
        kind = int(rng.integers(0, 5))
        if kind == 0:
            q, ctx = 1, int(rng.integers(0, 12000))
        elif kind == 1:
            q, ctx = int(rng.integers(2, 40)), int(rng.integers(0, 3000))
        elif kind == 2:
            q, ctx = int(rng.integers(40, 500)), int(rng.integers(0, 2000))
        elif kind == 3:
            q, ctx = int(rng.integers(1, 40)), 0
        else:
            q, ctx = 0, int(rng.integers(0, 50))
        q_lens.append(q)
        kv_lens.append(q + ctx)
    meta = wl.build_meta(f"dpr{seed}", q_lens, kv_lens, num_q_heads=h_kv * h_g, num_kv_heads=h_kv, head_dim=d, page_size=ps,
                         causal=bool(rng.integers(0, 4) > 0), seed=seed, token_capacity=sum(q_lens) + 4)
    _lists_match(meta)


@pytest.mark.parametrize("cfg", [1, 4])
def test_device_planned_step_matches_oracle(cfg):
    batch = wl.materialize(wl.workload_meta(cfg), _dev(), canaries=(cfg == 1))
    hz.full_parity(batch, device_plan=True)


def test_device_planned_cases():
    for ql, kl, kw in [
        ([1] * 9, [5, 31, 32, 33, 47, 48, 49, 255, 257], dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=128)),
        ([200, 1, 70, 12], [200, 500, 1000, 12], dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)),
        ([33, 300, 1], [60, 700, 90], dict(num_q_heads=16, num_kv_heads=1, head_dim=256, page_size=64)),
        ([3, 0, 1, 40, 17], [3, 0, 130, 40, 100], dict(num_q_heads=4, num_kv_heads=2, head_dim=64, page_size=16)),
        ([10, 20, 30, 7, 9, 64, 3, 3], [10, 20, 30, 7, 9, 64, 3, 3], dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)),
    ]:
        meta = wl.build_meta("dpc", ql, kl, seed=31, token_capacity=sum(ql) + 3, **kw)
        hz.full_parity(wl.materialize(meta, _dev()), device_plan=True, kv_chunk=64)


def test_device_planned_step_on_an_fp8_cache():
    for ql, kl, d in [([1, 1, 40, 200, 5], [900, 33, 300, 200, 29], 128), ([1, 12, 70], [500, 12, 170], 64)]:
        meta = wl.build_meta("dp8", ql, kl, num_q_heads=32, num_kv_heads=8, head_dim=d, page_size=16, seed=33,
                             kv_fp8=True, k_scale=0.03, v_scale=0.025)
        hz.full_parity(wl.materialize(meta, _dev(), canaries=True), device_plan=True)


def test_captured_graph_replays_with_new_lengths():
    """One CUDA graph of [plan on device, attention]; the second replay runs on other lengths, page
    table and inputs written in place into the same buffers."""
    shape = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)
    ql_a, kl_a = [1, 1, 1, 1, 40, 1], [300, 4000, 17, 900, 140, 64]
    ql_b, kl_b = [1, 1, 1, 1, 1, 70], [301, 4001, 2000, 16, 900, 70]
    metas = [wl.build_meta("g", ql, kl, seed=40 + i, num_pages=700, max_pages_per_seq=260, token_capacity=80, **shape)
             for i, (ql, kl) in enumerate([(ql_a, kl_a), (ql_b, kl_b)])]
    batches = [wl.materialize(m, _dev()) for m in metas]
    live = batches[0]  # the buffers the graph is captured on
    rapi = binding.Rpa.for_meta(metas[0])
    out = torch.full(live.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):  # one eager step first: the first calls allocate and set the kernels up
        rapi.rpa_plan_device(live.cu_q_lens, live.kv_lens, stream=side.cuda_stream)
        rapi.rpa_forward(live.q, live.new_k, live.new_v, live.kv_cache, live.page_table, live.cu_q_lens, live.kv_lens,
                         out, stream=side.cuda_stream)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            rapi.rpa_plan_device(live.cu_q_lens, live.kv_lens, stream=side.cuda_stream)
            rapi.rpa_forward(live.q, live.new_k, live.new_v, live.kv_cache, live.page_table, live.cu_q_lens,
                             live.kv_lens, out, stream=side.cuda_stream)
    for i, (meta, src) in enumerate(zip(metas, batches)):
        if i:  # new step: overwrite the captured buffers in place
            for name in ("q", "new_k", "new_v", "kv_cache", "page_table", "cu_q_lens", "kv_lens"):
                getattr(live, name).copy_(getattr(src, name))
        out.view(torch.int16).fill_(hz.SENTINEL)
        host = dict(q=wl.bf16_bits(live.q), new_k=wl.bf16_bits(live.new_k), new_v=wl.bf16_bits(live.new_v),
                    kv_cache=wl.bf16_bits(live.kv_cache).copy(), page_table=meta.page_table, cu_q_lens=meta.cu_q_lens,
                    kv_lens=meta.kv_lens)
        ref = hz.orc.forward(hz.oracle_shape(meta), **host)
        graph.replay()
        torch.cuda.synchronize()
        assert rapi.rpa_poll_status() == 0
        got = wl.bf16_bits(out)
        hz.compare_outputs(got[: meta.num_tokens], ref, f"replay {i}")
        assert np.all(got[meta.num_tokens:] == hz.SENTINEL)
        assert np.array_equal(wl.bf16_bits(live.kv_cache), host["kv_cache"])


def test_device_planner_rejects_bad_lengths():
    meta = wl.build_meta("bad", [1, 4, 1], [40, 30, 9], seed=5, **wl.LLAMA3_8B, page_size=16)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    out = torch.full(batch.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    before = wl.bf16_bits(batch.kv_cache).copy()
    bad = batch.kv_lens.clone()
    bad[1] = 2  # shorter than its query
    rapi.rpa_plan_device(batch.cu_q_lens, bad)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, bad, out)
    torch.cuda.synchronize()
    word = rapi.rpa_poll_status()
    assert word & (1 << 29) and word & (1 << 20)
    assert np.all(wl.bf16_bits(out) == hz.SENTINEL) and np.array_equal(before, wl.bf16_bits(batch.kv_cache))
    hz.full_parity(batch, rapi=rapi, device_plan=True)  # the handle works again with good lengths


def test_device_planner_on_empty_batches():
    shape = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)
    meta = wl.build_meta("dpe", [0, 0, 0], [0, 5, 40], seed=8, token_capacity=4, **shape)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    out = torch.full(batch.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    before = wl.bf16_bits(batch.kv_cache).copy()
    for n in (3, 0):  # three sequences without new tokens; no sequence at all
        rapi.rpa_plan_device(batch.cu_q_lens, batch.kv_lens, num_seqs=n)
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, num_seqs=n)
        torch.cuda.synchronize()
        counts, rows, tiles, groups = rapi.rpa_plan_device_dump(4, 4, 4)
        assert rapi.rpa_poll_status() == 0 and not counts[:6].any()
    assert np.all(wl.bf16_bits(out) == hz.SENTINEL) and np.array_equal(before, wl.bf16_bits(batch.kv_cache))


def test_next_step_planned_on_a_side_stream_while_the_previous_one_runs():
    """The plan of step i+1 is enqueued on a second stream right behind step i's kernels, with no host
    synchronisation in between; the handle keeps two sets of lists and orders them with events.
    Consecutive steps use different batches, so a step reading the wrong set cannot pass."""
    shapes = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, num_pages=700, max_pages_per_seq=80,
                  token_capacity=400)
    metas = [wl.build_meta("sideA", [1, 200, 1, 33], [900, 200, 33, 640], seed=51, **shapes),
             wl.build_meta("sideB", [70, 1, 1, 1], [70, 1270, 512, 17], seed=52, **shapes),
             wl.build_meta("sideC", [1, 1, 5, 300], [100, 1100, 5, 300], seed=53, **shapes)]
    side = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    rapi = binding.Rpa.for_meta(metas[0])
    steps = [0, 1, 2, 1, 0, 2]
    runs = []
    for k in steps:
        batch = wl.materialize(metas[k], _dev())
        host = dict(q=wl.bf16_bits(batch.q), new_k=wl.bf16_bits(batch.new_k), new_v=wl.bf16_bits(batch.new_v),
                    kv_cache=wl.bf16_bits(batch.kv_cache).copy(), page_table=metas[k].page_table,
                    cu_q_lens=metas[k].cu_q_lens, kv_lens=metas[k].kv_lens)
        runs.append((batch, host, torch.full_like(batch.q, float("nan"))))
    torch.cuda.synchronize()
    rapi.rpa_plan_device(runs[0][0].cu_q_lens, runs[0][0].kv_lens, side.cuda_stream)
    for i, (batch, host, out) in enumerate(runs):
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out, main.cuda_stream)
        if i + 1 < len(runs):
            nxt = runs[i + 1][0]
            rapi.rpa_plan_device(nxt.cu_q_lens, nxt.kv_lens, side.cuda_stream)
    torch.cuda.synchronize()
    assert rapi.rpa_poll_status() == 0
    for k, (batch, host, out) in zip(steps, runs):
        ref = hz.orc.forward(hz.oracle_shape(metas[k]), **host)
        T = metas[k].num_tokens
        hz.compare_outputs(wl.bf16_bits(out)[:T], ref, metas[k].name)
        assert np.array_equal(wl.bf16_bits(batch.kv_cache), host["kv_cache"])


def test_a_rejected_step_keeps_later_steps_from_running_until_the_status_is_polled():
    """The status word set by a rejected device-planned step is sticky: every later step returns at once,
    writing neither `out` nor the cache, until rpa_poll_status has reported (and cleared) it.  A loop that
    replays a graph and polls rarely must know that it drops steps meanwhile."""
    shape = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)
    meta = wl.build_meta("sticky", [1, 30, 2], [300, 130, 64], seed=9, **shape)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(meta)
    out = torch.full(batch.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    before = wl.bf16_bits(batch.kv_cache).copy()
    bad_kv = batch.kv_lens.clone()
    bad_kv[1] = 3  # kv_len < q_len
    rapi.rpa_plan_device(batch.cu_q_lens, bad_kv)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, bad_kv, out)
    # a good step right behind it, no poll in between: skipped
    rapi.rpa_plan_device(batch.cu_q_lens, batch.kv_lens)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, batch.kv_lens, out)
    torch.cuda.synchronize()
    assert np.all(wl.bf16_bits(out) == hz.SENTINEL) and np.array_equal(before, wl.bf16_bits(batch.kv_cache))
    assert rapi.rpa_poll_status() & (1 << 29)
    assert rapi.rpa_poll_status() == 0
    hz.full_parity(batch, rapi=rapi, device_plan=True)  # after the poll the same step runs
