"""CPU-only checks of the C-ABI library: it loads, exports what the header declares, validates
arguments, and its planner covers every (query row, key) pair exactly once with one cache writer
per new token.  No compute call is made (planning-only handles, device = -1)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2604_15464_b200 import binding, build, metrics
from paper_2604_15464_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "rpa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(rpa_[a-z_0-9]+)\s*\(", header))
    assert declared and declared == set(binding.EXPORTS) | (declared - set(binding.EXPORTS))
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in rpa.h but not exported"
    assert set(binding.EXPORTS) <= declared


def test_status_strings():
    lib = binding.load_library()
    assert lib.rpa_status_string(0) == b"ok"
    assert len({lib.rpa_status_string(i) for i in range(7)}) == 7


def _plan_only(meta, **over):
    return binding.Rpa.for_meta(meta, device=-1, **over)


def test_create_rejects_bad_shapes():
    ok = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, num_pages=64, max_pages_per_seq=8,
              max_num_seqs=4, max_num_tokens=64)
    binding.Rpa(binding.RpaConfig(**ok), device=-1).close()
    for bad, status in [(dict(num_q_heads=30), 1), (dict(head_dim=96), 2), (dict(page_size=24), 2),
                        (dict(num_pages=0), 1), (dict(num_q_heads=24, num_kv_heads=8), 2), (dict(max_num_seqs=0), 1)]:
        with pytest.raises(binding.RpaError) as e:
            binding.Rpa(binding.RpaConfig(**{**ok, **bad}), device=-1)
        assert e.value.status == status


def test_plan_rejects_bad_lengths_and_capacity():
    meta = wl.workload_meta(1)
    r = _plan_only(meta)
    with pytest.raises(binding.RpaError) as e:
        r.rpa_plan([0, 1, 2, 14, 19], [33, 7, 11, 29])  # kv_len < q_len
    assert e.value.status == 1
    with pytest.raises(binding.RpaError) as e:
        r.rpa_plan([0, 1, 2, 14, 19], [33, 7, 12, 65])  # needs 5 pages, table rows hold 4
    assert e.value.status == 3
    with pytest.raises(binding.RpaError) as e:
        r.rpa_plan([0, 1, 2, 14, 19, 20], [33, 7, 12, 29, 1])  # 5 sequences, capacity 4
    assert e.value.status == 3
    with pytest.raises(binding.RpaError) as e:
        r.rpa_plan([0, 1, 2, 14, 40], [33, 7, 12, 40])  # 40 tokens, capacity 19
    assert e.value.status == 3
    with pytest.raises(binding.RpaError) as e:
        r.rpa_plan_info()  # a failed plan leaves no plan behind
    assert e.value.status == 4


def test_forward_without_device_fails_loudly():
    meta = wl.workload_meta(1)
    r = _plan_only(meta)
    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    lib = binding.load_library()
    st = lib.rpa_forward(r._h, 16, 16, 16, 16, 16, 16, 16, meta.num_seqs, 16, None)
    assert st == 5  # RPA_ERR_CUDA: there is no CPU fallback


def _check_plan(meta, rapi, causal=True):
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    info = rapi.rpa_plan_info()
    rows, tiles, groups = rapi.rpa_plan_dump()
    h_g = meta.num_q_heads // meta.num_kv_heads
    cu = meta.cu_q_lens
    # coverage[(seq, tok, kv_head)] -> sorted list of [begin, end)
    cover, writers = {}, {}
    partial_owner = {}
    for seq, h, t0, nt, b, e, partial, flags in rows:
        assert 0 < nt <= 16 // h_g and b % 16 == 0 and 0 <= b < e
        ctx = int(meta.kv_lens[seq] - meta.q_lens[seq])
        assert t0 + nt <= meta.q_lens[seq]
        vis_end = ctx + t0 + nt if causal else int(meta.kv_lens[seq])
        assert e <= vis_end
        for j in range(nt):
            cover.setdefault((seq, t0 + j, h), []).append((b, e))
            if flags & 1:
                writers[(seq, t0 + j, h)] = writers.get((seq, t0 + j, h), 0) + 1
        if partial >= 0:
            assert partial not in partial_owner
            partial_owner[partial] = (seq, h, t0, nt)
    for seq, h, t0, nt, flags, n_seqs, *_ in tiles:
        if flags & 2:  # packed item: n_seqs whole sequences without context, first one = seq
            assert t0 == 0 and 2 <= n_seqs <= 64 and nt == cu[seq + n_seqs] - cu[seq]
            for r in range(seq, seq + n_seqs):
                assert meta.kv_lens[r] == meta.q_lens[r] >= 1
                for j in range(int(meta.q_lens[r])):
                    cover.setdefault((r, j, h), []).append((0, int(meta.kv_lens[r])))
                    writers[(r, j, h)] = writers.get((r, j, h), 0) + 1
            continue
        for j in range(nt):
            ctx = int(meta.kv_lens[seq] - meta.q_lens[seq])
            vis_end = ctx + t0 + nt if causal else int(meta.kv_lens[seq])
            cover.setdefault((seq, t0 + j, h), []).append((0, vis_end))
            if flags & 1:
                writers[(seq, t0 + j, h)] = writers.get((seq, t0 + j, h), 0) + 1
    n_rows = 0
    for r in range(meta.num_seqs):
        ctx = int(meta.kv_lens[r] - meta.q_lens[r])
        for i in range(int(meta.q_lens[r])):
            for h in range(meta.num_kv_heads):
                spans = sorted(cover[(r, i, h)])
                need = ctx + i + 1 if causal else int(meta.kv_lens[r])
                assert spans[0][0] == 0
                for (b0, e0), (b1, e1) in zip(spans, spans[1:]):
                    assert e0 == b1, "ranges must tile the visible keys without gap or overlap"
                assert spans[-1][1] >= need
                assert writers.get((r, i, h), 0) == 1, "exactly one cache writer per (token, kv head)"
                n_rows += 1
    assert n_rows == meta.num_tokens * meta.num_kv_heads
    # combine groups own exactly the partial slots of their items
    seen = set()
    for out_tok0, nt, h, first, n, *_ in groups:
        assert n >= 2
        for k in range(first, first + n):
            assert k in partial_owner and k not in seen
            seen.add(k)
            seq, ph, t0, pnt = partial_owner[k]
            assert ph == h and cu[seq] + t0 == out_tok0 and pnt == nt
    assert seen == set(partial_owner)
    # longest-first order
    lens = [-(-(e - b) // 16) for _, _, _, _, b, e, _, _ in rows]
    assert lens == sorted(lens, reverse=True)
    assert info["algorithmic_bytes"] == metrics.algorithmic_bytes(meta.q_lens, meta.kv_lens, meta.num_q_heads,
                                                                   meta.num_kv_heads, meta.head_dim)
    assert info["algorithmic_flops"] == metrics.attention_flops(meta.q_lens, meta.kv_lens, meta.num_q_heads,
                                                                 meta.head_dim, causal)
    return info, rows, groups


@pytest.mark.parametrize("chunk", [0, 16, 32])
def test_plan_covers_tiny_mixed_batch(chunk):
    meta = wl.workload_meta(1)
    r = _plan_only(meta)
    r.rpa_set_kv_chunk(chunk)
    info, rows, groups = _check_plan(meta, r)
    assert info["batch_case_name"] == "mixed" and info["num_decode_seqs"] == 2 and info["num_prefill_seqs"] == 2
    assert info["gpu_launches"] == 1  # split groups are merged inside the row kernel: no combine launch
    assert (len(groups) == 0) == (chunk == 0)
    # every split item names its combine group in the upper flag bits, unsplit items name none
    for seq, h, t0, nt, b, e, partial, flags in rows:
        group = (flags >> 8) - 1
        if partial < 0:
            assert group == -1
        else:
            first, n = groups[group][3], groups[group][4]
            assert first <= partial < first + n


def test_plan_classifies_and_covers_named_workloads():
    for cfg, case in [(2, "decode"), (4, "mixed"), (5, "decode")]:
        meta = wl.workload_meta(cfg)
        r = _plan_only(meta)
        info, rows, groups = _check_plan(meta, r)
        assert info["batch_case_name"] == case
        assert info["num_tokens"] == meta.num_tokens
    # the skewed workload must split its longest requests
    assert len(groups) > 0


def test_plan_noncausal_and_empty_sequences():
    meta = wl.build_meta("nc", [3, 0, 1, 40], [3, 0, 130, 40], num_q_heads=8, num_kv_heads=2, head_dim=64, page_size=16,
                         causal=False, seed=1)
    r = _plan_only(meta)
    r.rpa_set_kv_chunk(32)
    _check_plan(meta, r, causal=False)
    empty = wl.build_meta("e", [0, 0], [0, 5], num_q_heads=4, num_kv_heads=2, head_dim=64, page_size=16, seed=1)
    r = _plan_only(empty)
    r.rpa_plan(empty.cu_q_lens, empty.kv_lens)
    info = r.rpa_plan_info()
    assert info["batch_case_name"] == "empty" and info["num_row_items"] == 0 and info["gpu_launches"] == 0


def test_plan_packs_runs_of_short_sequences_without_context():
    # runs: (10, 20, 30) fills 60 of 64 tokens; 40 alone (next one has context); (5, 5) after it; a long one; (1, 1, 1)
    ql = [10, 20, 30, 40, 8, 5, 5, 300, 1, 1, 1]
    kl = [10, 20, 30, 40, 50, 5, 5, 300, 1, 1, 1]
    meta = wl.build_meta("pack", ql, kl, seed=3, **wl.LLAMA3_8B, page_size=16)
    r = _plan_only(meta)
    info, rows, groups = _check_plan(meta, r)
    _, tiles, _ = r.rpa_plan_dump()
    packed = [(int(t[0]), int(t[5]), int(t[3])) for t in tiles if t[4] & 2 and t[1] == 0]
    assert packed == [(0, 3, 60), (5, 2, 10), (8, 3, 3)]
    # the sequence with cached context and the long one are not packed; 40 alone is an ordinary tile item
    assert any(t[0] == 3 and not t[4] & 2 for t in tiles) and any(t[0] == 7 and not t[4] & 2 for t in tiles)
    assert all(rw[0] == 4 for rw in rows)  # only the 8-token chunk on 42 tokens of context runs on the row kernel
    # an FP8 cache (head_dim 128 has a tile kernel for it) packs the same runs
    meta8 = wl.build_meta("pack8", ql, kl, seed=3, **wl.LLAMA3_8B, page_size=16, kv_fp8=True, k_scale=0.1, v_scale=0.1)
    r8 = _plan_only(meta8)
    r8.rpa_plan(meta8.cu_q_lens, meta8.kv_lens)
    assert [(int(t[0]), int(t[5]), int(t[3])) for t in r8.rpa_plan_dump()[1] if t[4] & 2 and t[1] == 0] == packed
    # an explicit "rows only" setting does not pack
    r.rpa_set_tile_min_q(10 ** 6)
    _check_plan(meta, r)
    assert len(r.rpa_plan_dump()[1]) == 0


def test_split_kv_chunk_rules():
    """The chunk is half a resident CTA's share of the streamed keys; uniform batches are not split
    for nothing; small batches are cut so that their items fill whole waves of the 296 resident CTAs."""
    def plan(q_lens, kv_lens):
        meta = wl.build_meta("chunk", q_lens, kv_lens, seed=1, **wl.LLAMA3_8B, page_size=256)
        r = _plan_only(meta)
        info, rows, groups = _check_plan(meta, r)
        return info, rows, groups

    info, rows, groups = plan([1] * 128, [513] * 128)      # 1024 units of 513 keys on 296 slots: left whole
    assert info["num_row_items"] == 1024 and len(groups) == 0
    info, rows, groups = plan([1] * 128, [4097] * 128)
    assert info["num_row_items"] == 1024 and len(groups) == 0
    info, rows, groups = plan([1] * 8, [4097] * 8)          # 64 units: cut into parts that fill two waves, not 2.2
    assert 296 < info["num_row_items"] <= 2 * 296 and len(groups) == 64
    info, rows, groups = plan([1] * 4, [4097] * 4)          # 32 units: one wave
    assert info["num_row_items"] <= 296 and len(groups) == 32
    # one very long request among short ones is the only one split
    info, rows, groups = plan([1] * 256, [100000] + [1000] * 255)
    assert len(groups) == 8 and all(g[4] >= 2 for g in groups)
    long_parts = [r for r in rows if r[0] == 0]
    assert len(long_parts) == sum(g[4] for g in groups) and max(r[5] - r[4] for r in rows) <= info["kv_chunk_tokens"]


def test_fp8_lists_of_decode_sized_items_are_planned_for_more_resident_ctas():
    """With an FP8 cache and at most 8 grouped heads, a list whose items all have at most 8 query rows
    runs on a leaner instantiation of the row kernel (4 CTAs per SM at head_dim 128 instead of 3): the
    planner then fills 592 slots instead of 444.  One sequence with three new tokens (12 rows) turns
    the whole list back."""
    def chunk_and_items(q_lens, kv_lens, fp8):
        extra = dict(kv_fp8=True, k_scale=0.1, v_scale=0.1) if fp8 else {}
        meta = wl.build_meta("slots", q_lens, kv_lens, seed=2, **wl.LLAMA3_8B, page_size=16, **extra)
        r = _plan_only(meta)
        r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        info = r.rpa_plan_info()
        return info["kv_chunk_tokens"], info["num_row_items"]

    kv = [6000] * 40
    narrow = chunk_and_items([1] * 40, kv, True)          # 320 units of 6000 keys, cut for 592 slots
    wide = chunk_and_items([1] * 39 + [3], kv, True)      # ... for 444 slots
    assert narrow[0] < wide[0] and narrow[1] > wide[1] and narrow[1] % 8 == 0
    two_tokens = chunk_and_items([2] * 40, [6001] * 40, True)   # 2 tokens x 4 heads = 8 rows: still narrow
    assert two_tokens == narrow


def test_rpa_log_prints_one_plan_summary_per_call():
    """RPA_LOG=1 in the environment: rpa_plan describes on stderr what it made of the batch."""
    import subprocess
    import sys

    code = ("import sys; sys.path.insert(0, %r)\n"
            "from paper_2604_15464_b200 import binding, build, workloads as wl\n"
            "build.build()\n"
            "for cfg in (2, 4):\n"
            "    meta = wl.workload_meta(cfg)\n"
            "    r = binding.Rpa.for_meta(meta, device=-1)\n"
            "    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)\n" % ROOT)
    env = dict(os.environ, RPA_LOG="1")
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-1500:]
    lines = [l for l in res.stderr.splitlines() if l.startswith("[rpa] plan:")]
    assert len(lines) == 2
    assert "decode batch, 256 seqs (256 decode, 0 prefill), 256 new tokens" in lines[0] and "tile kernel 0 items" in lines[0]
    assert "mixed batch, 200 seqs (192 decode, 8 prefill), 4288 new tokens" in lines[1]
    quiet = subprocess.run([sys.executable, "-c", code], env={k: v for k, v in os.environ.items() if k != "RPA_LOG"},
                           capture_output=True, text=True, timeout=600)
    assert "[rpa] plan:" not in quiet.stderr


@pytest.mark.parametrize("seed", range(40))
def test_plan_invariants_on_random_batches(seed):
    """Seeded random batches through the host planner: whatever the shapes, page size, routing threshold,
    split chunk and mask, the work lists must tile every row's visible keys exactly once, name exactly
    one cache writer per (token, KV head), give every split item a partial slot of its own and every
    combine group exactly its items' slots, keep the row list longest-first, and count the paper's
    bytes and FLOPs (Sections 4.1.1 and 4.2.1)."""
    rng = np.random.default_rng(4000 + seed)
    d = int(rng.choice([64, 128, 256]))
    h_kv = int(rng.choice([1, 2, 8]))
    h_g = int(rng.choice([1, 2, 4, 8, 16]))
    ps = int(rng.choice([16, 32, 48, 64, 128, 256]))
    causal = bool(rng.integers(0, 4) > 0)
    n = int(rng.integers(1, 12))
    q_lens, kv_lens = [], []
    for _ in range(n):
        kind = int(rng.integers(0, 5))
        if kind == 0:
            q, ctx = 1, int(rng.integers(0, 20000))
        elif kind == 1:
            q, ctx = int(rng.integers(2, 40)), int(rng.integers(0, 3000))
        elif kind == 2:
            q, ctx = int(rng.integers(40, 700)), int(rng.integers(0, 2000))
        elif kind == 3:
            q, ctx = int(rng.integers(1, 40)), 0  # short prompt without context: may share a packed item
        else:
            q, ctx = 0, int(rng.integers(0, 50))
        q_lens.append(q)
        kv_lens.append(q + ctx)
    meta = wl.build_meta(f"rp{seed}", q_lens, kv_lens, num_q_heads=h_kv * h_g, num_kv_heads=h_kv, head_dim=d, page_size=ps,
                         causal=causal, seed=seed, token_capacity=sum(q_lens) + int(rng.integers(0, 9)))
    r = _plan_only(meta)
    chunk = int(rng.choice([0, 0, 256, 1024, 4096]))
    if chunk:
        r.rpa_set_kv_chunk(chunk)
    threshold = rng.choice([None, None, 1, 8, 10 ** 6])
    if threshold is not None:
        r.rpa_set_tile_min_q(int(threshold))
    if sum(q_lens) == 0:
        r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        assert r.rpa_plan_info()["batch_case_name"] == "empty"
        return
    try:
        info, rows, groups = _check_plan(meta, r, causal=causal)
    except binding.RpaError as e:
        # a forced small chunk on long contexts may need more split partials than the handle was sized
        # for: that is a clean refusal; the automatic chunk never does
        assert e.status == 3 and chunk != 0
        r.rpa_set_kv_chunk(0)
        info, rows, groups = _check_plan(meta, r, causal=causal)
    assert info["num_tokens"] == sum(q_lens)
    if threshold == 10 ** 6:
        assert info["num_tile_items"] == 0


def test_short_item_instantiation_is_chosen_by_the_longest_tile_routed_sequence():
    """The two-tile kernel's instantiation for short items: chosen when every sequence on the tile path has at
    most 256 key positions (2: at most 64; decode rows, which go to the row kernel, do not count), never for an FP8
    cache."""
    build.build()
    shape = dict(seed=3, page_size=16, **wl.LLAMA3_8B)
    for ql, kl, want in (([64] * 5, [64] * 5, 2), ([128, 200, 16], [128, 256, 16], 1), ([64, 1, 1], [64, 3000, 900], 2), ([65], [65], 1),
                         ([64, 40], [64, 257], 0), ([300], [300], 0), ([1, 1], [500, 700], 0)):
        meta = wl.build_meta("short_rule", ql, kl, **shape)
        r = binding.Rpa.for_meta(meta, device=-1)
        r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        info = r.rpa_plan_info()
        assert info["tile_short_items"] == want and (info["tile_kernel"] == 1 or not want)
        r.close()
    meta = wl.build_meta("short_rule_fp8", [64] * 5, [64] * 5, kv_fp8=True, k_scale=0.03, v_scale=0.03, **shape)
    r = binding.Rpa.for_meta(meta, device=-1)
    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    assert r.rpa_plan_info()["tile_short_items"] == 0
    r.close()


def test_pair_kernel_plans_cover_every_token_once_with_items_of_four_tiles():
    """rpa_set_tile_pair(1) on a handle without a device: the plan's tile items hold up to four query tiles
    (128 tokens at h_g = 4), never packed, one cache writer per (token, KV head), and the plan says which
    kernel would run them; the default mode leaves plans of such handles on the two-tile kernel's items."""
    build.build()
    meta = wl.build_meta("pair_plan", [300, 64, 1, 129, 17], [811, 64, 500, 129, 17], seed=3, page_size=16, **wl.LLAMA3_8B)
    r = binding.Rpa.for_meta(meta, device=-1)
    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    info = r.rpa_plan_info()
    assert info["tile_kernel"] == 1
    default_tiles = info["num_tile_items"]
    r.rpa_set_tile_pair(1)
    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    info = r.rpa_plan_info()
    rows, tiles, _ = r.rpa_plan_dump()
    assert info["tile_kernel"] == 3 and 0 < info["num_tile_items"] < default_tiles
    written = set()
    for seq, head, tok0, n_tok, flags, n_seqs, _, _ in tiles:
        assert 1 <= n_tok <= 128 and tok0 % 128 == 0 and not flags & 2  # kFlagPacked
        assert tok0 + n_tok <= meta.q_lens[seq]
        if flags & 1:  # kFlagWriteKv
            for t in range(tok0, tok0 + n_tok):
                assert (seq, head, t) not in written
                written.add((seq, head, t))
    for seq, head, tok0, n_tok, kv_begin, kv_end, partial, flags in rows:
        if flags & 1:
            for t in range(tok0, tok0 + n_tok):
                assert (seq, head, t) not in written
                written.add((seq, head, t))
    assert len(written) == meta.num_kv_heads * meta.num_tokens
    r.rpa_set_tile_pair(0)
    r.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    assert r.rpa_plan_info()["num_tile_items"] == default_tiles
    with pytest.raises(binding.RpaError):
        r.rpa_set_tile_pair(7)
    r.close()
