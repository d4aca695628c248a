"""The CTA-pair tile kernel (rpa_set_tile_pair(1)): two CTAs on neighbouring SMs run one item of four
query tiles, each staging half of every key block.  Same bar as every other path: outputs within the
tolerance of the fp64 oracle, cache bytes identical, rows past the batch untouched."""
import numpy as np
import pytest
import torch

from paper_2604_15464_b200 import binding
from paper_2604_15464_b200 import workloads as wl

import rpa_harness as hz
from test_gpu_tile_kernel import TILE_CASES

pytestmark = pytest.mark.gpu


def _dev():
    return torch.device("cuda", 0)


def _pair_api(meta):
    rapi = binding.Rpa.for_meta(meta)
    rapi.rpa_set_tile_pair(1)
    return rapi


@pytest.mark.parametrize("case", [c for c in TILE_CASES if c[4] == 128])
def test_pair_kernel_on_the_tile_cases(case):
    # short items (the second CTA of the pair has no rows), decode rows forced onto the tile path,
    # ragged contexts, every group size
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("pair", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=13,
                         token_capacity=sum(ql) + 5)
    rapi = _pair_api(meta)
    _, info = hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi, tile_min_q=1)
    assert info["num_tile_items"] > 0 and info["num_row_items"] == 0
    rapi.close()


PAIR_CASES = [
    # q_lens, kv_lens, h_q, h_kv, page_size, causal
    ([128], [128], 32, 8, 16, True),                               # one full item: four full tiles, one key block
    ([300, 129, 1000, 64], [811, 129, 1000, 4000], 32, 8, 16, True),  # full and partial items; more items than pairs
    ([4096], [4096], 32, 8, 16, True),                             # 256 items on 74 pairs: every pair runs several
    ([500, 260], [900, 2000], 32, 4, 64, True),                    # h_g = 8, pages of half a key block
    ([700], [1500], 4, 4, 32, True),                               # h_g = 1: an item is 512 tokens
    ([300, 129], [811, 400], 32, 8, 16, False),                    # no causal mask
    ([260, 90], [1000, 700], 32, 8, 48, True),                     # page size that divides neither 64 nor 128
    ([4736], [4736], 8, 2, 16, True),                              # 74 items: one per pair, every SM busy
]


@pytest.mark.parametrize("case", PAIR_CASES)
def test_pair_kernel_cases(case):
    ql, kl, hq, hkv, ps, causal = case
    meta = wl.build_meta("pair", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=128, page_size=ps, seed=29,
                         token_capacity=sum(ql) + 3, causal=causal)
    rapi = _pair_api(meta)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), rapi=rapi)
    assert info["num_tile_items"] > 0
    # an item covers four query tiles
    assert info["num_tile_items"] == hkv * sum(-(-q // (4 * (128 // (hq // hkv)))) for q in ql)
    rapi.close()


def test_pair_kernel_beside_the_row_kernel_in_a_mixed_batch():
    rng = np.random.default_rng(5)
    ql = [1] * 40 + [700, 300]
    kl = [int(x) for x in rng.integers(200, 3000, size=40)] + [900, 2300]
    meta = wl.build_meta("pair_mixed", ql, kl, num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=31)
    rapi = _pair_api(meta)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), rapi=rapi)
    assert info["num_tile_items"] > 0 and info["num_row_items"] > 0 and info["batch_case_name"] == "mixed"
    rapi.close()


def test_pair_kernel_two_calls_on_one_handle_and_back_to_the_two_tile_kernel():
    meta = wl.build_meta("pair_twice", [600, 200], [600, 1200], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=33)
    rapi = _pair_api(meta)
    hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi)
    first = rapi.rpa_plan_info()["num_tile_items"]
    hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi)  # the counters the pairs draw from were reset
    rapi.rpa_set_tile_pair(0)
    hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi)
    assert rapi.rpa_plan_info()["num_tile_items"] == 2 * first  # items of two query tiles again
    rapi.close()


def test_pair_kernel_is_chosen_for_long_prefill_only():
    # default mode: the pair kernel (items of 4 query tiles = 128 tokens at h_g = 4) when every sequence of the
    # batch has at least 256 new tokens and there are at least two pair items per SM; a shorter sequence, a
    # decode row or a batch too small to keep the pairs busy stays on the two-tile kernel
    shape = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16)
    for ql, kl, kernel in (([4800], [4800], 3), ([4800, 40], [4800, 1300], 1), ([4800, 1], [4800, 900], 1), ([600, 300], [600, 1300], 1)):
        meta = wl.build_meta("pair_auto", ql, kl, seed=37, **shape)
        rapi = binding.Rpa.for_meta(meta)
        rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
        info = rapi.rpa_plan_info()
        assert info["tile_kernel"] == kernel
        per_item = 128 if kernel == 3 else 64
        assert info["num_tile_items"] == 8 * sum(-(-q // per_item) for q in ql if q > 8)
        rapi.close()
    meta = wl.build_meta("pair_auto", [4800], [4800], seed=38, **shape)
    rapi = binding.Rpa.for_meta(meta)
    _, info = hz.sampled_parity(wl.materialize(meta, _dev()), seqs=[0], rows_per_seq=160, whole_cache=True, rapi=rapi)
    assert info["tile_kernel"] == 3
    rapi.close()


def test_device_planned_steps_keep_the_two_tile_kernel():
    meta = wl.build_meta("pair_devplan", [300, 1, 64], [800, 500, 64], num_q_heads=32, num_kv_heads=8, head_dim=128,
                         page_size=16, seed=35)
    rapi = _pair_api(meta)
    hz.full_parity(wl.materialize(meta, _dev()), rapi=rapi, device_plan=True)
    rapi.close()


def test_pair_kernel_is_refused_where_it_has_no_instantiation():
    for kw in (dict(head_dim=64), dict(head_dim=256), dict(head_dim=128, kv_fp8=True, k_scale=0.03, v_scale=0.03)):
        meta = wl.build_meta("pair_no", [64], [64], num_q_heads=32, num_kv_heads=8, page_size=16, seed=36, **kw)
        rapi = binding.Rpa.for_meta(meta)
        with pytest.raises(binding.RpaError) as err:
            rapi.rpa_set_tile_pair(1)
        assert err.value.status == 2  # RPA_ERR_UNSUPPORTED
        rapi.close()


def test_pair_kernel_on_the_llama_prefill_workload_sampled_rows():
    batch = wl.materialize(wl.workload_meta(3), _dev())
    rapi = _pair_api(batch.meta)
    (mx, mean), info = hz.sampled_parity(batch, seqs=[1, 2], rows_per_seq=192, whole_cache=True, rapi=rapi)
    assert info["batch_case_name"] == "prefill" and info["num_tile_items"] == 4 * 8 * 64
    rapi.close()


def test_pair_kernel_in_the_bounds_checked_build():
    """Good input: same results, nothing reported.  An out-of-range page id (one that still lies inside the
    real allocation) in a context page and in a page that receives new tokens: named in the status word,
    the read redirected to page 0, the write dropped."""
    import dataclasses

    from paper_2604_15464_b200 import build
    debug_lib = build.build(debug=True)
    tight = wl.build_meta("pair_dbg", [300, 260], [900, 260], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=39,
                          pool_slack=1.0)
    rapi = binding.Rpa.for_meta(tight, library_path=debug_lib)
    rapi.rpa_set_tile_pair(1)
    _, info = hz.full_parity(wl.materialize(tight, _dev(), canaries=True), rapi=rapi)
    assert info["tile_kernel"] == 3 and rapi.rpa_poll_status() == 0
    meta = dataclasses.replace(tight, num_pages=tight.num_pages + 8)  # the tensor holds 8 pages more than the handle knows of
    batch = wl.materialize(meta, _dev())
    bad = tight.num_pages + 5
    tail_before = wl.bf16_bits(batch.kv_cache[tight.num_pages:]).copy()
    out = torch.zeros_like(batch.q)
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    for seq, page_slot in ((0, 3), (1, (260 - 1) // 16)):  # a context page; the page of the last new tokens
        table = batch.page_table.clone()
        table[seq, page_slot] = bad
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, table, batch.cu_q_lens, batch.kv_lens, out)
        torch.cuda.synchronize()
        word = rapi.rpa_poll_status()
        assert word & (1 << 27) and (word >> 24) & 7 == 1 and (word & 0xFFFFFF) == bad
        assert np.array_equal(tail_before, wl.bf16_bits(batch.kv_cache[tight.num_pages:]))  # nothing went through the bad id
    hz.full_parity(wl.materialize(tight, _dev()), rapi=rapi)  # the handle keeps working
    rapi.close()


@pytest.mark.parametrize("seed", range(6))
def test_pair_kernel_random_long_prefill_batches(seed):
    """Seeded random pure-prefill batches (ragged lengths from 256 tokens up, with and without cached context,
    several head groupings and page sizes): whole-batch parity on the pair kernel."""
    rng = np.random.default_rng(4000 + seed)
    hq, hkv = [(32, 8), (16, 2), (8, 8), (32, 4), (16, 16), (64, 8)][seed % 6]
    tq4 = 4 * (128 // (hq // hkv))
    n = int(rng.integers(1, 5))
    ql = [int(rng.integers(2 * tq4, 2 * tq4 + 900)) for _ in range(n)]
    kl = [q + (int(rng.integers(0, 1500)) if rng.integers(0, 2) else 0) for q in ql]
    meta = wl.build_meta(f"pair_rand{seed}", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=128,
                         page_size=int(rng.choice([16, 32, 48, 128, 256])), seed=800 + seed, token_capacity=sum(ql) + 2,
                         causal=bool(seed % 5 != 4))
    rapi = _pair_api(meta)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=bool(seed % 2)), rapi=rapi)
    assert info["tile_kernel"] == 3
    rapi.close()
