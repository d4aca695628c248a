"""GPU parity on an FP8 (E4M3) cache with per-tensor scales against the fp64 oracle, for the row path
and the tensor-core tile path (head_dim 128): outputs within the bf16 tolerance, cache bytes (the
quantised codes of the new rows) bit-exact."""
import numpy as np
import pytest
import torch

from paper_2604_15464_b200 import build
from paper_2604_15464_b200 import workloads as wl

import rpa_harness as hz

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _dev():
    return torch.device("cuda", 0)


FP8_CASES = [
    # q_lens, kv_lens, h_q, h_kv, d, page_size
    ([1, 1, 12, 5], [33, 7, 12, 29], 4, 2, 64, 16),               # the tiny mixed batch's shapes
    ([1, 1, 1], [1, 16, 17], 32, 8, 128, 16),
    ([3, 0, 1, 40, 17], [3, 0, 130, 40, 100], 32, 8, 128, 16),
    ([7, 1, 33], [64, 1, 33], 8, 8, 128, 32),                     # MHA
    ([5, 9, 1], [21, 9, 300], 8, 1, 128, 16),                     # MQA
    ([1] * 9, [5, 31, 32, 33, 47, 48, 49, 255, 257], 32, 8, 128, 128),
    ([1, 4, 20], [700, 64, 20], 32, 8, 256, 16),                  # d = 256
    ([2, 19], [50, 19], 16, 1, 64, 16),                           # h_g = 16
]


@pytest.mark.parametrize("case", FP8_CASES)
@pytest.mark.parametrize("chunk", [0, 32])
def test_fp8_cache_cases(case, chunk):
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("fp8", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=23,
                         token_capacity=sum(ql) + 3, kv_fp8=True, k_scale=0.023, v_scale=0.031)
    _, info = hz.full_parity(wl.materialize(meta, _dev()), kv_chunk=chunk)
    # head_dim 128 and 256 have tile kernels for FP8 caches; head_dim 64 stays on the row kernel
    assert (info["num_tile_items"] > 0) == (d in (128, 256) and max(ql) * (hq // hkv) > 32)


FP8_TILE_CASES = [
    # q_lens, kv_lens, h_q, h_kv, page_size: every sequence forced onto the tile path
    ([64], [64], 32, 8, 16),                       # one item, no context: only the quantising pass and new-token blocks
    ([40], [300], 32, 8, 16),                      # context ends mid-page and mid-block
    ([200, 1, 70], [200, 500, 1000], 32, 8, 16),   # several blocks of both streams; a decode row
    ([130, 64], [130, 257], 32, 8, 128),           # 128-token pages
    ([96, 7], [96, 135], 8, 8, 32),                # h_g = 1
    ([50, 20], [77, 20], 8, 1, 16),                # h_g = 8
    ([16, 32, 5], [1016, 2080, 133], 32, 8, 16),   # short items: key blocks dealt to both accumulators
    ([20], [4117], 32, 8, 128),
]


@pytest.mark.parametrize("case", FP8_TILE_CASES)
def test_fp8_tile_kernel_cases(case):
    ql, kl, hq, hkv, ps = case
    meta = wl.build_meta("fp8t", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=128, page_size=ps, seed=27,
                         token_capacity=sum(ql) + 5, kv_fp8=True, k_scale=0.023, v_scale=0.031)
    _, info = hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)
    assert info["num_tile_items"] > 0 and info["num_row_items"] == 0


FP8_TILE1_CASES = [
    # head_dim 256 on the single-tile kernel: q_lens, kv_lens, h_q, h_kv, page_size
    ([32], [32], 32, 8, 16),                       # one item, no context: the quantising pass and a new-token block
    ([40], [300], 32, 8, 16),                      # context ends mid-page and mid-block
    ([200, 1, 70], [200, 500, 1000], 32, 8, 16),   # several blocks of both streams; a decode row
    ([130, 64], [130, 257], 32, 8, 128),           # pages larger than a key block
    ([96, 7], [96, 135], 8, 8, 32),                # h_g = 1
    ([33, 300], [60, 700], 16, 1, 256),            # h_g = 16, page 256
    ([20], [4117], 32, 8, 64),                     # 64 context blocks behind a short chunk
]


@pytest.mark.parametrize("case", FP8_TILE1_CASES)
def test_fp8_single_tile_kernel_cases(case):
    ql, kl, hq, hkv, ps = case
    meta = wl.build_meta("fp8t1", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=256, page_size=ps, seed=37,
                         token_capacity=sum(ql) + 5, kv_fp8=True, k_scale=0.023, v_scale=0.031)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)
    assert info["num_tile_items"] > 0 and info["num_row_items"] == 0
    if len(ql) > 1:  # the same lengths planned on the device (fixed grids, strided quantising pass)
        hz.full_parity(wl.materialize(meta, _dev()), device_plan=True)


def test_fp8_single_tile_kernel_noncausal():
    meta = wl.build_meta("fp8t1n", [33, 100], [290, 100], num_q_heads=8, num_kv_heads=2, head_dim=256, page_size=16,
                         seed=38, causal=False, kv_fp8=True, k_scale=0.05, v_scale=0.04)
    hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)


def test_fp8_tile_kernel_canaries_noncausal_and_mixed():
    meta = wl.build_meta("fp8tc", [40, 1, 130], [300, 77, 130], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=28, kv_fp8=True, k_scale=0.05, v_scale=0.04)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True))
    assert info["num_tile_items"] > 0 and info["num_row_items"] > 0  # both kernels, side by side
    meta = wl.build_meta("fp8tn", [33, 100], [290, 100], num_q_heads=8, num_kv_heads=2, head_dim=128, page_size=16,
                         seed=29, causal=False, kv_fp8=True, k_scale=0.05, v_scale=0.04)
    hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)


def test_fp8_cache_nan_canaries_and_noncausal():
    meta = wl.build_meta("fp8c", [1, 12, 5], [33, 12, 29], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=24, kv_fp8=True, k_scale=0.05, v_scale=0.04)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True))
    meta = wl.build_meta("fp8n", [4, 1, 20], [36, 90, 20], num_q_heads=8, num_kv_heads=2, head_dim=128, page_size=16,
                         seed=25, causal=False, kv_fp8=True, k_scale=0.05, v_scale=0.04)
    hz.full_parity(wl.materialize(meta, _dev()))


def test_fp8_update_saturates_instead_of_overflowing():
    # a scale so small that most new values exceed 448 * scale: the stored codes must be +-448, never NaN
    meta = wl.build_meta("fp8sat", [3, 1], [10, 40], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=26, kv_fp8=True, k_scale=0.001, v_scale=0.002)
    batch = wl.materialize(meta, _dev())
    hz.full_parity(batch)
    codes = wl.bf16_bits(batch.kv_cache)
    assert not np.any((codes & 0x7F) == 0x7F)


def test_fp8_llama_decode_full_batch():
    meta = wl.workload_meta(2)
    meta.kv_fp8, meta.k_scale, meta.v_scale = True, 0.02, 0.02
    (mx, mean), info = hz.full_parity(wl.materialize(meta, _dev()))
    assert info["batch_case_name"] == "decode"


def test_fp8_tile_kernel_packs_short_sequences():
    for ql, ps, causal in [([10, 20, 30, 7, 9, 64, 3, 3], 16, True), ([16] * 9 + [1, 2, 3], 128, False)]:
        meta = wl.build_meta("fp8p", ql, ql, num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=ps, seed=30,
                             causal=causal, kv_fp8=True, k_scale=0.04, v_scale=0.03)
        rapi = hz.binding.Rpa.for_meta(meta)
        hz.full_parity(wl.materialize(meta, _dev(), canaries=True), rapi=rapi)
        assert any(t[4] & 2 for t in rapi.rpa_plan_dump()[1]), "the batch must contain packed items"


NARROW_CASES = [
    # q_lens, kv_lens, h_q, h_kv, d, page_size: no row item has more than 8 query rows, so the 8-row
    # instantiation of the FP8 row kernel (transposed second product) serves the whole list
    ([1] * 7, [1, 15, 16, 17, 100, 513, 2049], 32, 8, 128, 16),    # G = 4, one token
    ([2, 1, 2, 0, 2], [2, 40, 333, 0, 1030], 32, 8, 128, 16),      # G = 4, two tokens: all 8 rows live
    ([1, 1, 1], [300, 31, 1500], 8, 1, 128, 32),                   # G = 8
    ([1, 3, 8, 5], [77, 3, 800, 150], 8, 8, 64, 16),               # G = 1: up to 8 tokens per item, causal steps inside
    ([1, 4, 2], [420, 4, 1111], 16, 8, 256, 16),                   # G = 2, d = 256
    ([1, 1, 2], [65, 700, 130], 8, 2, 64, 128),                    # d = 64, large pages
]


@pytest.mark.parametrize("case", NARROW_CASES)
@pytest.mark.parametrize("chunk", [0, 64])
@pytest.mark.parametrize("device_plan", [False, True])
def test_fp8_narrow_row_items(case, chunk, device_plan):
    ql, kl, hq, hkv, d, ps = case
    g = hq // hkv
    assert max(min(q, 16 // g) for q in ql) * g <= 8
    meta = wl.build_meta("fp8n", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=41,
                         token_capacity=sum(ql) + 2, kv_fp8=True, k_scale=0.027, v_scale=0.019)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), kv_chunk=chunk, tile_min_q=10**6,
                             device_plan=device_plan)
    assert info is None or info["num_tile_items"] == 0  # (a device-planned step has no host-side summary)


def test_fp8_narrow_noncausal_and_wide_beside_it():
    # non-causal: every row sees every key, the tail of the last tile is masked by length only
    meta = wl.build_meta("fp8nn", [2, 1, 2], [45, 700, 2], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=42, causal=False, kv_fp8=True, k_scale=0.03, v_scale=0.03)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=10**6)
    # one sequence with three tokens (12 rows) turns the whole list over to the 16-row instantiation
    for device_plan in (False, True):
        meta = wl.build_meta("fp8nw", [1, 3, 1], [500, 90, 33], num_q_heads=32, num_kv_heads=8, head_dim=128,
                             page_size=16, seed=43, kv_fp8=True, k_scale=0.03, v_scale=0.03)
        hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=10**6, device_plan=device_plan)


# ---- per-tensor quantisation of Q as well (Section 3.8): the oracle takes Q in E4M3 precision ----

QFP8_CASES = [
    # q_lens, kv_lens, h_q, h_kv, d, page_size, tile_min_q
    ([1, 1, 12, 5], [33, 7, 12, 29], 4, 2, 64, 16, None),           # row kernel, d = 64
    ([1] * 9, [5, 31, 32, 33, 47, 48, 49, 255, 257], 32, 8, 128, 128, None),  # decode rows (8-row instantiation)
    ([3, 0, 1, 40, 17], [3, 0, 130, 40, 100], 32, 8, 128, 16, None),          # default routing: rows and tiles
    ([200, 1, 70], [200, 500, 1000], 32, 8, 128, 16, 1),             # everything on the tile kernel
    ([16, 32, 5], [1016, 2080, 133], 32, 8, 128, 16, 1),             # short items split over both accumulators
    ([1, 4, 40], [700, 64, 300], 32, 8, 256, 16, 1),                 # d = 256: the single-tile kernel
    ([5, 9, 1], [21, 9, 300], 8, 1, 128, 16, 10 ** 6),               # MQA on the 16-row instantiation
]


@pytest.mark.parametrize("case", QFP8_CASES)
@pytest.mark.parametrize("device_plan", [False, True])
def test_fp8_cache_with_quantised_q(case, device_plan):
    ql, kl, hq, hkv, d, ps, tile_min_q = case
    meta = wl.build_meta("fp8q", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=29,
                         token_capacity=sum(ql) + 3, kv_fp8=True, k_scale=0.023, v_scale=0.031, q_scale=0.027)
    if device_plan and tile_min_q is not None:
        pytest.skip("the routing threshold is a host-planner knob in this test")
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=tile_min_q, device_plan=device_plan)


def test_quantised_q_really_is_quantised():
    """The same batch with and without a scale for Q must differ (by what three mantissa bits allow):
    a pass that were skipped, or a scale that were not folded, would show here or in the parity above."""
    shape = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=30, kv_fp8=True, k_scale=0.023, v_scale=0.031)
    a = wl.build_meta("fp8q-a", [1, 40], [300, 200], **shape)
    b = wl.build_meta("fp8q-b", [1, 40], [300, 200], q_scale=0.027, **shape)
    out_a, _ = hz.run_gpu(wl.materialize(a, _dev()))
    out_b, _ = hz.run_gpu(wl.materialize(b, _dev()))
    diff = np.abs(hz.bf16_to_f64(out_a[: a.num_tokens]) - hz.bf16_to_f64(out_b[: b.num_tokens]))
    assert 1e-4 < diff.max() < 0.5


def test_q_scale_needs_an_fp8_cache():
    from paper_2604_15464_b200 import binding

    meta = wl.build_meta("q-bf16", [1], [40], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=31)
    meta.q_scale = 0.05
    with pytest.raises(binding.RpaError) as err:
        binding.Rpa.for_meta(meta)
    assert err.value.status == 1  # RPA_ERR_INVALID_ARG
