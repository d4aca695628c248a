"""GPU parity of the tensor-core (tcgen05) tile kernel against the fp64 oracle: every sequence is
forced onto the tile path (tile_min_q = 1), over shapes that span several key blocks, ragged
context ends inside a page and inside a block, partial query tiles and both head dimensions."""
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


TILE_CASES = [
    # q_lens, kv_lens, h_q, h_kv, d, page_size
    ([64], [64], 32, 8, 128, 16),                      # exactly one item, one key block, no context
    ([128], [128], 32, 8, 128, 128),                   # two items, page = block
    ([40], [300], 32, 8, 128, 16),                     # context ends mid-page and mid-block
    ([200, 1, 70], [200, 500, 1000], 32, 8, 128, 16),  # several blocks of both streams; a decode row
    ([130, 64], [130, 257], 32, 8, 128, 128),          # context of 193 with 128-token pages
    ([96, 7], [96, 135], 8, 8, 128, 32),               # h_g = 1: 128 tokens per tile
    ([50, 20], [77, 20], 8, 1, 128, 16),               # h_g = 8
    ([33], [60], 16, 1, 64, 16),                       # h_g = 16, d = 64
    ([12, 5, 1, 1], [12, 29, 33, 7], 4, 2, 64, 16),    # the tiny mixed batch's shapes
    ([300], [700], 4, 2, 64, 64),                      # d = 64, several blocks
    # short items with several key blocks: the blocks are dealt to both accumulators and merged
    ([16, 32, 5], [1016, 2080, 133], 32, 8, 128, 16),  # odd and even block counts, ragged context
    ([20, 1], [4117, 300], 32, 8, 128, 128),           # 33 blocks; a decode row forced onto the tile path
    ([24], [280], 16, 1, 64, 16),                      # h_g = 16: one token per 16 rows, 3 blocks
    ([100], [1500], 8, 8, 128, 16),                    # h_g = 1: a 100-token item is still one tile
]


@pytest.mark.parametrize("case", TILE_CASES)
def test_tile_kernel_cases(case):
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("tile", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=13,
                         token_capacity=sum(ql) + 5)
    _, info = hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)
    assert info["num_tile_items"] > 0 and info["num_row_items"] == 0


TILE1_CASES = [
    # d_k = 256: the single-tile kernel with double-buffered scores (64-position key blocks)
    ([32], [32], 32, 8, 256, 16),                       # one item, one block, no context
    ([40], [300], 32, 8, 256, 16),                      # context ends mid-page and mid-block
    ([200, 1, 70], [200, 500, 1000], 32, 8, 256, 16),   # several blocks of both streams; a decode row
    ([130, 64], [130, 257], 32, 8, 256, 128),           # pages larger than a key block
    ([96, 7], [96, 135], 8, 8, 256, 32),                # h_g = 1
    ([33, 300], [60, 700], 16, 1, 256, 256),            # h_g = 16, page 256
]


@pytest.mark.parametrize("case", TILE1_CASES)
def test_single_tile_kernel_cases(case):
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("tile1", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=19,
                         token_capacity=sum(ql) + 5)
    _, info = hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)
    assert info["num_tile_items"] > 0 and info["num_row_items"] == 0


def test_single_tile_kernel_canaries_noncausal_and_routing():
    meta = wl.build_meta("t1c", [40, 64], [300, 100], num_q_heads=32, num_kv_heads=8, head_dim=256, page_size=16, seed=20)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)
    meta = wl.build_meta("t1n", [70, 40], [200, 40], num_q_heads=32, num_kv_heads=8, head_dim=256, page_size=16, seed=21,
                         causal=False)
    hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)
    meta = wl.build_meta("t1m", [1, 100, 1, 3], [900, 400, 50, 64], num_q_heads=32, num_kv_heads=8, head_dim=256,
                         page_size=16, seed=22)
    _, info = hz.full_parity(wl.materialize(meta, _dev()))
    assert info["num_tile_items"] > 0 and info["num_row_items"] > 0


def test_tile_kernel_nan_canaries():
    meta = wl.build_meta("tile_canary", [40, 64], [300, 100], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=14)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)


PACKED_CASES = [
    # q_lens (= kv_lens: no context), h_q, h_kv, d, page_size
    ([10, 20, 30], 32, 8, 128, 16),                       # 60 of 64 tokens: two tiles, sequences cut by the tile edge
    ([16] * 12, 32, 8, 128, 16),                          # three full items of four sequences
    ([1, 1, 1, 2, 3, 5, 8, 13, 21], 32, 8, 128, 16),      # one-token sequences; 55 tokens
    ([7, 9, 64, 3, 3, 100, 30, 30], 32, 8, 128, 128),     # runs interrupted by sequences too long to pack
    ([40, 50, 60, 100], 8, 8, 128, 32),                   # h_g = 1: items of 256 tokens
    ([2, 3, 2, 1], 8, 1, 128, 16),                        # h_g = 8: 16 tokens per item
    ([5, 6, 7, 8, 9], 4, 2, 64, 16),                      # d = 64
]


@pytest.mark.parametrize("case", PACKED_CASES)
@pytest.mark.parametrize("causal", [True, False])
def test_tile_kernel_packs_short_sequences(case, causal):
    ql, hq, hkv, d, ps = case
    meta = wl.build_meta("packed", ql, ql, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=19,
                         token_capacity=sum(ql) + 5, causal=causal)
    batch = wl.materialize(meta, _dev(), canaries=True)
    rapi = hz.binding.Rpa.for_meta(meta)
    _, info = hz.full_parity(batch, rapi=rapi)
    _, tiles, _ = rapi.rpa_plan_dump()
    assert any(t[4] & 2 for t in tiles), "the batch must contain packed items"


def test_packed_items_beside_context_and_decode_sequences():
    ql = [12, 20, 1, 8, 6, 6, 40, 1, 30, 30]
    kl = [12, 20, 700, 90, 6, 6, 300, 1, 30, 30]
    meta = wl.build_meta("packed-mixed", ql, kl, num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=20)
    _, info = hz.full_parity(wl.materialize(meta, _dev()))
    assert info["num_tile_items"] > 0 and info["num_row_items"] > 0


HALF_BLOCK_CASES = [
    # prompts without context whose only key block is at most half full (the softmax function of its own),
    # many more items than CTAs: every CTA runs several, so the first key block of the next item, its query
    # tiles and the output tiles of the one before are all in flight across item boundaries
    # q_lens, h_q, h_kv, d, page_size, causal
    ([64] * 40 + [33, 1, 64, 17] * 30, 32, 8, 128, 16, True),     # full and ragged tiles, one token, partial second tile
    ([48, 64, 20] * 70, 32, 8, 128, 48, False),                     # no causal mask; pages that do not divide a block
    ([64, 9, 64, 64, 31] * 20, 16, 16, 128, 16, True),              # h_g = 1: a 64-token prompt is half a query tile
    ([64, 40] * 90, 16, 2, 64, 32, True),                           # d = 64, h_g = 8
    # ... and beside items with a full block or several blocks (both softmax paths in one CTA's stream)
    ([128, 64, 200, 30] * 40, 32, 8, 128, 16, True),
]


@pytest.mark.parametrize("case", HALF_BLOCK_CASES)
def test_tile_kernel_items_of_a_single_half_full_block(case):
    ql, hq, hkv, d, ps, causal = case
    meta = wl.build_meta("half", ql, ql, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=23,
                         token_capacity=sum(ql) + 3, causal=causal)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)
    assert info["num_tile_items"] > 148 and info["num_row_items"] == 0 and info["tile_kernel"] == 1
    assert info["tile_short_items"] == (2 if max(ql) <= 64 else 1 if max(ql) <= 256 else 0)


@pytest.mark.parametrize("ql", [[64] * 3000, [128, 64, 300] * 400, [2048] * 6 + [40] * 500])
def test_tile_kernel_repeated_launches_agree_bit_for_bit(ql):
    """Persistent CTAs with many items each (loads, stores and barriers that live across item boundaries):
    twelve launches of one plan must give the same bits every time, with nothing in the status word; the first
    launch is checked against the oracle on sampled rows."""
    meta = wl.build_meta("repeat", ql, ql, num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16, seed=27)
    batch = wl.materialize(meta, _dev())
    rapi = hz.binding.Rpa.for_meta(meta)
    rapi.rpa_set_tile_pair(0)
    _, info = hz.sampled_parity(batch, seqs=[0, len(ql) // 2, len(ql) - 1], rows_per_seq=48, whole_cache=True, rapi=rapi)
    assert info["tile_kernel"] == 1 and info["num_tile_items"] > 4 * 148
    first = None
    for _ in range(12):
        out = torch.zeros_like(batch.q)
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens, batch.kv_lens, out)
        torch.cuda.synchronize()
        assert rapi.rpa_poll_status() == 0
        bits = wl.bf16_bits(out)
        if first is None:
            first = bits
        else:
            assert np.array_equal(first, bits)
    rapi.close()


def test_tile_kernel_split_items_noncausal():
    meta = wl.build_meta("split-nc", [16, 30], [700, 129], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=17, causal=False)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)


def test_tile_kernel_noncausal():
    meta = wl.build_meta("tile_nc", [70, 40], [200, 40], num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=16,
                         seed=15, causal=False)
    hz.full_parity(wl.materialize(meta, _dev()), tile_min_q=1)


def test_mixed_routing_uses_both_kernels():
    meta = wl.build_meta("both", [1, 100, 1, 3], [900, 400, 50, 64], num_q_heads=32, num_kv_heads=8, head_dim=128,
                         page_size=16, seed=16)
    _, info = hz.full_parity(wl.materialize(meta, _dev()))
    assert info["num_tile_items"] > 0 and info["num_row_items"] > 0


# Page sizes that neither divide a key block nor are a multiple of one (48, 80, 96, 112, 144, 192):
# a key block then spans pages at offsets that are not block-aligned, and the per-page boxes of the
# context gather must follow the page boundaries, not the block's.
@pytest.mark.parametrize("ps", [48, 80, 96, 112, 144, 192])
@pytest.mark.parametrize("d,fp8", [(128, False), (128, True), (256, False), (256, True), (64, False)])
def test_tile_kernels_on_page_sizes_that_do_not_align_with_key_blocks(ps, d, fp8):
    extra = dict(kv_fp8=True, k_scale=0.03, v_scale=0.025) if fp8 else {}
    h_q, h_kv = (32, 8) if d != 64 else (8, 2)
    meta = wl.build_meta(f"ps{ps}", [70, 16, 40, 1], [70 + 5 * ps + 7, 16 + 1000, 40 + ps, 2 * ps + 1], num_q_heads=h_q,
                         num_kv_heads=h_kv, head_dim=d, page_size=ps, seed=23 + ps, **extra)
    _, info = hz.full_parity(wl.materialize(meta, _dev(), canaries=True), tile_min_q=1)
    assert info["num_tile_items"] > 0
    # and with the default routing (row kernel for the decode row)
    hz.full_parity(wl.materialize(meta, _dev()))
