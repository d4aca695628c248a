"""The bounds-checked build of the library (-DRPA_DEBUG, ``librpa_b200_debug.so``): every page id, token
row and ring stage is checked before the access; the first violation is recorded in the device status
word (bit 27, kind in bits 24..26, the offending value below) and the access is skipped.  It stands in
for a memory checker.  Bad values used here always stay inside the real allocations, so that no
outcome of a check can fault the device."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2604_15464_b200 import binding, build
from paper_2604_15464_b200 import workloads as wl

import rpa_harness as hz

pytestmark = pytest.mark.gpu

DEBUG_BIT, KIND_PAGE, KIND_ROW = 1 << 27, 1, 2


@pytest.fixture(scope="module")
def debug_lib():
    build.build()
    return build.build(debug=True)


def _dev():
    return torch.device("cuda", 0)


@pytest.mark.parametrize("kv_fp8", [False, True])
@pytest.mark.parametrize("tile_min_q", [None, 1, 10 ** 6])
def test_debug_build_gives_the_same_results_and_reports_nothing_on_good_input(debug_lib, kv_fp8, tile_min_q):
    extra = dict(kv_fp8=True, k_scale=0.03, v_scale=0.025) if kv_fp8 else {}
    meta = wl.build_meta("dbg-ok", [1, 70, 5, 1, 130], [700, 330, 29, 33, 130], seed=61, page_size=16, **wl.LLAMA3_8B, **extra)
    rapi = binding.Rpa.for_meta(meta, library_path=debug_lib)
    hz.full_parity(wl.materialize(meta, _dev(), canaries=True), rapi=rapi, tile_min_q=tile_min_q, kv_chunk=64)
    assert rapi.rpa_poll_status() == 0
    rapi.close()


@pytest.mark.parametrize("tile_min_q", [1, 10 ** 6])  # the tensor-core tile path, the row path
def test_debug_build_names_the_first_bad_page_id_and_skips_the_access(debug_lib, tile_min_q):
    tight = wl.build_meta("dbg-page", [1, 40, 3], [500, 390, 64], seed=62, page_size=16, pool_slack=1.0, **wl.LLAMA3_8B)
    # the tensor holds 8 pages more than the handle is told about: an id in that tail is out of range for
    # the library while every address it could form stays inside the allocation
    meta = dataclasses.replace(tight, num_pages=tight.num_pages + 8)
    batch = wl.materialize(meta, _dev())
    rapi = binding.Rpa.for_meta(tight, library_path=debug_lib)
    rapi.rpa_set_tile_min_q(tile_min_q)
    bad = tight.num_pages + 5
    table = batch.page_table.clone()
    table[1, 3] = bad  # a context page of the chunked-prefill request
    tail_before = wl.bf16_bits(batch.kv_cache[tight.num_pages:]).copy()
    out = torch.zeros_like(batch.q)
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, table, batch.cu_q_lens, batch.kv_lens, out)
    torch.cuda.synchronize()
    word = rapi.rpa_poll_status()
    assert word & DEBUG_BIT and (word >> 24) & 7 == KIND_PAGE and (word & 0xFFFFFF) == bad
    assert np.array_equal(tail_before, wl.bf16_bits(batch.kv_cache[tight.num_pages:]))  # nothing went through the bad id
    assert rapi.rpa_poll_status() == 0  # reported once
    # a bad id on the page that receives the new tokens: the update is dropped, not redirected
    table = batch.page_table.clone()
    last_page = (int(meta.kv_lens[2]) - 1) // 16
    table[2, last_page] = bad
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, table, batch.cu_q_lens, batch.kv_lens, out)
    torch.cuda.synchronize()
    word = rapi.rpa_poll_status()
    assert word & DEBUG_BIT and (word >> 24) & 7 == KIND_PAGE and (word & 0xFFFFFF) == bad
    assert np.array_equal(tail_before, wl.bf16_bits(batch.kv_cache[tight.num_pages:]))
    # the handle keeps working
    hz.full_parity(wl.materialize(tight, _dev()), rapi=rapi, tile_min_q=tile_min_q)
    rapi.close()


@pytest.mark.parametrize("tile_min_q", [1, 10 ** 6])
def test_debug_build_catches_token_rows_beyond_the_declared_capacity(debug_lib, tile_min_q):
    # the handle is told the tensors hold T rows; they really hold 2T, and the device copy of cu_q_lens
    # is shifted so that the last sequence's rows end beyond T (but inside the allocation)
    meta = wl.build_meta("dbg-rows", [33, 40], [200, 300], seed=63, page_size=16, **wl.LLAMA3_8B)
    T = meta.num_tokens
    big = dataclasses.replace(meta, token_capacity=2 * T)
    batch = wl.materialize(big, _dev())
    rapi = binding.Rpa.for_meta(meta, library_path=debug_lib)  # max_num_tokens = T
    rapi.rpa_set_tile_min_q(tile_min_q)
    shifted = batch.cu_q_lens + 20
    out = torch.full(batch.q.shape, hz.SENTINEL, dtype=torch.int16, device=_dev()).view(torch.bfloat16)
    rapi.rpa_plan(meta.cu_q_lens, meta.kv_lens)
    rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, shifted, batch.kv_lens, out)
    torch.cuda.synchronize()
    word = rapi.rpa_poll_status()
    assert word & DEBUG_BIT and (word >> 24) & 7 == KIND_ROW and (word & 0xFFFFFF) > T
    assert np.all(wl.bf16_bits(out)[T:] == hz.SENTINEL)  # no row past the declared capacity was written
    rapi.close()
