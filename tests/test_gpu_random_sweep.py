"""Seeded random sweep: many small ragged batches with random shapes, lengths, page sizes, routing
thresholds, split chunks, cache types and planners (host or device), each compared in full with the
fp64 oracle (outputs, every cache byte, untouched rows).  Meant to catch index arithmetic that only
breaks on unlucky boundaries."""
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


def _random_case(rng, n_max=7, kinds=4):
    d = int(rng.choice([64, 128, 128, 128, 256]))
    h_kv = int(rng.choice([1, 2, 8]))
    h_g = int(rng.choice([1, 2, 4, 4, 8, 16]))
    ps = int(rng.choice([16, 16, 32, 64, 128, 256]))
    n = int(rng.integers(1, n_max))
    q_lens, kv_lens = [], []
    for _ in range(n):
        kind = rng.integers(0, kinds)
        if kind >= 4:  # short prompt without context: neighbours of this kind share a tile item
            q = int(rng.integers(1, 40))
            q_lens.append(q)
            kv_lens.append(q)
            continue
        if kind == 0:  # decode
            q = 1
            ctx = int(rng.integers(0, 700))
        elif kind == 1:  # short chunk / speculative rows
            q = int(rng.integers(2, 20))
            ctx = int(rng.integers(0, 300))
        elif kind == 2:  # prefill chunk
            q = int(rng.integers(20, 200))
            ctx = int(rng.integers(0, 400))
        else:  # empty or boundary-aligned
            q = int(rng.choice([0, 16, 64, 128]))
            ctx = int(rng.choice([0, ps, 128, 2 * ps - 1]))
        q_lens.append(q)
        kv_lens.append(q + ctx if q > 0 else int(rng.integers(0, 50)))
    return dict(q_lens=q_lens, kv_lens=kv_lens, num_q_heads=h_kv * h_g, num_kv_heads=h_kv, head_dim=d, page_size=ps,
                causal=bool(rng.integers(0, 5) > 0))


@pytest.mark.parametrize("seed", range(24))
def test_random_batches(seed):
    rng = np.random.default_rng(9000 + seed)
    case = _random_case(rng)
    fp8 = bool(rng.integers(0, 4) == 0)
    q_lens, kv_lens = case.pop("q_lens"), case.pop("kv_lens")
    meta = wl.build_meta(f"rand{seed}", q_lens, kv_lens, seed=100 + seed, token_capacity=sum(q_lens) + int(rng.integers(0, 5)),
                         kv_fp8=fp8, k_scale=0.03 if fp8 else 1.0, v_scale=0.025 if fp8 else 1.0, **case)
    kv_chunk = int(rng.choice([0, 0, 16, 48, 128]))
    if sum(q_lens) * case["num_kv_heads"] > 600:
        kv_chunk = 0  # a forced tiny chunk on many rows would exceed the handle's split-KV workspace
    tile_min_q = rng.choice([None, None, 1, 8, 10 ** 6])
    tile_min_q = None if tile_min_q is None else int(tile_min_q)
    batch = wl.materialize(meta, torch.device("cuda", 0), canaries=bool(rng.integers(0, 3) == 0))
    hz.full_parity(batch, kv_chunk=kv_chunk, tile_min_q=tile_min_q)


@pytest.mark.parametrize("seed", range(16))
def test_random_batches_with_short_prompts_and_device_planning(seed):
    """More sequences per batch, many of them short prompts without context (packed into shared
    tile items by the host planner), a long-context small-q request now and then (key blocks dealt to
    both accumulators), FP8 caches on the tile path, and every other batch planned on the device."""
    rng = np.random.default_rng(7000 + seed)
    case = _random_case(rng, n_max=14, kinds=7)
    q_lens, kv_lens = case.pop("q_lens"), case.pop("kv_lens")
    if rng.integers(0, 2):  # a small-q request on a long context
        q = int(rng.integers(2, 33))
        q_lens.append(q)
        kv_lens.append(q + int(rng.integers(1000, 5000)))
    fp8 = bool(rng.integers(0, 3) == 0)
    device_plan = bool(seed % 2)
    meta = wl.build_meta(f"randp{seed}", q_lens, kv_lens, seed=300 + seed, token_capacity=sum(q_lens) + int(rng.integers(0, 5)),
                         kv_fp8=fp8, k_scale=0.03 if fp8 else 1.0, v_scale=0.025 if fp8 else 1.0, **case)
    batch = wl.materialize(meta, torch.device("cuda", 0), canaries=bool(rng.integers(0, 3) == 0))
    hz.full_parity(batch, device_plan=device_plan)


@pytest.mark.parametrize("seed", range(12))
def test_random_batches_on_unaligned_page_sizes(seed):
    """The same draw on page sizes that are multiples of 16 but neither divide nor are a multiple of
    a key block of the tile kernels (64 or 128 positions)."""
    rng = np.random.default_rng(5000 + seed)
    case = _random_case(rng, n_max=9, kinds=5)
    case["page_size"] = int(rng.choice([48, 80, 96, 112, 144, 176, 192, 240]))
    q_lens, kv_lens = case.pop("q_lens"), case.pop("kv_lens")
    fp8 = bool(rng.integers(0, 3) == 0)
    meta = wl.build_meta(f"randu{seed}", q_lens, kv_lens, seed=500 + seed, token_capacity=sum(q_lens) + 3,
                         kv_fp8=fp8, k_scale=0.03 if fp8 else 1.0, v_scale=0.025 if fp8 else 1.0, **case)
    tile_min_q = [None, 1, 8][seed % 3]
    batch = wl.materialize(meta, torch.device("cuda", 0), canaries=bool(seed % 2))
    hz.full_parity(batch, tile_min_q=tile_min_q, device_plan=(tile_min_q is None and seed % 4 == 0))


@pytest.mark.parametrize("seed", range(10))
def test_random_batches_with_quantised_q_and_the_bounds_checked_build(seed):
    """FP8 caches with a scale for Q as well (FP8 score products on the d_k = 128 tile path), host- and
    device-planned, every other batch through the bounds-checked build of the library, which must
    report nothing on good input."""
    from paper_2604_15464_b200 import binding

    rng = np.random.default_rng(3000 + seed)
    case = _random_case(rng, n_max=10, kinds=6)
    q_lens, kv_lens = case.pop("q_lens"), case.pop("kv_lens")
    if rng.integers(0, 2):
        q = int(rng.integers(2, 200))
        q_lens.append(q)
        kv_lens.append(q + int(rng.integers(500, 3000)))
    meta = wl.build_meta(f"randq{seed}", q_lens, kv_lens, seed=700 + seed, token_capacity=sum(q_lens) + 2, kv_fp8=True,
                         k_scale=0.03, v_scale=0.025, q_scale=float(rng.choice([0.02, 0.03125, 0.05])), **case)
    lib = build.build(debug=True) if seed % 2 else None
    rapi = binding.Rpa.for_meta(meta, library_path=lib)
    batch = wl.materialize(meta, torch.device("cuda", 0), canaries=bool(seed % 3 == 0))
    hz.full_parity(batch, rapi=rapi, device_plan=bool(seed % 4 == 1))
    assert rapi.rpa_poll_status() == 0
    rapi.close()
