"""Shared plumbing of the GPU parity tests: run the CUDA path through the C-ABI binding, run the
fp64 oracle on a host copy of the same bits, and compare.  Holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np
import torch

from oracle import rpa_oracle as orc
from paper_2604_15464_b200 import binding
from paper_2604_15464_b200 import workloads as wl

# tolerance of the bf16 outputs against the fp64 oracle
MAX_ABS = 1.5e-2
MEAN_ABS = 2e-3
SENTINEL = 0x7FC1  # a NaN pattern no computation produces; marks rows the call must not touch


def oracle_shape(meta, num_pages=None):
    return orc.OracleShape(meta.num_q_heads, meta.num_kv_heads, meta.head_dim, meta.page_size,
                           meta.num_pages if num_pages is None else num_pages, meta.max_pages_per_seq, meta.sm_scale,
                           meta.causal, meta.kv_fp8, meta.k_scale, meta.v_scale, meta.q_scale)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def run_gpu(batch, *, kv_chunk=0, rapi=None, tile_min_q=None, device_plan=False):
    """plan + forward through the binding; returns (out bits [cap, h_q, d], cache bits after the call).
    device_plan: the lists are built by the device-side planner from the device copies of the lengths."""
    meta = batch.meta
    own = rapi is None
    if own:
        rapi = binding.Rpa.for_meta(meta, device=batch.q.device.index or 0)
    if kv_chunk:
        rapi.rpa_set_kv_chunk(kv_chunk)
    if tile_min_q is not None:
        rapi.rpa_set_tile_min_q(tile_min_q)
    out = torch.full(batch.q.shape, SENTINEL, dtype=torch.int16, device=batch.q.device).view(torch.bfloat16)
    if device_plan:
        rapi.rpa_plan_device(batch.cu_q_lens, batch.kv_lens)
        rapi.rpa_forward(batch.q, batch.new_k, batch.new_v, batch.kv_cache, batch.page_table, batch.cu_q_lens,
                         batch.kv_lens, out)
    else:
        rapi.run_batch(batch, out)
    torch.cuda.synchronize()
    status = rapi.rpa_poll_status()
    info = None if device_plan else rapi.rpa_plan_info()
    if own:
        rapi.close()
    assert status == 0, f"device status word {status:#x}"
    return wl.bf16_bits(out), info


def compare_outputs(got_bits: np.ndarray, ref: np.ndarray, what=""):
    got = bf16_to_f64(got_bits)
    if got.size == 0:
        return 0.0, 0.0
    assert np.all(np.isfinite(got)), f"{what}: non-finite outputs"
    err = np.abs(got - ref)
    big = int((np.abs(ref) >= 4.0).sum())  # bf16 half-ulp there is 1.56e-2, above the max-abs bar
    assert err.max() <= MAX_ABS, f"{what}: max-abs {err.max():.4g} > {MAX_ABS} ({big} reference values with |x|>=4)"
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.4g} > {MEAN_ABS}"
    return float(err.max()), float(err.mean())


def full_parity(batch, *, kv_chunk=0, rapi=None, tile_min_q=None, device_plan=False):
    """Whole-batch comparison: every output row, every cache byte, untouched rows."""
    meta = batch.meta
    host = dict(q=wl.bf16_bits(batch.q), new_k=wl.bf16_bits(batch.new_k), new_v=wl.bf16_bits(batch.new_v),
                kv_cache=wl.bf16_bits(batch.kv_cache).copy(), page_table=meta.page_table, cu_q_lens=meta.cu_q_lens,
                kv_lens=meta.kv_lens)
    ref = orc.forward(oracle_shape(meta), **host)
    got, info = run_gpu(batch, kv_chunk=kv_chunk, rapi=rapi, tile_min_q=tile_min_q, device_plan=device_plan)
    T = meta.num_tokens
    stats = compare_outputs(got[:T], ref, meta.name)
    assert np.all(got[T:] == SENTINEL), "rows past the last token were written"
    cache_after = wl.bf16_bits(batch.kv_cache)
    assert np.array_equal(cache_after, host["kv_cache"]), "cache differs from the oracle's (must be bit-exact)"
    return stats, info


def host_subset(batch, seqs):
    """Compact host copy of the sampled requests plus the oracle shape that goes with it."""
    host, n_pages, rows, pages = wl.host_subset(batch, seqs)
    return host, oracle_shape(batch.meta, num_pages=n_pages), rows, pages


def sampled_parity(batch, seqs, rows_per_seq=None, *, rng=None, rapi=None, kv_chunk=0, tile_min_q=None,
                   whole_cache=False):
    """Run the full batch on the GPU, check the sampled sequences' outputs and cache pages against
    the oracle (all their rows, or ``rows_per_seq`` random (token, head) pairs each).  With
    ``whole_cache`` every byte of the pool is compared as well: the oracle's update step (a bit copy
    per new token) is applied to a host copy of the whole cache taken before the call, so slots the
    call must leave alone are covered too."""
    meta = batch.meta
    rng = rng or np.random.default_rng(0)
    host, shape, rows, pages = host_subset(batch, seqs)  # snapshot BEFORE the call
    whole = None
    if whole_cache:
        whole = wl.bf16_bits(batch.kv_cache).copy()
        orc.update_cache(oracle_shape(meta), wl.bf16_bits(batch.new_k), wl.bf16_bits(batch.new_v), whole, meta.page_table,
                         meta.cu_q_lens, meta.kv_lens)
    got, info = run_gpu(batch, kv_chunk=kv_chunk, rapi=rapi, tile_min_q=tile_min_q)
    if whole is not None:
        assert np.array_equal(wl.bf16_bits(batch.kv_cache), whole), "the pool differs from the oracle's somewhere"
    orc.update_cache(shape, host["new_k"], host["new_v"], host["kv_cache"], host["page_table"], host["cu_q_lens"],
                     host["kv_lens"])
    idx = torch.tensor(pages, dtype=torch.long, device=batch.kv_cache.device)
    assert np.array_equal(wl.bf16_bits(batch.kv_cache[idx]), host["kv_cache"]), "sampled cache pages differ"
    triples = []
    for k, r in enumerate(seqs):
        ql = int(meta.q_lens[r])
        if rows_per_seq is None or ql * meta.num_q_heads <= rows_per_seq:
            triples += [(k, i, a) for i in range(ql) for a in range(meta.num_q_heads)]
        else:
            toks = rng.integers(0, ql, size=rows_per_seq)
            toks[0], toks[-1] = 0, ql - 1
            heads = rng.integers(0, meta.num_q_heads, size=rows_per_seq)
            triples += [(k, int(i), int(a)) for i, a in zip(toks, heads)]
    ref = orc.attend_rows(shape, host["q"], host["kv_cache"], host["page_table"], host["cu_q_lens"], host["kv_lens"],
                          triples)
    cu = meta.cu_q_lens
    sel = np.stack([got[cu[seqs[k]] + i, a] for k, i, a in triples])
    stats = compare_outputs(sel, ref, meta.name)
    T = meta.num_tokens
    assert np.all(got[T:] == SENTINEL), "rows past the last token were written"
    return stats, info
