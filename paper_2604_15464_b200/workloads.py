"""Seeded synthetic batches for ragged paged attention.

This module only *generates inputs*: request lengths, page tables and random tensor values.  It
holds none of the method's arithmetic, so both the CUDA path and the CPU checker can be fed from it
without sharing any computation.

The five named workloads follow the paper's evaluation family (Section 4: Llama-3-8B head shapes,
bf16, synthetic batches) with raggedness added:

  1  tiny mixed batch (4 requests, 4/2 heads, d=64, page 16, 32-page pool)
  2  pure decode, 256 requests, kv_len ~ U{512..4096}, page 16
  3  full causal prefill, 4 requests of 8192 tokens, page 128
  4  mixed: 192 decode requests (kv_len ~ U{256..8192}) + 8 chunks of 512 new tokens on a prior
     context ~ U{0..4096}, page 16, token capacity 8192
  "4b"  the same with chunks of 1000 tokens: 192 + 8000 = 8192 new tokens, exactly the capacity, and
     chunk lengths that are no multiple of a query tile
  5  skewed decode: 512 requests, log-normal kv_len (median 2048, sigma 1.5, cap 131072), page 128,
     pages scattered over a pool sized by the caller
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np
import torch


@dataclass
class BatchMeta:
    """Host-side description of one batch (no tensor values)."""

    name: str
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    q_lens: np.ndarray  # int32 [n]
    kv_lens: np.ndarray  # int32 [n], cached + new tokens
    page_table: np.ndarray  # int32 [n, max_pages_per_seq]
    token_capacity: int  # rows allocated for q / new_k / new_v / out (>= sum(q_lens))
    causal: bool = True
    scale: float = 0.0  # 0 -> 1/sqrt(head_dim)
    seed: int = 0
    kv_fp8: bool = False  # FP8 E4M3 cache with per-tensor scales (the paper's Section 3.8)
    k_scale: float = 1.0
    v_scale: float = 1.0
    q_scale: float = 0.0  # > 0: Q is quantised to E4M3 with this per-tensor scale as well (FP8 cache only)

    @property
    def num_seqs(self) -> int:
        return int(len(self.q_lens))

    @property
    def cu_q_lens(self) -> np.ndarray:
        cu = np.zeros(self.num_seqs + 1, dtype=np.int32)
        np.cumsum(self.q_lens, out=cu[1:])
        return cu

    @property
    def num_tokens(self) -> int:
        return int(self.q_lens.sum())

    @property
    def sm_scale(self) -> float:
        return self.scale if self.scale > 0 else 1.0 / math.sqrt(self.head_dim)

    def mapped_pages(self) -> np.ndarray:
        """Physical ids of every page some request maps (positions < kv_len)."""
        ids = []
        for r in range(self.num_seqs):
            n = -(-int(self.kv_lens[r]) // self.page_size)
            ids.append(self.page_table[r, :n])
        return np.concatenate(ids) if ids else np.zeros(0, dtype=np.int32)


@dataclass
class Batch:
    """A batch with tensor values on ``device`` (bf16) and metadata on the host and the device."""

    meta: BatchMeta
    q: torch.Tensor  # [token_capacity, h_q, d]
    new_k: torch.Tensor  # [token_capacity, h_kv, d]
    new_v: torch.Tensor
    kv_cache: torch.Tensor  # [num_pages, page_size, 2*h_kv, d]
    page_table: torch.Tensor  # int32 [n, max_pages_per_seq]
    cu_q_lens: torch.Tensor  # int32 [n+1]
    kv_lens: torch.Tensor  # int32 [n]
    extras: dict = field(default_factory=dict)


def build_meta(name: str, q_lens: Sequence[int], kv_lens: Sequence[int], *, num_q_heads: int, num_kv_heads: int,
               head_dim: int, page_size: int, num_pages: Optional[int] = None, pool_slack: float = 1.25,
               token_capacity: Optional[int] = None, causal: bool = True, scale: float = 0.0, seed: int = 0,
               max_pages_per_seq: Optional[int] = None, kv_fp8: bool = False, k_scale: float = 1.0,
               v_scale: float = 1.0, q_scale: float = 0.0) -> BatchMeta:
    """Lay the requests out on randomly permuted physical pages of a pool of ``num_pages`` pages."""
    q_lens = np.asarray(q_lens, dtype=np.int32)
    kv_lens = np.asarray(kv_lens, dtype=np.int32)
    assert q_lens.shape == kv_lens.shape and np.all(q_lens >= 0) and np.all(kv_lens >= q_lens)
    pages_per_seq = -(-kv_lens.astype(np.int64) // page_size)
    needed = int(pages_per_seq.sum())
    if num_pages is None:
        num_pages = max(int(math.ceil(needed * pool_slack)), 1)
    assert num_pages >= needed, f"pool of {num_pages} pages cannot map {needed}"
    if max_pages_per_seq is None:
        max_pages_per_seq = max(int(pages_per_seq.max()) if len(pages_per_seq) else 1, 1)
    rng = np.random.default_rng(seed)
    if num_pages <= 4 * needed + 1024:
        phys = rng.permutation(num_pages)[:needed].astype(np.int32)
    else:  # huge pool: draw distinct ids without materialising a full permutation
        phys = rng.choice(num_pages, size=needed, replace=False).astype(np.int32)
    # entries past a request's last page are never read; -1 makes a stray read easy to spot
    table = np.full((len(q_lens), max_pages_per_seq), -1, dtype=np.int32)
    at = 0
    for r, n in enumerate(pages_per_seq):
        table[r, : int(n)] = phys[at : at + int(n)]
        at += int(n)
    cap = int(q_lens.sum()) if token_capacity is None else int(token_capacity)
    assert cap >= int(q_lens.sum())
    return BatchMeta(name, num_q_heads, num_kv_heads, head_dim, page_size, int(num_pages), int(max_pages_per_seq),
                     q_lens, kv_lens, table, max(cap, 1), causal, scale, seed, kv_fp8, k_scale, v_scale, q_scale)


LLAMA3_8B = dict(num_q_heads=32, num_kv_heads=8, head_dim=128)


def workload_meta(config, seed: Optional[int] = None, *, num_pages: Optional[int] = None,
                  sigma: float = 1.5) -> BatchMeta:
    """Metadata of named workload ``config`` (1..5, or "4b").  ``seed`` defaults to 1000 + config
    (1004 for "4b": the same decode requests and contexts as workload 4)."""
    chunk = 512
    if config == "4b":
        config, chunk = 4, 1000
    seed = 1000 + config if seed is None else seed
    rng = np.random.default_rng(seed)
    if config == 1:
        return build_meta("tiny_mixed", [1, 1, 12, 5], [33, 7, 12, 29], num_q_heads=4, num_kv_heads=2, head_dim=64,
                          page_size=16, num_pages=32, seed=seed, max_pages_per_seq=4)
    if config == 2:
        kv = rng.integers(512, 4096, size=256, endpoint=True)
        return build_meta("llama3_8b_decode", np.ones(256, dtype=np.int32), kv, page_size=16, seed=seed,
                          num_pages=num_pages, **LLAMA3_8B)
    if config == 3:
        return build_meta("llama3_8b_prefill", [8192] * 4, [8192] * 4, page_size=128, num_pages=num_pages or 256,
                          seed=seed, **LLAMA3_8B)
    if config == 4:
        dec_kv = rng.integers(256, 8192, size=192, endpoint=True)
        ctx = rng.integers(0, 4096, size=8, endpoint=True)
        q = np.concatenate([np.ones(192, dtype=np.int64), np.full(8, chunk)])
        kv = np.concatenate([dec_kv, ctx + chunk])
        order = rng.permutation(200)  # requests arrive interleaved; nothing downstream may rely on an order
        name = "llama3_8b_mixed" if chunk == 512 else f"llama3_8b_mixed_chunk{chunk}"
        return build_meta(name, q[order], kv[order], page_size=16, seed=seed, token_capacity=8192,
                          num_pages=num_pages, **LLAMA3_8B)
    if config == 5:
        kv = np.exp(math.log(2048.0) + sigma * rng.standard_normal(512))
        kv = np.clip(np.rint(kv), 1, 131072).astype(np.int64)
        return build_meta("skewed_long_decode", np.ones(512, dtype=np.int32), kv, page_size=128, seed=seed,
                          num_pages=num_pages, **LLAMA3_8B)
    raise ValueError(f"unknown workload {config}")


def _randn_bf16(shape, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)


def _randn_cache(meta: BatchMeta, n_pages: int, gen: torch.Generator, device) -> torch.Tensor:
    """Cache pages of N(0,1) values in the cache's storage type: bf16, or for an FP8 cache the E4M3
    codes (uint8) of value / scale for the K and V combined heads (torch's own conversion)."""
    x = torch.randn((n_pages, meta.page_size, 2 * meta.num_kv_heads, meta.head_dim), generator=gen, device=device,
                    dtype=torch.float32)
    if not meta.kv_fp8:
        return x.to(torch.bfloat16)
    x[:, :, 0::2] /= meta.k_scale
    x[:, :, 1::2] /= meta.v_scale
    return x.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)


def materialize(meta: BatchMeta, device="cpu", *, canaries: bool = False, fill_all_pages: Optional[bool] = None) -> Batch:
    """Draw N(0,1) bf16 values for q, new_k, new_v and the cache.

    Only mapped pages get random values when the pool is much larger than what is mapped (the rest
    holds a constant); ``fill_all_pages`` overrides that choice.  With ``canaries`` every page no
    request maps, and every slot at or past a request's cached context, is filled with bf16 NaN:
    the call must overwrite the slots of the new tokens and must never let the others reach a result.
    """
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(int(meta.seed) * 7919 + 17)
    h_q, h_kv, d, ps = meta.num_q_heads, meta.num_kv_heads, meta.head_dim, meta.page_size
    cap = meta.token_capacity
    q = _randn_bf16((cap, h_q, d), gen, device)
    new_k = _randn_bf16((cap, h_kv, d), gen, device)
    new_v = _randn_bf16((cap, h_kv, d), gen, device)
    mapped = meta.mapped_pages()
    if fill_all_pages is None:
        fill_all_pages = meta.num_pages <= 2 * len(mapped) + 64
    # raw storage: int16 bf16 bit patterns, or uint8 E4M3 codes; NaN canary = 0x7FC0 / 0x7F
    raw_dtype, nan_bits, const_bits = (torch.uint8, 0x7F, 0x30) if meta.kv_fp8 else (torch.int16, 0x7FC0, 0x3F00)
    cache = torch.empty((meta.num_pages, ps, 2 * h_kv, d), dtype=raw_dtype, device=device)

    def raw(t):
        return t if meta.kv_fp8 else t.view(torch.int16)

    if fill_all_pages and not canaries:
        step = max(1, (1 << 28) // (ps * 2 * h_kv * d))
        for p0 in range(0, meta.num_pages, step):
            p1 = min(meta.num_pages, p0 + step)
            cache[p0:p1] = raw(_randn_cache(meta, p1 - p0, gen, device))
    else:
        cache.fill_(nan_bits if canaries else const_bits)
        idx = torch.from_numpy(np.sort(mapped).astype(np.int64)).to(device)
        step = max(1, (1 << 28) // (ps * 2 * h_kv * d))
        for p0 in range(0, len(idx), step):
            sel = idx[p0 : p0 + step]
            cache[sel] = raw(_randn_cache(meta, len(sel), gen, device))
    if canaries:
        c16 = cache
        for r in range(meta.num_seqs):
            ctx = int(meta.kv_lens[r] - meta.q_lens[r])
            n_pages = -(-int(meta.kv_lens[r]) // ps)
            for p in range(ctx // ps, n_pages):
                first = max(ctx - p * ps, 0)
                c16[int(meta.page_table[r, p]), first:] = int(nan_bits)
    if not meta.kv_fp8:
        cache = cache.view(torch.bfloat16)
    return Batch(meta, q, new_k, new_v, cache,
                 torch.from_numpy(meta.page_table.copy()).to(device),
                 torch.from_numpy(meta.cu_q_lens.copy()).to(device),
                 torch.from_numpy(meta.kv_lens.copy()).to(device))


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """Host copy of a bf16 tensor as uint16 bit patterns (a uint8 FP8 cache comes back as uint8 codes)."""
    if t.dtype == torch.uint8:
        return t.detach().contiguous().cpu().numpy()
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def host_subset(batch: Batch, seqs):
    """Compact host copy of the requests ``seqs`` only: their pages (renumbered 0..P-1), their rows
    of q/new_k/new_v and their lengths, for checks on batches whose pool is too large to copy.

    Returns (arrays dict keyed like the call's arguments, number of pages, token rows, page ids)."""
    meta = batch.meta
    ps = meta.page_size
    seqs = list(seqs)
    pages = []
    table = np.full((len(seqs), meta.max_pages_per_seq), -1, np.int32)
    for k, r in enumerate(seqs):
        n = -(-int(meta.kv_lens[r]) // ps)
        table[k, :n] = np.arange(len(pages), len(pages) + n)
        pages.extend(int(p) for p in meta.page_table[r, :n])
    idx = torch.tensor(pages, dtype=torch.long, device=batch.kv_cache.device)
    cache = bf16_bits(batch.kv_cache[idx]).copy()
    cu = meta.cu_q_lens
    rows = np.concatenate([np.arange(cu[r], cu[r + 1]) for r in seqs]) if seqs else np.zeros(0, np.int64)
    ridx = torch.from_numpy(rows.astype(np.int64)).to(batch.q.device)
    sub_cu = np.zeros(len(seqs) + 1, np.int32)
    np.cumsum(meta.q_lens[seqs], out=sub_cu[1:])
    host = dict(q=bf16_bits(batch.q[ridx]), new_k=bf16_bits(batch.new_k[ridx]), new_v=bf16_bits(batch.new_v[ridx]),
                kv_cache=cache, page_table=table, cu_q_lens=sub_cu, kv_lens=meta.kv_lens[seqs].astype(np.int32))
    return host, max(len(pages), 1), rows, pages
