"""Work-counting formulas used to turn a measured time into GB/s, TFLOP/s, MBU and MFU.

The paper defines its decode throughput (Section 4.1.1), its prefill speed with and without a
causal mask (Section 4.2.1) and MBU/MFU on uniform batches; the ragged generalisations below
reduce to them when every request has the same length.  Decimal units (1e9, 1e12) are used
everywhere except in ``paper_decode_throughput``, which keeps the paper's 1024**3 divisor so its
printed tables can be reproduced.
"""
from __future__ import annotations

from typing import Sequence

BF16_BYTES = 2


def algorithmic_bytes(q_lens: Sequence[int], kv_lens: Sequence[int], num_q_heads: int, num_kv_heads: int,
                      head_dim: int, data_bytes: int = BF16_BYTES) -> int:
    """Bytes the method must move: every K/V token of the context read once (cached or new), every
    new token written to the cache once, Q read and the output written.  A request without new tokens
    moves nothing (nobody attends to its context in this call).  With n equal requests of q_len 1 this
    is the numerator of the paper's decode throughput (Section 4.1.1)."""
    token_bytes = 2 * num_kv_heads * head_dim * data_bytes
    qo_bytes = 2 * num_q_heads * head_dim * data_bytes
    return int(sum((int(L) + int(q)) * token_bytes + int(q) * qo_bytes for q, L in zip(q_lens, kv_lens) if int(q) > 0))


def attention_flops(q_lens: Sequence[int], kv_lens: Sequence[int], num_q_heads: int, head_dim: int,
                    causal: bool = True) -> int:
    """Exact-pair FLOPs of QK^T and PV: 4*h_q*d per visible (query, key) pair.  Non-causal with one
    request of s tokens gives the paper's 4*s^2*h_q*d_k (Section 4.2.1)."""
    pairs = 0
    for q, L in zip(q_lens, kv_lens):
        q, L = int(q), int(L)
        pairs += q * (L - q) + q * (q + 1) // 2 if causal else q * L
    return 4 * num_q_heads * head_dim * pairs


def paper_decode_throughput(n: int, context: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
                            seconds: float, data_bytes: int = BF16_BYTES) -> float:
    """The paper's decode throughput exactly as printed (Section 4.1.1): bytes / 1024**3 / time."""
    return n * head_dim * ((context + 1) * 2 * num_kv_heads + 2 * num_q_heads) * data_bytes / (1024 ** 3 * seconds)


def paper_prefill_speed(s: int, num_q_heads: int, head_dim: int, seconds: float, causal: bool, c_kv: int = 0) -> float:
    """The paper's prefill speed in TFLOP/s (Section 4.2.1).  The causal form counts every loaded
    KV compute block of c_kv tokens, masked or not."""
    if causal:
        return 2 * s * (s + c_kv) * num_q_heads * head_dim / (1e12 * seconds)
    return 4 * s * s * num_q_heads * head_dim / (1e12 * seconds)


def utilisation(achieved: float, peak: float) -> float:
    """MBU or MFU as a fraction (Section 4.1.1, Section 4.2.1)."""
    return achieved / peak
