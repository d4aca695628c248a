"""Pins for the FP8 (E4M3) cache path of the CPU oracle (per-tensor quantisation, the paper's
Section 3.8): the quantiser against the format's definition and torch's own float8 conversion, the
attention against dense float64 attention on the dequantised values, and the update against a
direct re-quantisation of the new rows."""
import numpy as np
import pytest
import torch

from oracle import rpa_oracle as orc
from paper_2604_15464_b200 import workloads as wl


def test_e4m3_decode_matches_the_format_definition():
    # sign, 4 exponent bits (bias 7), 3 mantissa bits; no infinities; 0x7F / 0xFF are NaN
    assert orc.e4m3_to_double(0x00) == 0.0 and orc.e4m3_to_double(0x38) == 1.0
    assert orc.e4m3_to_double(0x7E) == 448.0 and orc.e4m3_to_double(0xFE) == -448.0
    assert orc.e4m3_to_double(0x01) == 2.0 ** -9 and orc.e4m3_to_double(0x08) == 2.0 ** -6
    assert np.isnan(orc.e4m3_to_double(0x7F)) and np.isnan(orc.e4m3_to_double(0xFF))
    vals = [orc.e4m3_to_double(c) for c in range(0x7F)]
    assert all(b > a for a, b in zip(vals, vals[1:]))  # codes are monotone in value
    ref = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    for c in range(256):
        v = orc.e4m3_to_double(c)
        assert (np.isnan(v) and np.isnan(ref[c])) or v == ref[c]


def test_e4m3_encode_round_trips_ties_and_saturates():
    for c in range(256):
        v = orc.e4m3_to_double(c)
        if np.isnan(v) or c == 0x80:
            continue
        assert orc.float_to_e4m3(v) == c
    # ties go to the even mantissa: halfway between 1.0 (0x38) and 1.125 (0x39) -> 0x38; next tie -> 0x3A
    assert orc.float_to_e4m3(1.0625) == 0x38 and orc.float_to_e4m3(1.1875) == 0x3A
    # subnormal quantum 2^-9; halfway to the first subnormal rounds to zero (even)
    assert orc.float_to_e4m3(2.0 ** -10) == 0x00 and orc.float_to_e4m3(1.5 * 2.0 ** -9) == 0x02
    assert orc.float_to_e4m3(7.5 * 2.0 ** -9) == 0x08  # carries into the first normal
    # saturation instead of overflow
    assert orc.float_to_e4m3(460.0) == 0x7E and orc.float_to_e4m3(1e9) == 0x7E and orc.float_to_e4m3(-1e9) == 0xFE
    assert orc.float_to_e4m3(float("inf")) == 0x7E


def test_e4m3_encode_matches_torch_conversion_inside_the_finite_range():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000) * 50, rng.standard_normal(5000) * 0.01,
                        rng.uniform(-448, 448, 5000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([orc.float_to_e4m3(v) for v in x], dtype=np.uint8)
    diff = got != ref
    # +0 / -0 aside, the two agree everywhere
    assert not np.any(diff & ((got & 0x7F) != 0))


def _f64(bits):
    return torch.from_numpy(bits.astype(np.int32) << 16).view(torch.float32).double()


CASES = [([1, 1, 12, 5], [33, 7, 12, 29], 4, 2, 64, 16), ([3, 0, 1, 40], [3, 0, 130, 40], 8, 2, 32, 8)]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("causal", [True, False])
def test_fp8_forward_matches_dense_attention_on_dequantised_kv(case, causal):
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("fp8", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=17,
                         causal=causal, kv_fp8=True, k_scale=0.023, v_scale=0.031)
    batch = wl.materialize(meta)
    shape = orc.OracleShape(hq, hkv, d, ps, meta.num_pages, meta.max_pages_per_seq, meta.sm_scale, causal, True,
                            meta.k_scale, meta.v_scale)
    cache = wl.bf16_bits(batch.kv_cache).copy()
    assert cache.dtype == np.uint8
    before = cache.copy()
    out = orc.forward(shape, wl.bf16_bits(batch.q), wl.bf16_bits(batch.new_k), wl.bf16_bits(batch.new_v), cache,
                      meta.page_table, meta.cu_q_lens, meta.kv_lens)
    # the update, re-derived with torch's conversion: code = e4m3(float32(new) * float32(1/scale))
    nk = _f64(wl.bf16_bits(batch.new_k)).float()
    nv = _f64(wl.bf16_bits(batch.new_v)).float()
    inv_k = np.float32(1.0) / np.float32(meta.k_scale)
    inv_v = np.float32(1.0) / np.float32(meta.v_scale)
    qk = (nk * float(inv_k)).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    qv = (nv * float(inv_v)).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    expect = before.copy()
    for r in range(meta.num_seqs):
        for i in range(int(meta.q_lens[r])):
            pos = int(meta.kv_lens[r] - meta.q_lens[r]) + i
            page, slot = int(meta.page_table[r, pos // ps]), pos % ps
            tok = int(meta.cu_q_lens[r]) + i
            expect[page, slot, 0::2] = qk[tok]
            expect[page, slot, 1::2] = qv[tok]
    same = (cache == expect) | (((cache & 0x7F) == 0) & ((expect & 0x7F) == 0))  # +-0 are the same value
    assert np.all(same)
    # attention on dequantised values, float64, dense
    deq = torch.from_numpy(cache).view(torch.float8_e4m3fn).double()
    deq[:, :, 0::2] *= float(np.float32(meta.k_scale))
    deq[:, :, 1::2] *= float(np.float32(meta.v_scale))
    q = _f64(wl.bf16_bits(batch.q))
    h_g = hq // hkv
    for r in range(meta.num_seqs):
        qlen, L = int(meta.q_lens[r]), int(meta.kv_lens[r])
        if qlen == 0:
            continue
        slots = torch.stack([deq[int(meta.page_table[r, t // ps]), t % ps] for t in range(L)])  # [L, 2h_kv, d]
        K = slots[:, 0::2].repeat_interleave(h_g, dim=1)
        V = slots[:, 1::2].repeat_interleave(h_g, dim=1)
        t0 = int(meta.cu_q_lens[r])
        S = torch.einsum("iad,tad->ait", q[t0 : t0 + qlen], K) * meta.sm_scale
        if causal:
            key = torch.arange(L)[None, :]
            qpos = (L - qlen + torch.arange(qlen))[:, None]
            S = S.masked_fill((key > qpos)[None], float("-inf"))
        ref = torch.einsum("ait,tad->iad", torch.softmax(S, dim=-1), V).numpy()
        assert np.max(np.abs(out[t0 : t0 + qlen] - ref)) < 1e-12


# ---- per-tensor quantisation of Q (Section 3.8: Q, K and V each share one scalar scale) ----

def _q_image_bits(q_bits, q_scale):
    """bf16 bit patterns of e4m3(float32(q) * float32(1/q_scale)), the E4M3 image of Q WITHOUT its
    scale, computed with torch's own float8 conversion (every E4M3 value is exact in bf16)."""
    qf = _f64(q_bits).float()
    inv = float(np.float32(1.0) / np.float32(q_scale))
    img = (qf * inv).clamp(-448, 448).to(torch.float8_e4m3fn).float()
    return img.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("q_scale", [0.0625, 0.03, 0.011])
def test_quantised_q_equals_the_unquantised_oracle_on_the_e4m3_image_of_q(case, q_scale):
    """With q_scale set the oracle must give what it gives without it on Q replaced by its E4M3 image
    (made by torch, not by the oracle) with the scale of Q folded into the softmax scale.  Pins the
    conversion, the place where the scale enters and that nothing but the scores sees it."""
    ql, kl, hq, hkv, d, ps = case
    meta = wl.build_meta("fp8q", ql, kl, num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=19,
                         kv_fp8=True, k_scale=0.023, v_scale=0.031)
    batch = wl.materialize(meta)
    args = (wl.bf16_bits(batch.new_k), wl.bf16_bits(batch.new_v))
    base = dict(num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, num_pages=meta.num_pages,
                max_pages_per_seq=meta.max_pages_per_seq, causal=True, kv_fp8=True, k_scale=meta.k_scale, v_scale=meta.v_scale)
    q_bits = wl.bf16_bits(batch.q)
    cache_a, cache_b = wl.bf16_bits(batch.kv_cache).copy(), wl.bf16_bits(batch.kv_cache).copy()
    got = orc.forward(orc.OracleShape(scale=meta.sm_scale, q_scale=q_scale, **base), q_bits, *args, cache_a,
                      meta.page_table, meta.cu_q_lens, meta.kv_lens)
    folded = meta.sm_scale * float(np.float32(q_scale))
    want = orc.forward(orc.OracleShape(scale=folded, q_scale=0.0, **base), _q_image_bits(q_bits, q_scale), *args, cache_b,
                       meta.page_table, meta.cu_q_lens, meta.kv_lens)
    assert np.array_equal(cache_a, cache_b)  # the cache update does not depend on the scale of Q
    assert np.max(np.abs(got - want)) < 1e-12
    # and it differs from the bf16-Q result by what E4M3's 3 mantissa bits allow, no more: a dropped
    # quantisation (or a scale applied twice) fails one of the two bounds
    cache_c = wl.bf16_bits(batch.kv_cache).copy()
    plain = orc.forward(orc.OracleShape(scale=meta.sm_scale, q_scale=0.0, **base), q_bits, *args, cache_c,
                        meta.page_table, meta.cu_q_lens, meta.kv_lens)
    diff = np.abs(got - plain)
    assert 1e-6 < diff.max() < 0.5


def test_q_scale_is_rejected_without_an_fp8_cache_and_when_negative():
    meta = wl.build_meta("fp8q-bad", [2], [9], num_q_heads=4, num_kv_heads=2, head_dim=32, page_size=8, seed=20)
    batch = wl.materialize(meta)
    base = dict(num_q_heads=4, num_kv_heads=2, head_dim=32, page_size=8, num_pages=meta.num_pages,
                max_pages_per_seq=meta.max_pages_per_seq, scale=meta.sm_scale)
    with pytest.raises(ValueError):
        orc.forward(orc.OracleShape(q_scale=0.05, **base), wl.bf16_bits(batch.q), wl.bf16_bits(batch.new_k),
                    wl.bf16_bits(batch.new_v), wl.bf16_bits(batch.kv_cache).copy(), meta.page_table, meta.cu_q_lens,
                    meta.kv_lens)


def test_q_saturates_at_the_largest_e4m3_value():
    """A query element beyond 448 * q_scale is clamped, as K and V are: with a single key the output
    is that key's value whatever Q is, so use two keys whose scores differ only through the clamp."""
    hq = hkv = 1
    d, ps = 16, 8
    meta = wl.build_meta("fp8q-sat", [1], [2], num_q_heads=hq, num_kv_heads=hkv, head_dim=d, page_size=ps, seed=21,
                         kv_fp8=True, k_scale=1.0, v_scale=1.0)
    q = torch.zeros(1, 1, d)
    q[0, 0, 0] = 1000.0  # far beyond 448 * q_scale
    to_bits = lambda t: t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    k_new = torch.zeros(1, 1, d); k_new[0, 0, 0] = 1.0
    v_new = torch.ones(1, 1, d)
    cache = np.zeros((meta.num_pages, ps, 2, d), np.uint8)  # cached key 0 = 0 -> score 0; value 0
    shape = orc.OracleShape(hq, hkv, d, ps, meta.num_pages, meta.max_pages_per_seq, 0.01, True, True, 1.0, 1.0, 1.0)
    out = orc.forward(shape, to_bits(q), to_bits(k_new), to_bits(v_new), cache, meta.page_table, meta.cu_q_lens, meta.kv_lens)
    # scores: key 0 -> 0, key 1 -> 0.01 * 448 * 1 (clamped), not 0.01 * 1000; value 1 for key 1, 0 for key 0
    w = np.exp(0.01 * 448.0)
    assert abs(out[0, 0, 0] - w / (1.0 + w)) < 1e-12
