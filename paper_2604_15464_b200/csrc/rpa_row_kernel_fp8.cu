#include <algorithm>
// Split-KV row kernel on an FP8 (E4M3) cache with per-tensor scales (the paper's Section 3.8).
//
// Same work items, ring structure, softmax and merge as rpa_row_kernel.cu; what changes is the data
// type of the cache.  A cached element is one byte standing for byte_value * scale, so a position
// costs half the HBM bytes.  Stages hold the raw FP8 bytes; fragments are converted to f16 in
// registers (every E4M3 value is exact in f16) and the products run as f16 warp MMAs with fp32
// accumulation; k_scale is folded into the softmax scale and v_scale into the final normalisation.
//   * K fragments: one ldmatrix over FP8 bytes hands each lane four consecutive d-elements of a
//     16-element step instead of the canonical (2c, 2c+1, 2c+8, 2c+9); Q fragments are read with the
//     same permutation of the contraction index, which leaves the dot product unchanged.
//   * V fragments: a transposing ldmatrix moves 2-byte units, i.e. pairs of d-elements, so one
//     register holds (token 2c, token 2c+1) x (d 2j, d 2j+1); a byte permute splits it into the
//     B fragments of two MMAs, one for the even and one for the odd d-elements of a 16-wide chunk.
//     A lane therefore ends up with four consecutive output columns.
//   * The batch's own new tokens are attended in quantised precision, like every later step will
//     see them: their rows are quantised on the way into shared memory, and the fused cache update
//     stores the same codes:  e4m3(float(x) * (1/scale)), round to nearest even, saturating.
//   * NARROW instantiation, for lists whose items all have at most 8 query rows (decode with up to
//     8 grouped heads): the score product keeps its shape with the upper 8 rows of the Q fragment
//     zero, but the second product runs transposed, O^T = V^T P^T.  The score accumulators of a lane
//     (row lane/4, keys 2c, 2c+1 of each 8-key half) are exactly the B fragment of P^T, the
//     transposed V registers split by byte permute into the even-d and odd-d halves of one A
//     fragment, and the output state shrinks to 8 rows: half the second product's MMAs, half the
//     accumulator registers, half the softmax arithmetic, and room for a fourth CTA per SM.
#include <cuda_bf16.h>

#include "rpa_fp8.cuh"
#include "rpa_kernels.h"
#include "rpa_ptx.cuh"
#include "rpa_row_common.cuh"

namespace rpa {

namespace {

template <int D, bool NARROW>
struct Row8Cfg {
    static constexpr int NW = 4;                 // warps per CTA
    static constexpr int ROWS = NARROW ? 8 : kRowTileRows;  // query rows of the tile
    // ring depth per warp (stages are half as large as with bf16); at d_k = 128 four stages and Q
    // fragments re-read from shared memory let three CTAs share an SM: the conversions make this
    // kernel issue-bound, and 12 warps hide their latency better than 8.  The narrow tile needs
    // fewer registers: three stages per warp make room for 16 warps.
    static constexpr int STAGES = NARROW ? (D == 64 ? 6 : 3) : (D == 128 ? 4 : 6);
    static constexpr int ROWB = D;               // bytes of one K (or V) row
    static constexpr int HALF = kKvTile * ROWB;  // bytes of the K part of a stage
    static constexpr int STAGE = 2 * HALF;
    static constexpr int CPR = D / 16;           // 16-byte chunks per K (or V) row
    static constexpr int CPP = 2 * CPR;          // chunks per position (K then V)
    static constexpr int LOAD_ITERS = kKvTile * CPP / 32;
    static constexpr int QROW = 2 * D + 32;      // bytes of one f16 Q row, padded against bank conflicts
    static constexpr int QBYTES = ROWS * QROW;
    static constexpr int OSTRIDE = D + 8;        // floats per row of the merge scratch
    static constexpr int SMEM = QBYTES + NW * STAGES * STAGE;
    static constexpr int CTAS_PER_SM = NARROW ? (D <= 128 ? 4 : 2) : (D == 64 ? 3 : D == 128 ? 3 : 1);
    static constexpr bool Q_IN_REGS = NARROW || D <= 64;
    static_assert(STAGES * STAGE >= ROWS * OSTRIDE * 4 + ROWS * 8, "merge scratch fits the ring");
    // physical 16-byte chunk of logical chunk ch in row r: spreads 8 rows over all banks
    __device__ static __forceinline__ int swz(int r, int ch) { return ROWB >= 128 ? (ch ^ (r & 7)) : (ch ^ ((r >> 1) & 3)); }
};

__device__ __forceinline__ void mma_f16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// One row item, start to finish, by the whole CTA.
template <int D, int G, bool NARROW>
__device__ __forceinline__ void row_item_fp8(const KernelArgs& a, int item_index, uint8_t* smem) {
    using C = Row8Cfg<D, NARROW>;
    constexpr int ROWS = C::ROWS;
    constexpr int NW = C::NW, STAGES = C::STAGES, ROWB = C::ROWB, CPR = C::CPR, CPP = C::CPP;
    constexpr int NTHREADS = NW * 32;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const RowItem it = a.row_items[item_index];
    const int h = it.kv_head;
    // Page ids of this warp's first 32 KV tiles: their addresses need the item only, so the loads go
    // out together with the loads of the sequence's lengths instead of after them.  (Positions of
    // the batch's own tokens have mapped pages too; whether a tile is read from the cache at all is
    // decided later.)
    const int32_t* pt_row = a.page_table + (int64_t)it.seq * a.max_pages_per_seq;
    int page_reg = 0;
    {
        const int t = it.kv_begin / kKvTile + warp + lane * NW;
        if (t * kKvTile < it.kv_end) page_reg = pt_row[t * kKvTile / a.page_size];
    }
    const int cu = a.cu_q_lens[it.seq];
    const int q_r = a.cu_q_lens[it.seq + 1] - cu;
    const int L = a.kv_lens[it.seq];
    const int c = L - q_r;  // cached context length
    const int ps = a.page_size;
    const int64_t slot_bytes = (int64_t)2 * a.h_kv * D;  // one byte per element
    const int64_t tok0 = (int64_t)cu + it.q_tok0;
    if (!debug_rows_ok(a, tok0, it.n_tok)) return;  // (bounds-checked build only)
    uint8_t* cache8 = reinterpret_cast<uint8_t*>(a.kv_cache);

    // ---- this warp's share of the KV tiles ----
    const int t_begin = it.kv_begin / kKvTile;
    const int t_end = (it.kv_end + kKvTile - 1) / kKvTile;
    const int n_my = t_end - t_begin - warp > 0 ? (t_end - t_begin - warp + NW - 1) / NW : 0;
    uint8_t* ring_ptr = smem + C::QBYTES + warp * STAGES * C::STAGE;
    const uint32_t ring = smem_u32(ring_ptr);
    const int fast_end = min(c, it.kv_end);  // tiles wholly below this come straight from one page

    auto load_tile = [&](int kl) {
        if ((kl & 31) == 0 && kl > 0) {  // refill the page ids of this warp's next 32 tiles
            const int t = t_begin + warp + (kl + lane) * NW;
            const int pos0 = t * kKvTile;
            page_reg = (t < t_end && pos0 < c) ? pt_row[pos0 / ps] : 0;
        }
        const int page = debug_read_page(a, __shfl_sync(0xffffffffu, page_reg, kl & 31));
        if (kl < n_my && !(a.ablation & kAblateLoads)) {
            const int pos0 = (t_begin + warp + kl * NW) * kKvTile;
            const int stage_off = (kl % STAGES) * C::STAGE;
            if (!debug_stage_ok(a, kl % STAGES, STAGES)) return;
            if (pos0 + kKvTile <= fast_end) {
                const uint8_t* base = cache8 + ((int64_t)page * ps + pos0 % ps) * slot_bytes + (int64_t)2 * h * D;
#pragma unroll
                for (int i = 0; i < C::LOAD_ITERS; ++i) {
                    const int ci = i * 32 + lane;
                    const int r = ci / CPP, cc = ci % CPP;
                    const int is_v = cc >= CPR, ch = cc - is_v * CPR;
                    cp_async_16(ring + stage_off + is_v * C::HALF + r * ROWB + (C::swz(r, ch) << 4), base + r * slot_bytes + cc * 16,
                                16);
                }
            } else {
#pragma unroll
                for (int i = 0; i < C::LOAD_ITERS; ++i) {
                    const int ci = i * 32 + lane;
                    const int r = ci / CPP, cc = ci % CPP;
                    const int is_v = cc >= CPR, ch = cc - is_v * CPR;
                    const int p = pos0 + r;
                    const int dst_off = stage_off + is_v * C::HALF + r * ROWB + (C::swz(r, ch) << 4);
                    if (p >= c && p < it.kv_end) {
                        // one of the batch's own new tokens: quantise its row on the way in
                        const uint16_t* src = (is_v ? a.new_v : a.new_k) + (((int64_t)cu + (p - c)) * a.h_kv + h) * D + ch * 16;
                        *reinterpret_cast<uint4*>(ring_ptr + dst_off) = quantise16(src, is_v ? a.inv_v_scale : a.inv_k_scale);
                    } else {
                        const uint8_t* src = cache8;
                        uint32_t bytes = 0;  // past kv_end: zero-fill (masked scores, finite V rows)
                        if (p < c) {
                            const int pg = debug_read_page(a, pt_row[p / ps]);
                            src = cache8 + ((int64_t)pg * ps + p % ps) * slot_bytes + (int64_t)2 * h * D + cc * 16;
                            bytes = 16;
                        }
                        cp_async_16(ring + dst_off, src, bytes);
                    }
                }
            }
        }
        cp_async_commit();
    };
    // The first stages go out before anything else of the item: the cache update and the Q tile below
    // wait on global loads of their own, and the K/V stream should not queue behind them.
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) load_tile(s);

    // ---- fused cache update: quantise this item's K and V rows, 16 elements per thread and step ----
    if ((it.flags & kFlagWriteKv) && !(a.ablation & kAblateUpdate)) {
        for (int idx = tid; idx < it.n_tok * CPP; idx += NTHREADS) {
            const int j = idx / CPP, cc = idx % CPP;
            const bool is_v = cc >= CPR;
            const int ch = cc - (is_v ? CPR : 0);
            const int pos = c + it.q_tok0 + j;
            const int page = pt_row[pos / ps];
            if (!debug_write_page_ok(a, page)) continue;
            uint8_t* dst = cache8 + ((int64_t)page * ps + pos % ps) * slot_bytes + (int64_t)2 * h * D + cc * 16;
            const uint16_t* src = (is_v ? a.new_v : a.new_k) + ((tok0 + j) * a.h_kv + h) * D + ch * 16;
            *reinterpret_cast<uint4*>(dst) = quantise16(src, is_v ? a.inv_v_scale : a.inv_k_scale);
        }
    }

    // ---- Q tile as f16: row rho = token rho / G, grouped head rho % G; rows past n_tok are zero ----
    uint8_t* q_s = smem;
    for (int idx = tid; idx < ROWS * (D / 8); idx += NTHREADS) {
        const int row = idx / (D / 8), ch = idx % (D / 8);
        const int j = row / G, g = row % G;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < it.n_tok) {
            const uint4 x = ld_global_nc_v4(a.q + ((tok0 + j) * a.h_q + h * G + g) * D + ch * 8);
            v.x = pack_f16x2(bf16_bits_lo(x.x), bf16_bits_hi(x.x));
            v.y = pack_f16x2(bf16_bits_lo(x.y), bf16_bits_hi(x.y));
            v.z = pack_f16x2(bf16_bits_lo(x.z), bf16_bits_hi(x.z));
            v.w = pack_f16x2(bf16_bits_lo(x.w), bf16_bits_hi(x.w));
        }
        *reinterpret_cast<uint4*>(q_s + row * C::QROW + ch * 16) = v;
    }
    __syncthreads();
    // Q fragment of step ks, in the contraction order the K fragments come in: a lane's slots
    // (2c, 2c+1) hold d = 16ks + 4c, +1 and its slots (2c+8, 2c+9) hold d = 16ks + 4c + 2, +3.
    const uint8_t* q_lane = q_s + (lane >> 2) * C::QROW + (lane & 3) * 8;
    auto load_q_frag = [&](uint32_t (&f)[4], int ks) {
        const uint2 lo = *reinterpret_cast<const uint2*>(q_lane + ks * 32);
        f[0] = lo.x;
        f[2] = lo.y;
        if constexpr (NARROW) {
            f[1] = f[3] = 0u;  // rows 8-15 of the fragment do not exist
        } else {
            const uint2 hi = *reinterpret_cast<const uint2*>(q_lane + 8 * C::QROW + ks * 32);
            f[1] = hi.x;
            f[3] = hi.y;
        }
    };
    uint32_t qf[C::Q_IN_REGS ? D / 16 : 1][4];
    if (C::Q_IN_REGS) {
#pragma unroll
        for (int ks = 0; ks < (C::Q_IN_REGS ? D / 16 : 1); ++ks) load_q_frag(qf[ks], ks);
    }


    // per-thread softmax state for rows rho0 = lane/4 and rho0 + 8
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    // wide: o[2g + parity] holds output columns 16g + 2n + parity of a 16-wide chunk g;
    // narrow: o[g] holds O^T, columns (16g + 2*(lane/4), +1) of rows 2c and 2c+1
    constexpr int NO = NARROW ? D / 16 : D / 8;
    float o[NO][4];
#pragma unroll
    for (int n = 0; n < NO; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

    int lim[2];  // last visible position of each of the two rows
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        const int j = min(((lane >> 2) + 8 * e) / G, it.n_tok - 1);
        lim[e] = min(a.causal ? c + it.q_tok0 + j : L - 1, it.kv_end - 1);
    }
    const int unmasked_end = min(it.kv_end, a.causal ? c + it.q_tok0 + 1 : L);

    for (int k = 0; k < n_my; ++k) {
        cp_async_wait<STAGES - 2>();
        __syncwarp();
        load_tile(k + STAGES - 1);
        if (a.ablation & kAblateCompute) continue;  // data movement only

        const uint32_t k_s = ring + (k % STAGES) * C::STAGE, v_s = k_s + C::HALF;
        const int pos0 = (t_begin + warp + k * NW) * kKvTile;

        // S = Q K^T for 16 rows x 16 positions
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
        {
            const int mi = lane >> 3, r = ((mi & 1) << 3) + (lane & 7);
            const uint32_t base = k_s + r * ROWB;
#pragma unroll
            for (int kp = 0; kp < D / 32; ++kp) {
                uint32_t b[4];  // tokens 0-7 / 8-15 of step 2kp, then of step 2kp+1; four consecutive d each
                ldmatrix_x4(b, base + (C::swz(r, 2 * kp + (mi >> 1)) << 4));
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int ks = 2 * kp + half;
                    uint32_t qk[4];
                    if (!C::Q_IN_REGS) load_q_frag(qk, ks);
                    const uint32_t(&qa)[4] = C::Q_IN_REGS ? qf[C::Q_IN_REGS ? ks : 0] : qk;
                    uint32_t k0, k1, k2, k3;
                    e4m3x4_to_f16x2x2(b[2 * half], k0, k1);
                    e4m3x4_to_f16x2x2(b[2 * half + 1], k2, k3);
                    mma_f16_16816(s[0], qa, k0, k1);
                    mma_f16_16816(s[1], qa, k2, k3);
                }
            }
        }
        const bool need_mask = pos0 + kKvTile > unmasked_end;
        if constexpr (NARROW) {
            // this lane's row lane/4: keys (2c, 2c+1) of both 8-key halves
            float p[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int pos = pos0 + (e >> 1) * 8 + 2 * (lane & 3) + (e & 1);
                float v = s[e >> 1][e & 1] * a.scale_log2;
                if (need_mask && pos > lim[0]) v = -INFINITY;
                p[e] = v;
            }
            float mx = fmaxf(fmaxf(p[0], p[1]), fmaxf(p[2], p[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(m_run[0], mx);
            const float m_use = m_new == -INFINITY ? 0.f : m_new;  // a row that has seen nothing yet
            const float alpha = fast_exp2(m_run[0] - m_use);
            m_run[0] = m_new;
#pragma unroll
            for (int e = 0; e < 4; ++e) p[e] = fast_exp2(p[e] - m_use);
            l_run[0] = l_run[0] * alpha + (p[0] + p[1]) + (p[2] + p[3]);
            // P^T as the B fragment: slots (2c, 2c+1) of the first half, (2c+8, 2c+9) of the second
            const uint32_t pb0 = pack_f16x2(p[0], p[1]), pb1 = pack_f16x2(p[2], p[3]);
            // O^T = alpha * O^T + V^T P^T; the accumulators of this lane belong to rows 2c and 2c+1,
            // whose factors live in lanes 8c and 8c+4
            if (__any_sync(0xffffffffu, alpha != 1.f)) {
                const float a0 = __shfl_sync(0xffffffffu, alpha, 8 * (lane & 3));
                const float a1 = __shfl_sync(0xffffffffu, alpha, 8 * (lane & 3) + 4);
#pragma unroll
                for (int n = 0; n < NO; ++n) {
                    o[n][0] *= a0;
                    o[n][1] *= a1;
                    o[n][2] *= a0;
                    o[n][3] *= a1;
                }
            }
            const int mi = lane >> 3, r = ((mi & 1) << 3) + (lane & 7);
            const uint32_t base = v_s + r * ROWB;
#pragma unroll
            for (int gp = 0; gp < D / 32; ++gp) {
                uint32_t b[4];  // (token 2c, 2c+1) x (d 2j, 2j+1) of tokens 0-7 / 8-15, chunk 2gp then 2gp+1
                ldmatrix_x4_trans(b, base + (C::swz(r, 2 * gp + (mi >> 1)) << 4));
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    // A fragment of V^T: rows 0-7 are the even d-elements of the chunk, rows 8-15 the odd ones
                    uint32_t va[4];  // bytes (0,2 | 1,3): one d-element of two tokens per half
                    e4m3x4_to_f16x2x2(__byte_perm(b[2 * half], 0, 0x3120u), va[0], va[1]);
                    e4m3x4_to_f16x2x2(__byte_perm(b[2 * half + 1], 0, 0x3120u), va[2], va[3]);
                    mma_f16_16816(o[2 * gp + half], va, pb0, pb1);
                }
            }
        } else {
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int pos = pos0 + nt * 8 + 2 * (lane & 3) + (e & 1);
                    float v = s[nt][e] * a.scale_log2;
                    if (need_mask && pos > lim[e >> 1]) v = -INFINITY;
                    s[nt][e] = v;
                }
            // online softmax (Algorithm 1, lines "m~, P, l~, C~o"), base-2 exponentials
            float alpha[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float mx = fmaxf(fmaxf(s[0][2 * e], s[0][2 * e + 1]), fmaxf(s[1][2 * e], s[1][2 * e + 1]));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run[e], mx);
                const float m_use = m_new == -INFINITY ? 0.f : m_new;  // a row that has seen nothing yet
                alpha[e] = fast_exp2(m_run[e] - m_use);
                m_run[e] = m_new;
                float sum = 0.f;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    s[nt][2 * e] = fast_exp2(s[nt][2 * e] - m_use);
                    s[nt][2 * e + 1] = fast_exp2(s[nt][2 * e + 1] - m_use);
                    sum += s[nt][2 * e] + s[nt][2 * e + 1];
                }
                l_run[e] = l_run[e] * alpha[e] + sum;
            }
            uint32_t pf[4];
            pf[0] = pack_f16x2(s[0][0], s[0][1]);
            pf[1] = pack_f16x2(s[0][2], s[0][3]);
            pf[2] = pack_f16x2(s[1][0], s[1][1]);
            pf[3] = pack_f16x2(s[1][2], s[1][3]);
            // O = alpha * O + P V; once the running maxima have settled alpha is exactly 1 and the
            // rescale of the accumulator is skipped (the test is warp-uniform)
            if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
                for (int n = 0; n < D / 8; ++n) {
                    o[n][0] *= alpha[0];
                    o[n][1] *= alpha[0];
                    o[n][2] *= alpha[1];
                    o[n][3] *= alpha[1];
                }
            }
            {
                const int mi = lane >> 3, r = ((mi & 1) << 3) + (lane & 7);
                const uint32_t base = v_s + r * ROWB;
#pragma unroll
                for (int gp = 0; gp < D / 32; ++gp) {
                    uint32_t b[4];  // (token 2c, 2c+1) x (d 2j, 2j+1) of tokens 0-7 / 8-15, chunk 2gp then 2gp+1
                    ldmatrix_x4_trans(b, base + (C::swz(r, 2 * gp + (mi >> 1)) << 4));
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const int g = 2 * gp + half;
                        // bytes (0,2 | 1,3): the even d-element of two tokens, then the odd one
                        uint32_t e0, o0, e1, o1;
                        e4m3x4_to_f16x2x2(__byte_perm(b[2 * half], 0, 0x3120u), e0, o0);
                        e4m3x4_to_f16x2x2(__byte_perm(b[2 * half + 1], 0, 0x3120u), e1, o1);
                        mma_f16_16816(o[2 * g], pf, e0, e1);
                        mma_f16_16816(o[2 * g + 1], pf, o0, o1);
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
#pragma unroll
    for (int e = 0; e < 2; ++e) {
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 1);
        l_run[e] += __shfl_xor_sync(0xffffffffu, l_run[e], 2);
    }
    __syncwarp();

    // ---- merge the warps' states through shared memory (each warp reuses its own ring) ----
    float* o_s = reinterpret_cast<float*>(ring_ptr);
    float* ml_s = o_s + ROWS * C::OSTRIDE;
    if constexpr (NARROW) {
        const int r0 = 2 * (lane & 3), col = 2 * (lane >> 2);  // rows 2c, 2c+1; two consecutive columns per chunk
#pragma unroll
        for (int g = 0; g < D / 16; ++g) {
            *reinterpret_cast<float2*>(o_s + r0 * C::OSTRIDE + g * 16 + col) = make_float2(o[g][0], o[g][2]);
            *reinterpret_cast<float2*>(o_s + (r0 + 1) * C::OSTRIDE + g * 16 + col) = make_float2(o[g][1], o[g][3]);
        }
        if ((lane & 3) == 0) {
            ml_s[lane >> 2] = m_run[0];
            ml_s[ROWS + (lane >> 2)] = l_run[0];
        }
    } else {
        const int r0 = lane >> 2, col = 4 * (lane & 3);  // four consecutive columns per 16-wide chunk
#pragma unroll
        for (int g = 0; g < D / 16; ++g) {
            *reinterpret_cast<float4*>(o_s + r0 * C::OSTRIDE + g * 16 + col) =
                make_float4(o[2 * g][0], o[2 * g + 1][0], o[2 * g][1], o[2 * g + 1][1]);
            *reinterpret_cast<float4*>(o_s + (r0 + 8) * C::OSTRIDE + g * 16 + col) =
                make_float4(o[2 * g][2], o[2 * g + 1][2], o[2 * g][3], o[2 * g + 1][3]);
        }
        if ((lane & 3) == 0) {
            ml_s[r0] = m_run[0];
            ml_s[r0 + 8] = m_run[1];
            ml_s[ROWS + r0] = l_run[0];
            ml_s[ROWS + r0 + 8] = l_run[1];
        }
    }
    __syncthreads();
    constexpr int WARP_FLOATS = STAGES * C::STAGE / 4;
    const float* o_all = reinterpret_cast<const float*>(smem + C::QBYTES);
    for (int idx = tid; idx < ROWS * (D / 4); idx += NTHREADS) {
        const int row = idx / (D / 4), c4 = idx % (D / 4);
        const int j = row / G, g = row % G;
        if (j >= it.n_tok) continue;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, o_all[w * WARP_FLOATS + ROWS * C::OSTRIDE + row]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float* base = o_all + w * WARP_FLOATS;
            const float mw = base[ROWS * C::OSTRIDE + row];
            const float f = mw == -INFINITY ? 0.f : fast_exp2(mw - M);
            const float4 v = *reinterpret_cast<const float4*>(base + row * C::OSTRIDE + c4 * 4);
            acc.x += f * v.x;
            acc.y += f * v.y;
            acc.z += f * v.z;
            acc.w += f * v.w;
            lsum += f * base[ROWS * C::OSTRIDE + ROWS + row];
        }
        if (it.partial < 0) {
            const float inv = a.out_scale / lsum;  // v_scale folded into the normalisation
            uint2 packed;
            packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
            packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(a.out + ((tok0 + j) * a.h_q + h * G + g) * D + c4 * 4) = packed;
        } else {
            const int64_t prow = (int64_t)it.partial * kRowTileRows + row;
            *reinterpret_cast<float4*>(a.partial_o + prow * D + c4 * 4) = acc;
            if (c4 == 0) *reinterpret_cast<float2*>(a.partial_ml + prow * 2) = make_float2(M, lsum);
        }
    }
    // ---- the CTA that delivers a group's last partial also combines the group ----
    if (it.partial >= 0 && a.group_counters != nullptr) {
        __shared__ int s_last;
        const int group = (it.flags >> kFlagGroupShift) - 1;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const int ticket = atomicAdd(a.group_counters + group, 1);
            s_last = ticket == a.groups[group].n_partials - 1;
            if (s_last) a.group_counters[group] = 0;
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            const CombineGroup gr = a.groups[group];
            combine_group<D>(a, gr, tid, NTHREADS);
        }
    }
}

template <int D, int G, bool NARROW>
__global__ void __launch_bounds__(Row8Cfg<D, NARROW>::NW * 32, Row8Cfg<D, NARROW>::CTAS_PER_SM) rpa_row_kernel_fp8(const KernelArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    if (a.validated && (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput)) return;  // inputs were rejected
    row_item_fp8<D, G, NARROW>(a, blockIdx.x, smem);
}

// The same items from a list planned on the device: a fixed grid striding over a list whose length
// is read from device memory (see rpa_row_kernel_strided).  The planner also leaves the largest
// number of query rows of any item; the narrow and the wide instantiation are both launched (on two
// streams: they never both work) and the one the list does not call for returns at once.
template <int D, int G, bool NARROW>
__global__ void __launch_bounds__(Row8Cfg<D, NARROW>::NW * 32, Row8Cfg<D, NARROW>::CTAS_PER_SM)
    rpa_row_kernel_fp8_strided(const KernelArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    if (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput) return;  // the planner rejected the lengths
    if (G <= 8 && (a.dev_counts[kDevCountRowRows] <= 8) != NARROW) return;          // the other instantiation's list
    const int n = a.dev_counts[kDevCountRows];
    // the list is sorted longest first: dealing it back and forth (CTA b takes b, 2G-1-b, 2G+b, ...)
    // pairs the longest items of one pass with the shortest of the next
    const int G_ = (int)gridDim.x, b = (int)blockIdx.x;
    for (int w = 0; w * G_ < n; ++w) {
        const int i = (w & 1) ? (w + 1) * G_ - 1 - b : w * G_ + b;
        if (i >= n) continue;
        row_item_fp8<D, G, NARROW>(a, i, smem);
        __syncthreads();  // the next item reuses the shared memory
    }
}

template <int D, int G>
cudaError_t launch_row8(const KernelArgs& a, cudaStream_t stream) {
    if (G <= 8 && a.row_rows_max > 0 && a.row_rows_max <= 8) {  // (0: the caller did not say - the 16-row one serves any list)
        using C = Row8Cfg<D, (G <= 8)>;
        rpa_row_kernel_fp8<D, G, (G <= 8)><<<a.num_row_items, C::NW * 32, C::SMEM, stream>>>(a);
    } else {
        using C = Row8Cfg<D, false>;
        rpa_row_kernel_fp8<D, G, false><<<a.num_row_items, C::NW * 32, C::SMEM, stream>>>(a);
    }
    return cudaGetLastError();
}

template <int D, int G>
cudaError_t launch_row8_strided(const KernelArgs& a, int grid, bool narrow, cudaStream_t stream) {
    if (narrow) {
        if (G > 8) return cudaSuccess;  // no such instantiation: the 16-row one serves every list
        using C = Row8Cfg<D, (G <= 8)>;
        const int narrow_grid = grid / Row8Cfg<D, false>::CTAS_PER_SM * C::CTAS_PER_SM;  // the same passes over more slots
        rpa_row_kernel_fp8_strided<D, G, (G <= 8)><<<narrow_grid, C::NW * 32, C::SMEM, stream>>>(a);
        return cudaGetLastError();
    }
    using C = Row8Cfg<D, false>;
    rpa_row_kernel_fp8_strided<D, G, false><<<grid, C::NW * 32, C::SMEM, stream>>>(a);
    return cudaGetLastError();
}

template <int D, int G, bool NARROW>
cudaError_t prepare_row8_one() {
    using C = Row8Cfg<D, NARROW>;
    cudaError_t e = cudaFuncSetAttribute(rpa_row_kernel_fp8<D, G, NARROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(rpa_row_kernel_fp8_strided<D, G, NARROW>, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM);
}

template <int D, int G>
cudaError_t prepare_row8() {
    if (G <= 8) {
        const cudaError_t e = prepare_row8_one<D, G, (G <= 8)>();
        if (e != cudaSuccess) return e;
    }
    return prepare_row8_one<D, G, false>();
}

#define RPA_DISPATCH_DG8(D_, G_, FN, ...)                                                  \
    do {                                                                                   \
        switch ((D_) * 100 + (G_)) {                                                       \
            case 6401: return FN<64, 1>(__VA_ARGS__);                                      \
            case 6402: return FN<64, 2>(__VA_ARGS__);                                      \
            case 6404: return FN<64, 4>(__VA_ARGS__);                                      \
            case 6408: return FN<64, 8>(__VA_ARGS__);                                      \
            case 6416: return FN<64, 16>(__VA_ARGS__);                                     \
            case 12801: return FN<128, 1>(__VA_ARGS__);                                    \
            case 12802: return FN<128, 2>(__VA_ARGS__);                                    \
            case 12804: return FN<128, 4>(__VA_ARGS__);                                    \
            case 12808: return FN<128, 8>(__VA_ARGS__);                                    \
            case 12816: return FN<128, 16>(__VA_ARGS__);                                   \
            case 25601: return FN<256, 1>(__VA_ARGS__);                                    \
            case 25602: return FN<256, 2>(__VA_ARGS__);                                    \
            case 25604: return FN<256, 4>(__VA_ARGS__);                                    \
            case 25608: return FN<256, 8>(__VA_ARGS__);                                    \
            case 25616: return FN<256, 16>(__VA_ARGS__);                                   \
        }                                                                                  \
    } while (0)

}  // namespace

int row_kernel_fp8_ctas_per_sm(int head_dim) {
    return head_dim == 64 ? Row8Cfg<64, false>::CTAS_PER_SM : head_dim == 128 ? Row8Cfg<128, false>::CTAS_PER_SM
                                                                               : Row8Cfg<256, false>::CTAS_PER_SM;
}

int row_kernel_fp8_narrow_ctas_per_sm(int head_dim) {
    return head_dim == 64 ? Row8Cfg<64, true>::CTAS_PER_SM : head_dim == 128 ? Row8Cfg<128, true>::CTAS_PER_SM
                                                                              : Row8Cfg<256, true>::CTAS_PER_SM;
}

cudaError_t row_kernel_fp8_prepare(int head_dim, int group) {
    RPA_DISPATCH_DG8(head_dim, group, prepare_row8);
    return cudaErrorInvalidValue;
}

cudaError_t launch_row_kernel_fp8_strided(const KernelArgs& a, int grid, bool narrow, cudaStream_t stream) {
    if (grid <= 0 || !a.dev_counts) return cudaErrorInvalidValue;
    RPA_DISPATCH_DG8(a.head_dim, a.h_q / a.h_kv, launch_row8_strided, a, grid, narrow, stream);
    return cudaErrorInvalidValue;
}

// Per-tensor quantisation of Q (Section 3.8): every element of the call's query rows becomes
// e4m3(float(q) * (1/q_scale)), the conversion K uses.  The pass writes the E4M3 VALUES as bf16 (each
// is exact in bf16) into a scratch tensor the attention kernels then read in place of q, with q_scale
// folded into the softmax scale, and the raw codes beside them.  `total_rows` bounds the rows when
// the host knows T; with a device-made plan the bound is cu_q_lens[num_seqs], read on the device.
__global__ void __launch_bounds__(256) rpa_quantise_q_kernel(const uint16_t* q, uint16_t* q_img, uint8_t* q_codes, int64_t total_rows,
                                                             const int32_t* cu_q_lens, int32_t num_seqs, int32_t row_elems,
                                                             float inv_q_scale, const uint32_t* status, int32_t check_status) {
    if (check_status && (*reinterpret_cast<const volatile uint32_t*>(status) & kStatusBadInput)) return;
    const int64_t rows = cu_q_lens ? (int64_t)cu_q_lens[num_seqs] : total_rows;
    const int64_t n16 = rows * row_elems / 16;  // (row_elems is a multiple of 64)
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x) {
        const uint4 codes = quantise16(q + i * 16, inv_q_scale);
        *reinterpret_cast<uint4*>(q_codes + i * 16) = codes;
        uint4 lo, hi;
        lo.x = e4m3x2_to_bf16x2(codes.x & 0xffffu);
        lo.y = e4m3x2_to_bf16x2(codes.x >> 16);
        lo.z = e4m3x2_to_bf16x2(codes.y & 0xffffu);
        lo.w = e4m3x2_to_bf16x2(codes.y >> 16);
        hi.x = e4m3x2_to_bf16x2(codes.z & 0xffffu);
        hi.y = e4m3x2_to_bf16x2(codes.z >> 16);
        hi.z = e4m3x2_to_bf16x2(codes.w & 0xffffu);
        hi.w = e4m3x2_to_bf16x2(codes.w >> 16);
        *reinterpret_cast<uint4*>(q_img + i * 16) = lo;
        *reinterpret_cast<uint4*>(q_img + i * 16 + 8) = hi;
    }
}

cudaError_t launch_quantise_q(const uint16_t* q, uint16_t* q_img, uint8_t* q_codes, int64_t total_rows, const int32_t* cu_q_lens,
                              int32_t num_seqs, int64_t max_rows, int32_t row_elems, float inv_q_scale, const uint32_t* status,
                              bool check_status, cudaStream_t stream) {
    const int64_t n16 = (cu_q_lens ? max_rows : total_rows) * row_elems / 16;
    if (n16 <= 0) return cudaSuccess;
    const int grid = (int)std::min<int64_t>((n16 + 255) / 256, 148 * 16);
    rpa_quantise_q_kernel<<<grid, 256, 0, stream>>>(q, q_img, q_codes, total_rows, cu_q_lens, num_seqs, row_elems, inv_q_scale, status,
                                                    check_status ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_row_kernel_fp8(const KernelArgs& a, cudaStream_t stream) {
    if (a.num_row_items <= 0) return cudaSuccess;
    RPA_DISPATCH_DG8(a.head_dim, a.h_q / a.h_kv, launch_row8, a, stream);
    return cudaErrorInvalidValue;
}

}  // namespace rpa
