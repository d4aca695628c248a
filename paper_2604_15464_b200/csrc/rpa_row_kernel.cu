// Split-KV row kernel: decode and short-query attention with the fused cache update.
//
// One CTA serves one RowItem: up to 16 query rows (n_tok consecutive new tokens x the h_g query
// heads that share one KV head -- the paper's GQA packing of C_q into (c_q*h_g, d_k), Section
// 3.1.2) against KV positions [kv_begin, kv_end).  The path is HBM-bound (Section 4.1.2: decode
// time is the K/V fetch), so the design goal is bytes in flight: every warp owns a private ring of
// 16-position K/V stages filled by 16-byte cp.async copies, one fully coalesced 2*d_k*2-byte slot
// read per warp instruction, with the page id of each stage prefetched 32 stages ahead.  Cached
// positions (< c_r) come from the paged cache through the page table; positions of the batch's own
// new tokens come from new_k/new_v, so no CTA ever reads a slot another CTA writes in this call.
// The score and PV products use warp-level bf16 MMAs with fp32 accumulation on the 16-row tile;
// softmax follows Algorithm 1's (m, l) recurrences in the log2 domain.  Warps of a CTA take
// alternating stages of the item's KV range and merge their (m, l, O) states through shared
// memory; items whose KV range was split write an unnormalised partial, and the CTA that delivers
// a group's last partial (an atomic ticket per group) merges the group and writes the output.
//
// The cache update of Algorithm 1 ("Update U_kv") is done by the item flagged kFlagWriteKv: it
// copies its tokens' K and V rows into their cache slots with 16-byte moves before its main loop.
#include <cuda_bf16.h>

#include "rpa_kernels.h"
#include "rpa_ptx.cuh"
#include "rpa_row_common.cuh"

namespace rpa {

namespace {

template <int D>
struct RowCfg {
    static constexpr int NW = 4;                       // warps per CTA
    static constexpr int STAGES = D == 64 ? 4 : 3;     // ring depth per warp
    static constexpr int ROWB = D * 2;                 // bytes of one K (or V) row
    static constexpr int HALF = kKvTile * ROWB;        // bytes of the K part of a stage
    static constexpr int STAGE = 2 * HALF;
    static constexpr int CPR = D / 8;                  // 16-byte chunks per K (or V) row
    static constexpr int CPP = 2 * CPR;                // chunks per position (K then V)
    static constexpr int LOAD_ITERS = kKvTile * CPP / 32;
    static constexpr int QBYTES = kRowTileRows * ROWB;
    static constexpr int OSTRIDE = D + 8;              // floats per row of the merge scratch
    static constexpr int SMEM = QBYTES + NW * STAGES * STAGE;
    static constexpr int CTAS_PER_SM = D == 64 ? 3 : D == 128 ? 2 : 1;
    static constexpr bool Q_IN_REGS = D <= 128;        // d_k = 256: the accumulator alone takes 128 registers
    static_assert(STAGES * STAGE >= kRowTileRows * OSTRIDE * 4 + kRowTileRows * 8, "merge scratch fits the ring");
};

// One row item, start to finish, by the whole CTA.
template <int D, int G>
__device__ __forceinline__ void row_item(const KernelArgs& a, int item_index, uint8_t* smem) {
    using C = RowCfg<D>;
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
    const int64_t slot_elems = (int64_t)2 * a.h_kv * D;  // elements between consecutive cache slots
    const int64_t tok0 = (int64_t)cu + it.q_tok0;
    if (!debug_rows_ok(a, tok0, it.n_tok)) return;  // (bounds-checked build only)

    // ---- this warp's share of the KV tiles ----
    const int t_begin = it.kv_begin / kKvTile;
    const int t_end = (it.kv_end + kKvTile - 1) / kKvTile;
    const int n_my = t_end - t_begin - warp > 0 ? (t_end - t_begin - warp + NW - 1) / NW : 0;
    const uint32_t ring = smem_u32(smem) + C::QBYTES + warp * STAGES * C::STAGE;
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
            const uint32_t stage = ring + (kl % STAGES) * C::STAGE;
            if (!debug_stage_ok(a, kl % STAGES, STAGES)) return;
            if (pos0 + kKvTile <= fast_end) {
                const uint16_t* base = a.kv_cache + ((int64_t)page * ps + pos0 % ps) * slot_elems + (int64_t)2 * h * D;
#pragma unroll
                for (int i = 0; i < C::LOAD_ITERS; ++i) {
                    const int ci = i * 32 + lane;
                    const int r = ci / CPP, cc = ci % CPP;
                    const int is_v = cc >= CPR, ch = cc - is_v * CPR;
                    cp_async_16(stage + is_v * C::HALF + r * ROWB + ((ch ^ (r & 7)) << 4), base + r * slot_elems + cc * 8, 16);
                }
            } else {
#pragma unroll
                for (int i = 0; i < C::LOAD_ITERS; ++i) {
                    const int ci = i * 32 + lane;
                    const int r = ci / CPP, cc = ci % CPP;
                    const int is_v = cc >= CPR, ch = cc - is_v * CPR;
                    const int p = pos0 + r;
                    const uint16_t* src = a.kv_cache;
                    uint32_t bytes = 16;
                    if (p >= it.kv_end) {
                        bytes = 0;  // zero-fill: masked scores, and finite V rows for the PV product
                    } else if (p < c) {
                        const int pg = debug_read_page(a, pt_row[p / ps]);
                        src = a.kv_cache + ((int64_t)pg * ps + p % ps) * slot_elems + (int64_t)2 * h * D + cc * 8;
                    } else {
                        src = (is_v ? a.new_v : a.new_k) + (((int64_t)cu + (p - c)) * a.h_kv + h) * D + ch * 8;
                    }
                    cp_async_16(stage + is_v * C::HALF + r * ROWB + ((ch ^ (r & 7)) << 4), src, bytes);
                }
            }
        }
        cp_async_commit();
    };
    // The first stages go out before anything else of the item: the cache update and the Q tile below
    // wait on global loads of their own, and the K/V stream should not queue behind them.
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) load_tile(s);

    // ---- fused cache update: K and V rows of this item's tokens, 16 bytes per thread and step ----
    if ((it.flags & kFlagWriteKv) && !(a.ablation & kAblateUpdate)) {
        for (int idx = tid; idx < it.n_tok * CPP; idx += NTHREADS) {
            const int j = idx / CPP, cc = idx % CPP;
            const int pos = c + it.q_tok0 + j;
            const int page = pt_row[pos / ps];
            if (!debug_write_page_ok(a, page)) continue;
            uint16_t* dst = a.kv_cache + ((int64_t)page * ps + pos % ps) * slot_elems + (int64_t)2 * h * D + cc * 8;
            const uint16_t* src = (cc < CPR ? a.new_k : a.new_v) + ((tok0 + j) * a.h_kv + h) * D + (cc % CPR) * 8;
            *reinterpret_cast<uint4*>(dst) = ld_global_nc_v4(src);
        }
    }

    // ---- Q tile: row rho = token rho / G, grouped head rho % G; rows past n_tok are zero ----
    uint8_t* q_s = smem;
    for (int idx = tid; idx < kRowTileRows * CPR; idx += NTHREADS) {
        const int row = idx / CPR, ch = idx % CPR;
        const int j = row / G, g = row % G;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (j < it.n_tok) v = ld_global_nc_v4(a.q + ((tok0 + j) * a.h_q + h * G + g) * D + ch * 8);
        *reinterpret_cast<uint4*>(q_s + row * ROWB + ((ch ^ (row & 7)) << 4)) = v;
    }
    __syncthreads();
    // Q fragments of all d_k/16 steps stay in registers when they fit; otherwise they are re-read
    // from shared memory per step (the Q tile is never overwritten).
    uint32_t qf[C::Q_IN_REGS ? D / 16 : 1][4];
    const int q_mi = lane >> 3, q_r8 = ((q_mi & 1) << 3) + (lane & 7);
    const uint32_t q_frag_base = smem_u32(q_s) + q_r8 * ROWB;
    if (C::Q_IN_REGS) {
#pragma unroll
        for (int ks = 0; ks < (C::Q_IN_REGS ? D / 16 : 1); ++ks)
            ldmatrix_x4(qf[ks], q_frag_base + (((ks * 2 + (q_mi >> 1)) ^ (q_r8 & 7)) << 4));
    }


    // per-thread softmax state for rows rho0 = lane/4 and rho0 + 8
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    float o[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

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
            const int mi = lane >> 3, r = ((mi >> 1) << 3) + (lane & 7);
            const uint32_t base = k_s + r * ROWB;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t b[4];
                ldmatrix_x4(b, base + (((ks * 2 + (mi & 1)) ^ (r & 7)) << 4));
                if (C::Q_IN_REGS) {
                    mma_bf16_16816(s[0], qf[C::Q_IN_REGS ? ks : 0], b[0], b[1]);
                    mma_bf16_16816(s[1], qf[C::Q_IN_REGS ? ks : 0], b[2], b[3]);
                } else {
                    uint32_t qk[4];
                    ldmatrix_x4(qk, q_frag_base + (((ks * 2 + (q_mi >> 1)) ^ (q_r8 & 7)) << 4));
                    mma_bf16_16816(s[0], qk, b[0], b[1]);
                    mma_bf16_16816(s[1], qk, b[2], b[3]);
                }
            }
        }
        const bool need_mask = pos0 + kKvTile > unmasked_end;
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
        pf[0] = pack_bf16x2(s[0][0], s[0][1]);
        pf[1] = pack_bf16x2(s[0][2], s[0][3]);
        pf[2] = pack_bf16x2(s[1][0], s[1][1]);
        pf[3] = pack_bf16x2(s[1][2], s[1][3]);
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
            for (int nd = 0; nd < D / 16; ++nd) {
                uint32_t b[4];
                ldmatrix_x4_trans(b, base + (((nd * 2 + (mi >> 1)) ^ (r & 7)) << 4));
#pragma unroll
                for (int q2 = 0; q2 < 2; ++q2) mma_bf16_16816(o[2 * nd + q2], pf, b[2 * q2], b[2 * q2 + 1]);
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
    float* o_s = reinterpret_cast<float*>(smem + C::QBYTES + warp * STAGES * C::STAGE);
    float* ml_s = o_s + kRowTileRows * C::OSTRIDE;
    {
        const int r0 = lane >> 2, col = 2 * (lane & 3);
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
            *reinterpret_cast<float2*>(o_s + r0 * C::OSTRIDE + n * 8 + col) = make_float2(o[n][0], o[n][1]);
            *reinterpret_cast<float2*>(o_s + (r0 + 8) * C::OSTRIDE + n * 8 + col) = make_float2(o[n][2], o[n][3]);
        }
        if ((lane & 3) == 0) {
            ml_s[r0] = m_run[0];
            ml_s[r0 + 8] = m_run[1];
            ml_s[16 + r0] = l_run[0];
            ml_s[16 + r0 + 8] = l_run[1];
        }
    }
    __syncthreads();
    constexpr int WARP_FLOATS = STAGES * C::STAGE / 4;
    const float* o_all = reinterpret_cast<const float*>(smem + C::QBYTES);
    for (int idx = tid; idx < kRowTileRows * (D / 4); idx += NTHREADS) {
        const int row = idx / (D / 4), c4 = idx % (D / 4);
        const int j = row / G, g = row % G;
        if (j >= it.n_tok) continue;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, o_all[w * WARP_FLOATS + kRowTileRows * C::OSTRIDE + row]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float lsum = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float* base = o_all + w * WARP_FLOATS;
            const float mw = base[kRowTileRows * C::OSTRIDE + row];
            const float f = mw == -INFINITY ? 0.f : fast_exp2(mw - M);
            const float4 v = *reinterpret_cast<const float4*>(base + row * C::OSTRIDE + c4 * 4);
            acc.x += f * v.x;
            acc.y += f * v.y;
            acc.z += f * v.z;
            acc.w += f * v.w;
            lsum += f * base[kRowTileRows * C::OSTRIDE + 16 + row];
        }
        if (it.partial < 0) {
            const float inv = 1.f / lsum;
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
        __threadfence();  // this thread's partial rows are visible device-wide before the ticket is taken
        __syncthreads();
        if (tid == 0) {
            const int ticket = atomicAdd(a.group_counters + group, 1);
            s_last = ticket == a.groups[group].n_partials - 1;
            if (s_last) a.group_counters[group] = 0;  // ready for the next call
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            const CombineGroup gr = a.groups[group];
            combine_group<D>(a, gr, tid, NTHREADS);
        }
    }
}

template <int D, int G>
__global__ void __launch_bounds__(RowCfg<D>::NW * 32, RowCfg<D>::CTAS_PER_SM) rpa_row_kernel(const KernelArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    if (a.validated && (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput)) return;  // inputs were rejected
    row_item<D, G>(a, blockIdx.x, smem);
}

// The same items from a list whose length only the device knows (planned by rpa_plan_kernel in the
// same step): a fixed grid, CTA b takes items b, b + grid, ...  The list is sorted longest first,
// so the stride deals every CTA a similar mix.
template <int D, int G>
__global__ void __launch_bounds__(RowCfg<D>::NW * 32, RowCfg<D>::CTAS_PER_SM) rpa_row_kernel_strided(const KernelArgs a) {
    extern __shared__ __align__(128) uint8_t smem[];
    if (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput) {  // the planner rejected the lengths
        if (a.pdl_secondary && threadIdx.x == 0) pdl_wait();  // (every CTA comes this way: nothing to make room for)
        return;
    }
    const int n = a.dev_counts[kDevCountRows];
    // the list is sorted longest first: dealing it back and forth (CTA b takes b, 2G-1-b, 2G+b, ...)
    // pairs the longest items of one pass with the shortest of the next
    const int G_ = (int)gridDim.x, b = (int)blockIdx.x;
    for (int w = 0; w * G_ < n; ++w) {
        const int i = (w & 1) ? (w + 1) * G_ - 1 - b : w * G_ + b;
        if (i >= n) continue;
        row_item<D, G>(a, i, smem);
        __syncthreads();  // the next item reuses the shared memory
    }
    // Launched as the programmatic dependent of the tile kernel: this kernel must not be seen as
    // complete before that one is (what follows on the stream relies on both).  The last CTA to
    // finish waits for it; the others leave and make room for the CTAs still to come.
    if (a.pdl_secondary && threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(a.tile_counters + 2, 1) == (int)gridDim.x - 1) {
            a.tile_counters[2] = 0;  // zero again for the next launch
            pdl_wait();
        }
    }
}

// Stand-alone combine, one CTA per group (used when the row kernel is not asked to combine itself).
template <int D>
__global__ void __launch_bounds__(128) rpa_combine_kernel(const KernelArgs a) {
    const CombineGroup gr = a.groups[blockIdx.x];
    combine_group<D>(a, gr, threadIdx.x, blockDim.x);
}

// One thread per sequence: the device copy of its lengths must match the plan, and every page it
// maps must lie inside the pool.  Runs before the attention kernels when validation is switched on.
__global__ void rpa_validate_kernel(const KernelArgs a, int num_seqs, const int32_t* plan_kv_lens) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= num_seqs) return;
    const int L = a.kv_lens[r];
    bool bad = L != plan_kv_lens[r] || a.cu_q_lens[r + 1] < a.cu_q_lens[r];
    if (!bad) {
        const int pages = (L + a.page_size - 1) / a.page_size;
        const int32_t* row = a.page_table + (int64_t)r * a.max_pages_per_seq;
        for (int p = 0; p < pages; ++p) {
            const int id = row[p];
            if (id < 0 || id >= a.num_pages) bad = true;
        }
    }
    if (bad) atomicOr(a.status, kStatusBadInput | (uint32_t)(r & 0xFFFFF));
}

template <int D, int G>
cudaError_t launch_row(const KernelArgs& a, cudaStream_t stream) {
    rpa_row_kernel<D, G><<<a.num_row_items, RowCfg<D>::NW * 32, RowCfg<D>::SMEM, stream>>>(a);
    return cudaGetLastError();
}

template <int D, int G>
cudaError_t launch_row_strided(const KernelArgs& a, int grid, cudaStream_t stream) {
    if (!a.pdl_secondary) {
        rpa_row_kernel_strided<D, G><<<grid, RowCfg<D>::NW * 32, RowCfg<D>::SMEM, stream>>>(a);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(RowCfg<D>::NW * 32);
    cfg.dynamicSmemBytes = RowCfg<D>::SMEM;
    cfg.stream = stream;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rpa_row_kernel_strided<D, G>, a);
}

template <int D, int G>
cudaError_t prepare_row() {
    cudaError_t e = cudaFuncSetAttribute(rpa_row_kernel<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, RowCfg<D>::SMEM);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(rpa_row_kernel_strided<D, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, RowCfg<D>::SMEM);
}

#define RPA_DISPATCH_DG(D_, G_, FN, ...)                        \
    do {                                                        \
        if ((D_) == 128) {                                      \
            switch (G_) {                                       \
                case 1: return FN<128, 1>(__VA_ARGS__);         \
                case 2: return FN<128, 2>(__VA_ARGS__);         \
                case 4: return FN<128, 4>(__VA_ARGS__);         \
                case 8: return FN<128, 8>(__VA_ARGS__);         \
                case 16: return FN<128, 16>(__VA_ARGS__);       \
            }                                                   \
        } else if ((D_) == 64) {                                \
            switch (G_) {                                       \
                case 1: return FN<64, 1>(__VA_ARGS__);          \
                case 2: return FN<64, 2>(__VA_ARGS__);          \
                case 4: return FN<64, 4>(__VA_ARGS__);          \
                case 8: return FN<64, 8>(__VA_ARGS__);          \
                case 16: return FN<64, 16>(__VA_ARGS__);        \
            }                                                   \
        } else if ((D_) == 256) {                               \
            switch (G_) {                                       \
                case 1: return FN<256, 1>(__VA_ARGS__);         \
                case 2: return FN<256, 2>(__VA_ARGS__);         \
                case 4: return FN<256, 4>(__VA_ARGS__);         \
                case 8: return FN<256, 8>(__VA_ARGS__);         \
                case 16: return FN<256, 16>(__VA_ARGS__);       \
            }                                                   \
        }                                                       \
    } while (0)

}  // namespace

bool row_kernel_supported(int head_dim, int group) {
    return (head_dim == 64 || head_dim == 128 || head_dim == 256) &&
           (group == 1 || group == 2 || group == 4 || group == 8 || group == 16);
}

int row_kernel_ctas_per_sm(int head_dim, int) {
    return head_dim == 64 ? RowCfg<64>::CTAS_PER_SM : head_dim == 128 ? RowCfg<128>::CTAS_PER_SM : RowCfg<256>::CTAS_PER_SM;
}

cudaError_t row_kernel_prepare(int head_dim, int group) {
    RPA_DISPATCH_DG(head_dim, group, prepare_row);
    return cudaErrorInvalidValue;
}

cudaError_t launch_row_kernel(const KernelArgs& a, cudaStream_t stream) {
    if (a.num_row_items <= 0) return cudaSuccess;
    RPA_DISPATCH_DG(a.head_dim, a.h_q / a.h_kv, launch_row, a, stream);
    return cudaErrorInvalidValue;
}

cudaError_t launch_row_kernel_strided(const KernelArgs& a, int grid, cudaStream_t stream) {
    if (grid <= 0 || !a.dev_counts) return cudaErrorInvalidValue;
    RPA_DISPATCH_DG(a.head_dim, a.h_q / a.h_kv, launch_row_strided, a, grid, stream);
    return cudaErrorInvalidValue;
}

cudaError_t launch_validate_kernel(const KernelArgs& a, int32_t num_seqs, const int32_t* plan_kv_lens, cudaStream_t stream) {
    if (num_seqs <= 0) return cudaSuccess;
    rpa_validate_kernel<<<(num_seqs + 127) / 128, 128, 0, stream>>>(a, num_seqs, plan_kv_lens);
    return cudaGetLastError();
}

cudaError_t launch_combine_kernel(const KernelArgs& a, cudaStream_t stream) {
    if (a.num_groups <= 0 || a.group_counters != nullptr) return cudaSuccess;  // the row kernel combines itself
    if (a.head_dim == 128)
        rpa_combine_kernel<128><<<a.num_groups, 128, 0, stream>>>(a);
    else if (a.head_dim == 256)
        rpa_combine_kernel<256><<<a.num_groups, 128, 0, stream>>>(a);
    else
        rpa_combine_kernel<64><<<a.num_groups, 128, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace rpa
