// Tensor-core tile kernel, single-tile variant: one 128-row query tile per CTA with the score
// accumulator double-buffered in TMEM.
//
// Used where two query tiles do not fit the 512 TMEM columns: at d_k = 256 the output accumulator
// alone takes 256 columns.  The freed space holds a second score buffer instead, which changes the
// pipeline: the score product of block j+2 runs while the softmax warps work on block j+1 and the
// PV product of block j is still in flight, so the softmax never waits for its own tile's products
// (Algorithm 1's compute blocks, software-pipelined two deep).  Key blocks are BN positions
// (64 at d_k = 256) in a two-deep K ring and a two-deep V ring.  A single tile per CTA re-reads
// K/V from L2 twice as often per FLOP as the two-tile kernel and has one softmax group instead of
// two, so it is used only where two tiles cannot fit.
//
// Work item, key streams (cached context gathered page by page with TMA, then the batch's own new
// tokens from new_k/new_v), GQA row packing, masking, lazy rescale, fused cache update and bounded
// waits are the same as in rpa_tile_kernel.cu; an item covers 128/h_g tokens.
// Warp roles (256 threads): warp 0 TMA producer, warp 1 MMA issuer and TMEM owner, warps 2-3 fused
// cache update, warps 4-7 softmax (one query row per thread).
// TMEM: S[0], S[1] (BN columns each; P aliases the first BN/2 of its buffer), O (d_k columns) and
// the query tile itself (d_k/2 columns, bf16 pairs): the softmax threads copy their rows from the
// shared-memory tile into TMEM when an item starts, and the score products take Q as their TMEM
// operand.  A score product of 128 x BN x 16 then reads only its K slice from shared memory (2 KB at
// BN = 64) instead of 6 KB, which lets it run at the tensor pipe's pace: with Q in shared memory
// the 64-wide products were paced by the shared-memory port.
#include <cuda.h>
#include <cuda_bf16.h>

#include "rpa_fp8.cuh"
#include "rpa_kernels.h"
#include "rpa_ptx.cuh"
#include "rpa_sm100.cuh"
#include "rpa_tile_common.cuh"

namespace rpa {

using namespace sm100;

namespace {

constexpr int kT1Threads = 256;
constexpr uint32_t kT1TmemCols = 512;
constexpr float kT1RescaleThreshold = 8.f;  // log2 units

template <int D>
struct Tile1Cfg {
    static constexpr int BN = D == 256 ? 64 : 128;      // key positions per block
    static constexpr int NBLK = D / 64;                 // 64-element (128-byte) column blocks per row
    static constexpr int QBLK_BYTES = 128 * 128;        // one column block of the 128-row Q tile
    static constexpr int KBLK_BYTES = BN * 128;         // one column block of a K or V stage
    static constexpr int Q_BYTES = NBLK * QBLK_BYTES;
    static constexpr int KV_BYTES = NBLK * KBLK_BYTES;  // one K (or V) stage
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = Q_BYTES;
    static constexpr int OFF_V = OFF_K + 2 * KV_BYTES;
    static constexpr int OFF_UPD = OFF_V + 2 * KV_BYTES;  // staging of the fused cache update
    static constexpr int OFF_BAR = OFF_UPD + TileUpdate<D>::STAGE_BYTES;
    static_assert(Q_BYTES == 2 * KV_BYTES, "the query tile and the K ring swap roles");
    static constexpr int SMEM = OFF_BAR + kTileBarBlockBytes + 1024;  // + barriers and item slots + slack for 1024-byte alignment
    static_assert(SMEM <= 232448, "shared memory budget");
    static constexpr uint32_t TM_S0 = 0, TM_S1 = BN, TM_O = 2 * BN, TM_Q = 2 * BN + D;
    static_assert(2 * BN + D + D / 2 <= 512, "TMEM budget");
};

// S_FULL / P_READY: index = score buffer (block parity)
// O_DONE: index = block parity as well, so that a waiter always knows the previous completion of
// the barrier it waits on has happened (a parity wait can only tell apart one step)
// T1_Q: one barrier per query region, alive across items (see the region swap below); T1_NEXT: the
// next item's slot has been filled; T1_QT: the query tile has been copied into TMEM; T1_KCONV /
// T1_VCONV (FP8 cache): the stage's code bytes have been expanded to bf16
enum { T1_Q = 0, T1_KFULL = 2, T1_KEMPTY = 4, T1_VFULL = 6, T1_VEMPTY = 8, T1_SFULL = 10, T1_PREADY = 12, T1_ODONE = 14, T1_UPD = 16, T1_EPI = 18, T1_NEXT = 19, T1_QT = 20, T1_KCONV = 21, T1_VCONV = 23, T1_COUNT = 25 };
static_assert(8 * T1_COUNT + 24 <= 256, "barriers, abort flag, TMEM slot and progress fit below the item slots");

template <int D, int G, bool FP8>
__global__ void __launch_bounds__(kT1Threads, 1)
rpa_tile1_kernel(const KernelArgs a, const __grid_constant__ TileMaps maps) {
    using C = Tile1Cfg<D>;
    constexpr int BN = C::BN;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bars = smem_base + C::OFF_BAR;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_BAR + 8 * T1_COUNT);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_BAR + 8 * T1_COUNT + 8);
    // key blocks of the running item whose PV product has been issued (written by the MMA warp)
    volatile int* progress = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * T1_COUNT + 16);
    // two slots of RAW_INTS ints: the running item's list entry and lengths, and the next item's
    volatile int* item_slots = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 256);
    auto bar = [&](int slot) { return bars + 8u * slot; };

    // first of a programmatic pair: the kernel behind this one on the stream may start as soon as
    // every CTA of this one has got its SM (or has left)
    if (a.pdl_primary && threadIdx.x == 0) pdl_launch_dependents();
    if ((a.validated || a.dev_counts) && (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput)) return;  // inputs were rejected
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (a.dev_counts && (int)blockIdx.x >= a.dev_counts[kDevCountTileCtas]) {
        // device-planned step: the planner gave this kernel fewer CTAs than were launched
        if (tid == 0 && atomicAdd(a.tile_counters + 1, 1) == (int)gridDim.x - 1) {
            a.tile_counters[0] = 0;
            a.tile_counters[1] = 0;
        }
        return;
    }
    const int ps = a.page_size;
    if (tid == 0) *abort_flag = 0u;
    if (warp == 1) {
        tmem_alloc(smem_u32(tmem_slot), kT1TmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_s[2] = {tmem_base + C::TM_S0, tmem_base + C::TM_S1};
    const uint32_t tm_o = tmem_base + C::TM_O, tm_q = tmem_base + C::TM_Q;

    // With one CTA per item the item is the block index; with fewer CTAs than items the CTA is
    // persistent and draws items from the device-wide counter until the list is exhausted.
    const int n_items = tile_item_count(a);
    const bool persistent = a.dev_counts != nullptr || (int)gridDim.x < n_items;
    if (tid == 0) {
        mbar_init(bar(T1_Q + 0), 1);
        mbar_init(bar(T1_Q + 1), 1);
        fence_mbar_init();
    }
    int q_prefetched_for = -1;  // producer: the iteration whose query tile is already on its way
    for (int iter = 0;; ++iter) {
        tc_fence_before();
        __syncthreads();  // everyone is done with the previous item
        if (*abort_flag) break;
        volatile int* slot = item_slots + (iter & 1) * RAW_INTS;
        if (warp == 0 && iter == 0) draw_and_fetch_tile(a, persistent, (int)blockIdx.x, slot, lane);
        if (tid == 0) {
            *progress = 0;
            mbar_init(bar(T1_EPI), 128);
            mbar_init(bar(T1_NEXT), 1);
            mbar_init(bar(T1_QT), 128);
            for (int s = 0; s < 2; ++s) {
                mbar_init(bar(T1_KFULL + s), 1);
                mbar_init(bar(T1_KEMPTY + s), 1);
                mbar_init(bar(T1_VFULL + s), 1);
                mbar_init(bar(T1_VEMPTY + s), 1);
                mbar_init(bar(T1_SFULL + s), 1);
                mbar_init(bar(T1_PREADY + s), 128);
                mbar_init(bar(T1_ODONE + s), 1);
                mbar_init(bar(T1_UPD + s), 1);
                mbar_init(bar(T1_KCONV + s), 64);
                mbar_init(bar(T1_VCONV + s), 64);
            }
            fence_mbar_init();
        }
        __syncthreads();
        tc_fence_after();
        if (slot[RAW_ITEM] >= n_items) break;
        const TileCtx it = tile_ctx_from_raw(a, slot, BN);
      if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;  // (bounds-checked build: every thread of the CTA takes this exit together)
        const int h = it.h, cu = it.cu, q_r = it.q_r, L = it.L, c = it.c;
        const int n_ctx_blocks = it.n_ctx_blocks, n_new_visible = it.n_new_visible, n_blocks = it.n_blocks;
        const int32_t* pt_row = it.pt_row;
        // The query tile and the K ring are two regions of the same size that swap roles from item to
        // item: the K ring is idle from an item's last score product on, so the producer loads the
        // next item's query tile into it while the last PV products and the epilogue run.
        const uint32_t q_off = (iter & 1) ? C::OFF_K : C::OFF_Q, k_off = (iter & 1) ? C::OFF_Q : C::OFF_K;

        if (warp == 0) {
            // ================================ TMA producer ================================
            auto load_q = [&](uint32_t region, uint32_t q_bar, int head, int tok_row) {  // one thread
                mbar_arrive_expect_tx(q_bar, C::Q_BYTES);
#pragma unroll
                for (int b = 0; b < C::NBLK; ++b) tma_load_3d(region + b * C::QBLK_BYTES, &maps.q, b * 64, head * G, tok_row, q_bar);
            };
            if (lane == 0) {
                prefetch_tmap(&maps.q);
                prefetch_tmap(&maps.out);
                prefetch_tmap(&maps.cache);
                prefetch_tmap(&maps.new_k);
                prefetch_tmap(&maps.new_v);
                if (q_prefetched_for != iter)  // the CTA's first item (later ones were loaded during their predecessor)
                    load_q(smem_base + q_off, bar(T1_Q + (iter & 1)), h, cu + it.q_tok0);
            }
            const int box_rows = page_box_rows(ps, BN);
            const int sub_blocks = BN / box_rows;
            bool ok = true;
            for (int j = 0; j < n_blocks && ok; ++j) {
                const bool ctx = j < n_ctx_blocks;
                int page = 0, slot0 = 0;
                bool sub_valid = false;
                int n_sub_valid = 0;
                if (ctx) {
                    const int pos = j * BN + lane * box_rows;
                    sub_valid = lane < sub_blocks && pos < c;
                    if (sub_valid) {
                        page = debug_read_page(a, pt_row[pos / ps]);
                        slot0 = pos % ps;
                    }
                    n_sub_valid = __popc(__ballot_sync(0xffffffffu, sub_valid));
                }
                const int new_row0 = cu + (j - n_ctx_blocks) * BN;
                const uint32_t bytes = ctx ? (uint32_t)n_sub_valid * box_rows * D * (FP8 ? 1 : 2) : (uint32_t)C::KV_BYTES;
#pragma unroll
                for (int kv = 0; kv < 2; ++kv) {  // 0: K stage, 1: V stage
                    const int st = j & 1;
                    const int full = (kv ? T1_VFULL : T1_KFULL) + st, empty = (kv ? T1_VEMPTY : T1_KEMPTY) + st;
                    if (j >= 2) ok = ok && mbar_wait(bar(empty), ((j >> 1) - 1) & 1, abort_flag, a.status, 0x50 + kv);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const uint32_t dst = smem_base + (kv ? (uint32_t)C::OFF_V : k_off) + st * C::KV_BYTES;
                    if (lane == 0) mbar_arrive_expect_tx(bar(full), bytes);
                    __syncwarp();
                    if (ctx) {
                        if (sub_valid) {
                            if constexpr (FP8) {
                                // raw code rows, 128 bytes per box, land in the upper half of the stage
#pragma unroll
                                for (int b = 0; b < C::NBLK / 2; ++b)
                                    tma_load_4d(dst + (C::NBLK / 2 + b) * C::KBLK_BYTES + lane * box_rows * 128, &maps.cache, b * 128,
                                                2 * h + kv, slot0, page, bar(full));
                            } else {
#pragma unroll
                                for (int b = 0; b < C::NBLK; ++b)
                                    tma_load_4d(dst + b * C::KBLK_BYTES + lane * box_rows * 128, &maps.cache, b * 64, 2 * h + kv,
                                                slot0, page, bar(full));
                            }
                        }
                    } else if (lane == 0) {
#pragma unroll
                        for (int b = 0; b < C::NBLK; ++b)
                            tma_load_3d(dst + b * C::KBLK_BYTES, kv ? &maps.new_v : &maps.new_k, b * 64, h, new_row0, bar(full));
                    }
                }
            }
            // the next item's query tile, into this item's K ring once its last score product has read it
            if (ok) ok = mbar_wait(bar(T1_NEXT), 0, abort_flag, a.status, 0x52);
            const volatile int* nxt = item_slots + ((iter + 1) & 1) * RAW_INTS;
            if (ok && nxt[RAW_ITEM] < n_items) {
#pragma unroll
                for (int st = 0; st < 2; ++st) {
                    const int uses = (n_blocks + 1 - st) >> 1;  // key blocks of this item that went through stage st
                    if (uses > 0) ok = ok && mbar_wait(bar(T1_KEMPTY + st), (uses - 1) & 1, abort_flag, a.status, 0x53);
                }
                ok = __all_sync(0xffffffffu, ok);
                if (ok) {
                    if (lane == 0) load_q(smem_base + k_off, bar(T1_Q + ((iter + 1) & 1)), nxt[RAW_HEAD], nxt[RAW_CU] + nxt[RAW_TOK0]);
                    q_prefetched_for = iter + 1;
                }
            }
        } else if (warp == 1) {
            // ================================ MMA issuer ================================
            // All 32 lanes stay on this path to the end of the item whatever the waits return (a wait
            // that gave up has set the abort flag, every later one returns at once, and the products
            // of an aborted item are never read): the elected issue needs the whole warp.
            constexpr uint32_t idesc_qk = instr_desc_bf16(128, BN, 0, 0);
            constexpr uint32_t idesc_pv = instr_desc_bf16(128, D, 0, 1);
            constexpr uint32_t desc_hi = smem_desc_sw128_hi(1024);
            const uint32_t k_lo = smem_desc_sw128_lo(smem_base + k_off, 16);
            const uint32_t v_lo = smem_desc_sw128_lo(smem_base + C::OFF_V, C::KBLK_BYTES);
            auto issue_qk = [&](int j) {  // S[j&1] = Q K(j)^T over d_k in steps of 16
                const uint32_t kl = k_lo + (j & 1) * (C::KV_BYTES >> 4);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {  // Q from TMEM: 8 columns (16 bf16) per step
                    const uint32_t k_off = ((ks / 4) * C::KBLK_BYTES + (ks % 4) * 32) >> 4;
                    umma_ts_warp(tm_s[j & 1], tm_q + ks * 8, make_desc(kl + k_off, desc_hi), idesc_qk, ks > 0);
                }
            };
            auto issue_pv = [&](int j) {  // O (+)= P(j) V(j) over BN positions in steps of 16
                const uint32_t vl = v_lo + (j & 1) * (C::KV_BYTES >> 4);
#pragma unroll
                for (int kk = 0; kk < BN / 16; ++kk)
                    umma_ts_warp(tm_o, tm_s[j & 1] + kk * 8, make_desc(vl + kk * (2048 >> 4), desc_hi), idesc_pv, !(j == 0 && kk == 0));
            };
            // barrier that says block j's K (or V) operand is in place: with an FP8 cache a context
            // block is ready once the converter warps have expanded it, not when its bytes land
            auto k_ready = [&](int j) { return bar((FP8 && j < n_ctx_blocks ? T1_KCONV : T1_KFULL) + (j & 1)); };
            auto v_ready = [&](int j) { return bar((FP8 && j < n_ctx_blocks ? T1_VCONV : T1_VFULL) + (j & 1)); };
            (void)mbar_wait(bar(T1_QT), 0, abort_flag, a.status, 0x60);  // the softmax threads have put Q into TMEM
            for (int j = 0; j < 2 && j < n_blocks; ++j) {  // the first two score products
                (void)mbar_wait(k_ready(j), 0, abort_flag, a.status, 0x61);
                tc_fence_after();
                // The whole (converged) warp runs the issue code and one elected lane issues: issued from
                // inside a one-lane branch, a product cost the issuing thread about 80 cycles (operands
                // moved one by one to where the instruction takes them), more than a 128 x 64 x 16
                // product takes to execute, and the issuing thread paced the kernel.
                issue_qk(j);
                tc_commit_warp(bar(T1_SFULL + j));
                tc_commit_warp(bar(T1_KEMPTY + j));
                __syncwarp();
            }
            for (int j = 0; j < n_blocks; ++j) {
                const int st = j & 1, ph = (j >> 1) & 1;
                (void)mbar_wait(v_ready(j), ph, abort_flag, a.status, 0x62);
                // rows of V past the block's valid positions may hold stale or foreign data: make
                // them finite (zero) so that masked probabilities (exactly 0) cannot produce NaN
                const bool ctx = j < n_ctx_blocks;
                const int n_valid = ctx ? min(BN, c - j * BN) : min(BN, n_new_visible - (j - n_ctx_blocks) * BN);
                if (n_valid < BN) {
                    uint8_t* v_s = smem + C::OFF_V + st * C::KV_BYTES;
                    for (int idx = lane; idx < (BN - n_valid) * C::NBLK * 8; idx += 32) {
                        const int r = n_valid + idx / (C::NBLK * 8), rem = idx % (C::NBLK * 8);
                        *reinterpret_cast<uint4*>(v_s + (rem / 8) * C::KBLK_BYTES + r * 128 + (rem % 8) * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                (void)mbar_wait(bar(T1_PREADY + st), ph, abort_flag, a.status, 0x63);
                tc_fence_after();
                issue_pv(j);
                tc_commit_warp(bar(T1_ODONE + st));
                tc_commit_warp(bar(T1_VEMPTY + st));
                if (lane == 0) *progress = j + 1;
                __syncwarp();
                if (j + 2 < n_blocks) {  // the score product two blocks ahead reuses this block's S buffer and K stage
                    (void)mbar_wait(k_ready(j + 2), ((j + 2) >> 1) & 1, abort_flag, a.status, 0x64);
                        tc_fence_after();
                    issue_qk(j + 2);
                    tc_commit_warp(bar(T1_SFULL + st));
                    tc_commit_warp(bar(T1_KEMPTY + st));
                    __syncwarp();
                }
            }
        } else if (warp < 4) {
            // ================================ fused cache update ================================
            // One warp draws the next item and fetches its list entry and lengths while this item
            // runs, so that the next turn of the loop starts without that chain of loads - but not
            // before the item is within four key blocks of its end: a CTA that reserved its next
            // item at the start of a long one would keep it from the CTAs that fall idle meanwhile.
            // A short item fetches first thing, a long one after its share of the update.
            auto fetch_next = [&]() {
                if (lane == 0) {
                    const long long t0 = clock64();
                    while (*progress < n_blocks - 4 && !*abort_flag && clock64() - t0 < 2000000000LL) __nanosleep(256);
                }
                __syncwarp();
                draw_and_fetch_tile(a, persistent, n_items, item_slots + ((iter + 1) & 1) * RAW_INTS, lane);
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(T1_NEXT));  // the producer may now load the next item's query tile
            };
            const bool fetch_early = n_blocks <= 4;
            if (warp == 3 && fetch_early) fetch_next();
            if constexpr (FP8) {
                // FP8 cache: the item's own tokens were quantised and stored by the pass that ran
                // before this kernel.  These two warps expand the context blocks instead: a thread
                // turns the raw rows of one position (128 code bytes each, in the upper half of the
                // stage) into the 64-column blocks of the bf16 operand layout, every E4M3 value
                // being exact in bf16.  Blocks 2b and 2b+1 come from raw row b; the last ones land
                // on raw rows this thread has read by then.
                const int t = tid - 64, box_rows = page_box_rows(ps, BN);
                bool okc = true;
                for (int j = 0; j < n_ctx_blocks && okc; ++j) {
                    const int st = j & 1, ph = (j >> 1) & 1;
                    const int rows = min(BN, (min(BN, c - j * BN) + box_rows - 1) / box_rows * box_rows);
#pragma unroll
                    for (int kv = 0; kv < 2; ++kv) {
                        okc = okc && mbar_wait(bar((kv ? T1_VFULL : T1_KFULL) + st), ph, abort_flag, a.status, 0x58 + kv);
                        if (!okc) break;
                        uint8_t* stage = smem + (kv ? (uint32_t)C::OFF_V : k_off) + st * C::KV_BYTES;
                        for (int r = t; r < rows; r += 64) {
#pragma unroll
                            for (int b = 0; b < C::NBLK / 2; ++b) {
                                const uint8_t* raw = stage + (C::NBLK / 2 + b) * C::KBLK_BYTES + r * 128;
                                uint4 w[8];
#pragma unroll
                                for (int cch = 0; cch < 8; ++cch) w[cch] = *reinterpret_cast<const uint4*>(raw + ((cch ^ (r & 7)) << 4));
#pragma unroll
                                for (int half = 0; half < 2; ++half) {
                                    uint8_t* dst_row = stage + (2 * b + half) * C::KBLK_BYTES + r * 128;
#pragma unroll
                                    for (int cch = 0; cch < 4; ++cch) {
                                        const uint4 x = w[half * 4 + cch];
                                        uint4 lo, hi;
                                        lo.x = e4m3x2_to_bf16x2(x.x & 0xffffu);
                                        lo.y = e4m3x2_to_bf16x2(x.x >> 16);
                                        lo.z = e4m3x2_to_bf16x2(x.y & 0xffffu);
                                        lo.w = e4m3x2_to_bf16x2(x.y >> 16);
                                        hi.x = e4m3x2_to_bf16x2(x.z & 0xffffu);
                                        hi.y = e4m3x2_to_bf16x2(x.z >> 16);
                                        hi.z = e4m3x2_to_bf16x2(x.w & 0xffffu);
                                        hi.w = e4m3x2_to_bf16x2(x.w >> 16);
                                        *reinterpret_cast<uint4*>(dst_row + (((2 * cch) ^ (r & 7)) << 4)) = lo;
                                        *reinterpret_cast<uint4*>(dst_row + (((2 * cch + 1) ^ (r & 7)) << 4)) = hi;
                                    }
                                }
                            }
                        }
                        fence_proxy_async_smem();
                        mbar_arrive(bar((kv ? T1_VCONV : T1_KCONV) + st));
                    }
                }
            } else if (!(a.ablation & kAblateUpdate) && (it.flags & kFlagWriteKv)) {
                tile_update_cache<D>(a, it, warp - 2, lane, smem_base + C::OFF_UPD);
            }
            if (warp == 3 && !fetch_early) fetch_next();
        } else {
            // ================================ softmax warps ================================
            const int quarter = warp & 3;         // TMEM lanes this warp may touch: 32*quarter ..
            const int row = quarter * 32 + lane;  // query row of this thread
            const int tok_in_tile = row / G, g = row % G;
            const int tok = it.q_tok0 + tok_in_tile;  // token index inside the sequence
            const bool row_valid = tok_in_tile < it.n_tok;
            const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
            const uint32_t o_addr = tm_o + lane_sel;
            const int lim = a.causal ? c + min(tok, q_r - 1) : L - 1;  // last visible key position of this row

            float m_ref = -INFINITY, l_sum = 0.f;
            // ---- this thread's query row: shared memory (128-byte swizzle, as the TMA wrote it) -> TMEM ----
            bool ok = mbar_wait(bar(T1_Q + (iter & 1)), (iter >> 1) & 1, abort_flag, a.status, 0x72);
            if (ok) {
                const uint32_t q_row = smem_base + q_off + row * 128;
#pragma unroll
                for (int b = 0; b < C::NBLK; ++b) {
                    uint32_t r32[32];
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        const uint4 v = ld_shared_v4(q_row + b * C::QBLK_BYTES + ((ch ^ (row & 7)) << 4));
                        r32[4 * ch + 0] = v.x;
                        r32[4 * ch + 1] = v.y;
                        r32[4 * ch + 2] = v.z;
                        r32[4 * ch + 3] = v.w;
                    }
                    tmem_st32(tm_q + lane_sel + b * 32, r32);
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(T1_QT));
            }
            for (int j = 0; j < n_blocks && ok; ++j) {
                const uint32_t s_addr = tm_s[j & 1] + lane_sel;
                ok = mbar_wait(bar(T1_SFULL + (j & 1)), (j >> 1) & 1, abort_flag, a.status, 0x70);
                if (!ok) break;
                tc_fence_after();
                float s[BN];
#pragma unroll
                for (int ch = 0; ch < BN / 32; ++ch) {
                    uint32_t r32[32];
                    tmem_ld32(s_addr + ch * 32, r32);
#pragma unroll
                    for (int i = 0; i < 32; ++i) s[ch * 32 + i] = __uint_as_float(r32[i]);
                }
                tc_wait_ld();
                // visible keys of this row inside the block: positions pos_base .. pos_base + n_vis - 1
                const bool ctx = j < n_ctx_blocks;
                const int pos_base = ctx ? j * BN : c + (j - n_ctx_blocks) * BN;
                const int n_valid = ctx ? min(BN, c - pos_base) : min(BN, c + n_new_visible - pos_base);
                const int n_vis = min(n_valid, lim - pos_base + 1);
                if (__any_sync(0xffffffffu, n_vis < BN)) {
#pragma unroll
                    for (int i = 0; i < BN; ++i)
                        if (i >= n_vis) s[i] = -INFINITY;
                }
                float mxp[8];  // independent partial maxima: no long dependency chain
#pragma unroll
                for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(s[i], s[i + 8]);
#pragma unroll
                for (int i = 16; i < BN; i += 16)
#pragma unroll
                    for (int k = 0; k < 8; ++k) mxp[k] = max3(mxp[k], s[i + k], s[i + k + 8]);
                const float mx = max3(max3(mxp[0], mxp[1], mxp[2]), max3(mxp[3], mxp[4], mxp[5]), fmaxf(mxp[6], mxp[7]));
                const float mx2 = mx * a.scale_log2;
                if (j == 0) {
                    m_ref = mx2;
                } else {
                    const bool grow = mx2 - m_ref > kT1RescaleThreshold;
                    if (__any_sync(0xffffffffu, grow)) {
                        // the previous PV product must have landed before O is touched
                        ok = mbar_wait(bar(T1_ODONE + ((j - 1) & 1)), ((j - 1) >> 1) & 1, abort_flag, a.status, 0x72);
                        if (!ok) break;
                        tc_fence_after();
                        const float f = grow ? fast_exp2(m_ref - mx2) : 1.f;
#pragma unroll
                        for (int ch = 0; ch < D / 32; ++ch) {
                            uint32_t r32[32];
                            tmem_ld32(o_addr + ch * 32, r32);
                            tc_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) r32[i] = __float_as_uint(__uint_as_float(r32[i]) * f);
                            tmem_st32(o_addr + ch * 32, r32);
                        }
                        l_sum *= f;
                        if (grow) m_ref = mx2;
                    }
                }
                const float m_use = m_ref == -INFINITY ? 0.f : m_ref;
                const float neg_m = -m_use;
                float lp[4] = {0.f, 0.f, 0.f, 0.f};  // independent partial sums
#pragma unroll
                for (int ch = 0; ch < BN / 64; ++ch) {
                    uint32_t p32[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const float p0 = fast_exp2(fmaf(s[ch * 64 + 2 * i], a.scale_log2, neg_m));
                        const float p1 = fast_exp2(fmaf(s[ch * 64 + 2 * i + 1], a.scale_log2, neg_m));
                        lp[i & 3] += p0 + p1;
                        p32[i] = pack_bf16x2(p0, p1);
                    }
                    tmem_st32(s_addr + ch * 32, p32);
                }
                l_sum += (lp[0] + lp[1]) + (lp[2] + lp[3]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(bar(T1_PREADY + (j & 1)));
            }
            // ---- epilogue: O / l -> bf16 -> out, once the last PV product has landed (products
            // complete in order, so that covers the one before it too) ----
            if (ok) ok = mbar_wait(bar(T1_ODONE + ((n_blocks - 1) & 1)), ((n_blocks - 1) >> 1) & 1, abort_flag, a.status, 0x75);
            if (ok) {
                tc_fence_after();
                const float inv = a.out_scale / l_sum;  // out_scale: 1, or v_scale of an FP8 cache
                if (it.n_tok == 128 / G) {
                    // A full tile goes out through shared memory: each thread parks its row in the
                    // Q buffer (free since the last score product completed) in the swizzled layout
                    // of the tensor map, and one thread stores the tile with the copy engine.
                    const uint32_t q_buf = smem_base + q_off;
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t r32[32];
                        tmem_ld32(o_addr + ch * 32, r32);
                        tc_wait_ld();
                        const uint32_t blk = q_buf + (ch / 2) * C::QBLK_BYTES + row * 128;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            const uint32_t dst_s = blk + ((((ch & 1) * 4 + i) ^ (row & 7)) << 4);
                            st_shared_v4(dst_s,
                                         pack_bf16x2(__uint_as_float(r32[8 * i + 0]) * inv, __uint_as_float(r32[8 * i + 1]) * inv),
                                         pack_bf16x2(__uint_as_float(r32[8 * i + 2]) * inv, __uint_as_float(r32[8 * i + 3]) * inv),
                                         pack_bf16x2(__uint_as_float(r32[8 * i + 4]) * inv, __uint_as_float(r32[8 * i + 5]) * inv),
                                         pack_bf16x2(__uint_as_float(r32[8 * i + 6]) * inv, __uint_as_float(r32[8 * i + 7]) * inv));
                        }
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(bar(T1_EPI));
                    if (row == 0) {
                        if (mbar_wait(bar(T1_EPI), 0, abort_flag, a.status, 0x76)) {
#pragma unroll
                            for (int b = 0; b < C::NBLK; ++b)
                                tma_store_3d(&maps.out, q_buf + b * C::QBLK_BYTES, b * 64, h * G, cu + it.q_tok0);
                            bulk_commit();
                            bulk_wait_read();  // the Q buffer may be overwritten by the next item's load
                        }
                    }
                } else {
                    uint16_t* dst = a.out + (((int64_t)cu + tok) * a.h_q + h * G + g) * D;
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t r32[32];
                        tmem_ld32(o_addr + ch * 32, r32);
                        tc_wait_ld();
                        if (row_valid) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint4 v;
                                v.x = pack_bf16x2(__uint_as_float(r32[8 * i + 0]) * inv, __uint_as_float(r32[8 * i + 1]) * inv);
                                v.y = pack_bf16x2(__uint_as_float(r32[8 * i + 2]) * inv, __uint_as_float(r32[8 * i + 3]) * inv);
                                v.z = pack_bf16x2(__uint_as_float(r32[8 * i + 4]) * inv, __uint_as_float(r32[8 * i + 5]) * inv);
                                v.w = pack_bf16x2(__uint_as_float(r32[8 * i + 6]) * inv, __uint_as_float(r32[8 * i + 7]) * inv);
                                *reinterpret_cast<uint4*>(dst + ch * 32 + i * 8) = v;
                            }
                        }
                    }
                }
            }
        }
    }
    // ---- teardown: everyone arrives, then the allocating warp frees TMEM ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kT1TmemCols);
    }
    if (tid == 0) {  // the last CTA to leave resets the counters for the next launch
        __threadfence();
        if (atomicAdd(a.tile_counters + 1, 1) == (int)gridDim.x - 1) {
            a.tile_counters[0] = 0;
            a.tile_counters[1] = 0;
        }
    }
}

template <int D, int G>
cudaError_t launch_tile1(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    TileMaps maps;
    if (!cached_tile_maps(cache, a, token_rows, D, G, 128 / G, Tile1Cfg<D>::BN, &maps)) return cudaErrorInvalidValue;
    const int grid = a.dev_counts ? a.num_tile_ctas : a.num_tile_ctas > 0 && a.num_tile_ctas < a.num_tile_items ? a.num_tile_ctas : a.num_tile_items;
    if (a.kv_fp8) {  // the quantising pass first: cache update of the items' own tokens, bf16 copies of their codes
        if (cudaError_t e = launch_quantise_new<D>(a, stream); e != cudaSuccess) return e;
        rpa_tile1_kernel<D, G, true><<<grid, kT1Threads, Tile1Cfg<D>::SMEM, stream>>>(a, maps);
    } else {
        rpa_tile1_kernel<D, G, false><<<grid, kT1Threads, Tile1Cfg<D>::SMEM, stream>>>(a, maps);
    }
    return cudaGetLastError();
}

template <int D, int G>
cudaError_t prepare_tile1() {
    cudaError_t e = cudaFuncSetAttribute(rpa_tile1_kernel<D, G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile1Cfg<D>::SMEM);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(rpa_tile1_kernel<D, G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Tile1Cfg<D>::SMEM);
}

#define RPA_TILE1_DISPATCH(D_, G_, FN, ...)                     \
    do {                                                        \
        if ((D_) == 256) {                                      \
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

bool tile1_kernel_supported(int head_dim, int group) {
    return head_dim == 256 && (group == 1 || group == 2 || group == 4 || group == 8 || group == 16);
}

cudaError_t tile1_kernel_prepare(int head_dim, int group) {
    RPA_TILE1_DISPATCH(head_dim, group, prepare_tile1);
    return cudaErrorInvalidValue;
}

cudaError_t launch_tile1_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    if (a.num_tile_items <= 0 && !a.dev_counts) return cudaSuccess;
    RPA_TILE1_DISPATCH(a.head_dim, a.h_q / a.h_kv, launch_tile1, a, token_rows, cache, stream);
    return cudaErrorInvalidValue;
}

}  // namespace rpa
