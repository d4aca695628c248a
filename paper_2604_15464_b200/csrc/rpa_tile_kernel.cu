// Tensor-core tile kernel: prefill and chunked-prefill attention on tcgen05 with TMEM accumulators.
//
// A CTA serves one TileItem at a time: up to 2*TQ consecutive new tokens of one sequence for one KV
// head, as two query tiles A and B of 128 rows each (row = token*h_g + grouped head: the paper's GQA
// packing of C_q into (c_q*h_g, d_k), Section 3.1.2, so the K/V operand is shared by all heads of
// the group).  The tiles walk the sequence's keys in blocks of 128 positions: first the cached
// context, gathered page by page through the page table, then the batch's own new tokens straight
// from new_k/new_v (so no CTA reads a cache slot that another CTA writes in this call).  Per block,
// S = Q K^T and O += P V run on tcgen05.mma (Algorithm 1's inner products), the (m, l) recurrences
// of Algorithm 1 run in the softmax warps on S read back from TMEM, and P returns to TMEM as bf16
// as the A operand of the PV product.
//
// Warp roles (384 threads, three warpgroups): warp 0 = TMA producer (Q once, K/V stages through
// mbarrier rings), warp 1 = MMA issuer (one elected thread) and owner of the TMEM allocation,
// warps 2-3 = fused cache update (FP8 cache: expansion of the context blocks' codes to bf16) and the
// fetch of the CTA's next item, warps 4-7 = softmax of tile A, warps 8-11 = softmax of tile B (one
// query row per thread; the first warpgroup hands most of its registers to the softmax
// warpgroups).  The issue order PV_A(j), QK_A(j+1), PV_B(j), QK_B(j+1) keeps the tensor pipe busy
// with one tile's products while the other tile's softmax runs.  O is rescaled only when a row's
// running maximum grows by more than 2^8 (exact after the final division by l).  TMEM: S_A, S_B
// (128 columns each, P aliases the first 64), O_A, O_B (d_k columns each).
//
// Items that fill one query tile only are not left with half the machine idle: with at least two
// key blocks the blocks are dealt to both accumulators (softmax group x takes blocks j = x mod 2 of
// tile A's rows) and merged in the epilogue.  A packed item holds several whole sequences without
// context; a row then sees the keys of its own sequence only (Section 5's remedy for short
// sequences).  CTAs are persistent: they draw items from a device-wide counter, the next item's
// list entry and lengths being fetched while the current one runs.
//
// The cache update of Algorithm 1 ("Update U_kv") for the item's own tokens goes through the
// bulk-copy engine.  Every wait is bounded; on expiry the CTA sets the device status word, drains
// and frees its TMEM.
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

constexpr int kBlockN = 128;       // KV positions per block
constexpr int kTileThreads = 384;  // 12 warps = 3 warpgroups
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;  // log2 units

template <int D>
struct TileCfg {
    static constexpr int NBLK = D / 64;             // 64-element (128-byte) column blocks per row
    static constexpr int BLK_BYTES = 128 * 128;     // one column block of a 128-row tile
    static constexpr int TILE_BYTES = NBLK * BLK_BYTES;
    static constexpr int KS = 2, VS = 2;            // K and V ring depths
    static constexpr int OFF_QA = 0;
    static constexpr int OFF_K = 2 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + KS * TILE_BYTES;
    static constexpr int OFF_UPD = OFF_V + VS * TILE_BYTES;  // staging of the fused cache update
    static constexpr int OFF_BAR = OFF_UPD + TileUpdate<D>::STAGE_BYTES;
    static constexpr int SMEM = OFF_BAR + kTileBarBlockBytes + 1024;  // + barriers and item slots + slack for 1024-byte alignment
    static_assert(SMEM <= 232448, "shared memory budget");
};

// barrier slots (8 bytes each) inside the barrier block
// BAR_Q has one barrier per Q region and lives across items (a Q load for the next item may be in
// flight while the others are re-initialised), and so does BAR_K0, on which an item's first key
// block arrives (bf16 cache: it is fetched while the item before still runs).  BAR_NEXT (the next
// item's slot has been filled: one phase per item) and BAR_UPD (the rows of an update warp's round
// have landed: armed and waited for by that warp alone, which keeps the phase) live across items as
// well: every barrier that does not have to start afresh saves the item 70 cycles.
enum { BAR_Q = 0, BAR_K0 = 2, BAR_NEXT = 4, BAR_UPD = 5, BAR_KFULL = 7, BAR_KEMPTY = 9, BAR_VFULL = 11, BAR_VEMPTY = 13, BAR_SFULL = 15, BAR_PREADY = 17, BAR_ODONE = 19, BAR_EPI = 21, BAR_KCONV = 23, BAR_VCONV = 25, BAR_COUNT = 27 };
static_assert(8 * BAR_COUNT + 24 <= 256, "barriers, abort flag, TMEM slot and progress fit below the item slots");


// Softmax of an item's only key block when at most half of it holds keys (a short prompt, a packed
// item of short prompts): the scores of 64 positions come out of TMEM, the probabilities of the
// other 64 are zero without an exponential being taken - with both tiles at once the exponentials
// of 256 rows are what such an item waits for.  A function of its own, not inlined: the same
// shortcut as a branch inside the kernel's softmax loop cost that loop 2 % on long prefill.
// n_vis: visible positions of this thread's row from the block's start; n_before: positions at the
// block's start that belong to earlier sequences of a packed item.  Returns the row's reference
// maximum (log2 units, scaled) and sum.
__device__ __noinline__ float2 softmax_half_block(uint32_t s_addr, int n_vis, int n_before, float scale_log2) {
    constexpr int HALF = kBlockN / 2;
    float s[HALF];
#pragma unroll
    for (int ch = 0; ch < HALF / 32; ++ch) {
        uint32_t r32[32];
        tmem_ld32(s_addr + ch * 32, r32);
#pragma unroll
        for (int i = 0; i < 32; ++i) s[ch * 32 + i] = __uint_as_float(r32[i]);
    }
    tc_wait_ld();
#pragma unroll
    for (int i = 0; i < HALF; ++i)
        if (i >= n_vis || i < n_before) s[i] = -INFINITY;
    float mxp[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(s[i], s[i + 8]);
#pragma unroll
    for (int i = 16; i < HALF; i += 16)
#pragma unroll
        for (int k = 0; k < 8; ++k) mxp[k] = max3(mxp[k], s[i + k], s[i + k + 8]);
    const float mx = fmaxf(max3(mxp[0], mxp[1], mxp[2]), max3(fmaxf(mxp[3], mxp[4]), max3(mxp[5], mxp[6], mxp[7]), -INFINITY));
    const float m_ref = mx * scale_log2;
    const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
    float lp[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    uint32_t p32[32];
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        float x0, x1;
        fma2_bcast(x0, x1, s[2 * i], s[2 * i + 1], scale_log2, neg_m);
        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
        add2(lp[2 * (i & 3)], lp[2 * (i & 3) + 1], p0, p1);
        p32[i] = pack_bf16x2(p0, p1);
    }
    tmem_st32(s_addr, p32);
#pragma unroll
    for (int i = 0; i < 32; ++i) p32[i] = 0u;
    tmem_st32(s_addr + 32, p32);
    tc_wait_st();
    return make_float2(m_ref, ((lp[0] + lp[1]) + (lp[2] + lp[3])) + ((lp[4] + lp[5]) + (lp[6] + lp[7])));
}

// QF8 (FP8 cache with a per-tensor scale for Q as well, d_k = 128): the score product runs as
// tcgen05.mma kind::f8f6f4 straight on code bytes - the query tile arrives as E4M3 codes (16 KB
// instead of 32), a key block as the raw code rows of the cache (or of the scratch copy of the
// batch's own K codes), 32 elements of d_k per instruction at twice the bf16 rate - so no key is
// expanded to bf16 any more; V keeps its bf16 expansion, P being bf16.
//
// SHORT: the instantiation for batches whose items all have one or two key blocks (bf16 cache): the
// cache update goes through the copy engine and an item whose only block is at most half full takes
// softmax_half_block.  Both are worth 10-20 % there and cost items that stream many key blocks
// 2-5 % by their mere presence in the kernel, hence two instantiations.
template <int D, int G, bool FP8, bool QF8, bool SHORT = false>
__global__ void __launch_bounds__(kTileThreads, 1)
rpa_tile_kernel(const KernelArgs a, const __grid_constant__ TileMaps maps) {
    static_assert(!QF8 || (FP8 && D == 128), "the FP8 score product is built for an FP8 cache and d_k = 128");
    using C = TileCfg<D>;
    constexpr int TQ = 128 / G;  // tokens per query tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bars = smem_base + C::OFF_BAR;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_BAR + 8 * BAR_COUNT);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_BAR + 8 * BAR_COUNT + 8);
    // key blocks of the running item whose PV product has been issued (written by the MMA warp)
    volatile int* progress = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * BAR_COUNT + 16);
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
        tmem_alloc(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_s[2] = {tmem_base, tmem_base + 128u};
    const uint32_t tm_o[2] = {tmem_base + 256u, tmem_base + 256u + D};

    // With one CTA per item the item is the block index.  With fewer CTAs than items the CTA is
    // persistent: it draws items from a device-wide counter (the list is sorted heaviest first
    // inside each KV head, so this is list scheduling) until the list is exhausted.  Between items
    // every role meets at two CTA-wide barriers around the draw and the re-initialisation of the
    // mbarriers.  The last CTA to leave resets the counters for the next launch.
    const int n_items = tile_item_count(a);
    const bool persistent = a.dev_counts != nullptr || (int)gridDim.x < n_items;
    if (tid == 0) {
        mbar_init(bar(BAR_Q + 0), 1);
        mbar_init(bar(BAR_Q + 1), 1);
        mbar_init(bar(BAR_K0 + 0), 1);
        mbar_init(bar(BAR_K0 + 1), 1);
        mbar_init(bar(BAR_NEXT), 1);
        mbar_init(bar(BAR_UPD + 0), 1);
        mbar_init(bar(BAR_UPD + 1), 1);
        fence_mbar_init();
    }
    // Every barrier but BAR_Q starts afresh with each item, between the two CTA-wide barriers, at the
    // hands of one thread, about 70 cycles a barrier.  Sharing the barriers out (one per lane of the
    // producer warp, or a few per warp) lost arrivals: lane 0 of the four warps of the first
    // warpgroup, with each barrier invalidated first, worked on short items and failed on long ones,
    // every other split failed everywhere.  Invalidating each barrier before it is initialised again
    // works with one thread too, but doubles the cost (2048 prompts of 64 tokens: 623 -> 683 us), so
    // the barriers are initialised over their old state, as they always were; every one of them has
    // completed its last phase and has no waiter by then.
    auto init_barriers = [&]() {
        for (int sl = BAR_KFULL; sl < BAR_COUNT; ++sl) {
            const bool converters = sl >= BAR_KCONV && sl < BAR_VCONV + 2;
            if (converters && !FP8) continue;  // (never used without an FP8 cache: still in their first phase)
            const bool all_rows = sl == BAR_PREADY || sl == BAR_PREADY + 1 || sl == BAR_EPI || sl == BAR_EPI + 1;
            mbar_init(bar(sl), all_rows ? 128 : converters ? 64 : 1);
        }
        fence_mbar_init();
    };
    if (warp < 4) {
      // first warpgroup: producer, MMA issuer, cache update; it needs few registers
      asm volatile("setmaxnreg.dec.sync.aligned.u32 56;\n");
      int q_prefetched_for = -1;  // producer: the iteration whose query tiles are already on their way
      int k0_prefetched_for = -1;  // producer: ... and whose first key block is
      bool out_stores_pending = false;  // producer: output tiles of the previous item may still be leaving the V ring
      uint32_t upd_parity = 0;  // update warps: running phase of the warp's own barrier
      for (int iter = 0;; ++iter) {
      tc_fence_before();
      __syncthreads();  // everyone is done with the previous item
      if (*abort_flag) break;
      volatile int* slot = item_slots + (iter & 1) * RAW_INTS;
      if (warp == 0 && iter == 0) draw_and_fetch_tile(a, persistent, (int)blockIdx.x, slot, lane);
      if (tid == 0) {
          init_barriers();
          *progress = 0;
      }
      __syncthreads();
      tc_fence_after();
      if (slot[RAW_ITEM] >= n_items) break;
      const TileCtx it = tile_ctx_from_raw(a, slot, kBlockN);
      if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;  // (bounds-checked build: every thread of the CTA takes this exit together)
      const int h = it.h, cu = it.cu, q_r = it.q_r, c = it.c;
      const int n_ctx_blocks = it.n_ctx_blocks, n_new_visible = it.n_new_visible, n_blocks = it.n_blocks;
      const int32_t* pt_row = it.pt_row;
      (void)q_r;
      // The query tiles and the K ring are two regions of the same size and layout that swap roles from
      // item to item: the K ring is idle from an item's last score product on, so the producer loads
      // the next item's query tiles into it while the last PV products and the epilogue run.
      const uint32_t q_off = (iter & 1) ? C::OFF_K : C::OFF_QA, k_off = (iter & 1) ? C::OFF_QA : C::OFF_K;
      if (warp == 0) {
        // ================================ TMA producer ================================
        const uint32_t q_region = smem_base + q_off, k_region = smem_base + k_off;
        auto load_q = [&](uint32_t region, uint32_t q_bar, int n_tok, int head, int tok_row) {  // one thread
            const int n_tiles = n_tok > TQ ? 2 : 1;  // a short item uses tile A only
            if (a.ablation & kAblateLoads) {  // bench switch: the barrier completes without data
                mbar_arrive(q_bar);
                return;
            }
            mbar_arrive_expect_tx(q_bar, n_tiles * (QF8 ? C::BLK_BYTES : C::TILE_BYTES));
            for (int x = 0; x < n_tiles; ++x) {
                if constexpr (QF8) {  // 128 rows of 128 code bytes
                    tma_load_3d(region + x * C::TILE_BYTES, &maps.q, 0, head * G, tok_row + x * TQ, q_bar);
                } else {
#pragma unroll
                    for (int b = 0; b < C::NBLK; ++b)
                        tma_load_3d(region + x * C::TILE_BYTES + b * C::BLK_BYTES, &maps.q, b * 64, head * G, tok_row + x * TQ, q_bar);
                }
            }
        };
        if (lane == 0) {
            if (iter == 0) {
                prefetch_tmap(&maps.q);
                prefetch_tmap(&maps.out);
                prefetch_tmap(&maps.cache);
                prefetch_tmap(&maps.new_k);
                prefetch_tmap(&maps.new_v);
            }
            if (q_prefetched_for != iter)  // the CTA's first item (later ones were loaded during their predecessor)
                load_q(q_region, bar(BAR_Q + (iter & 1)), it.n_tok, h, cu + it.q_tok0);
        }
        const int box_rows = page_box_rows(ps, kBlockN);
        const int sub_blocks = kBlockN / box_rows;
        bool ok = true;
        // where a block comes from: for a context block, this lane's page and first slot
        struct Src {
            int page, slot0, n_sub_valid;
            bool sub_valid;
        };
        auto source_of = [&](int j) {
            Src s{0, 0, 0, false};
            if (j < n_ctx_blocks) {
                const int pos = j * kBlockN + lane * box_rows;
                s.sub_valid = lane < sub_blocks && pos < c;
                if (s.sub_valid) {
                    s.page = debug_read_page(a, pt_row[pos / ps]);
                    s.slot0 = pos % ps;
                }
                s.n_sub_valid = __popc(__ballot_sync(0xffffffffu, s.sub_valid));
            }
            return s;
        };
        // fills stage j & 1 of the K (kv = 0) or V (kv = 1) ring with block j
        auto fill = [&](int j, int kv, const Src& src) -> bool {
            const bool ctx = j < n_ctx_blocks;
            const int new_row0 = cu + (j - n_ctx_blocks) * kBlockN;
            const uint32_t bytes = ctx ? (uint32_t)src.n_sub_valid * box_rows * D * (FP8 ? 1 : 2) : (uint32_t)C::TILE_BYTES;
            const int st = j & 1;
            if (!debug_stage_ok(a, st, C::KS)) return false;
            const int full = (kv ? BAR_VFULL : BAR_KFULL) + st, empty = (kv ? BAR_VEMPTY : BAR_KEMPTY) + st;
            bool good = true;
            if (j >= 2) good = mbar_wait(bar(empty), ((j >> 1) - 1) & 1, abort_flag, a.status, 0x10 + kv);
            good = __all_sync(0xffffffffu, good);
            if (!good) return false;
            const uint32_t dst = (kv ? smem_base + C::OFF_V : k_region) + st * C::TILE_BYTES;
            if (a.ablation & kAblateLoads) {
                if (lane == 0) mbar_arrive(bar(full));
                return true;
            }
            if (lane == 0) mbar_arrive_expect_tx(bar(full), (QF8 && !ctx && kv == 0) ? (uint32_t)C::BLK_BYTES : bytes);
            __syncwarp();
            if (ctx) {
                if (src.sub_valid) {
                    if constexpr (FP8) {
                        // raw FP8 rows (d_k bytes each) land in the upper half of the stage
                        tma_load_4d(dst + C::BLK_BYTES + lane * box_rows * 128, &maps.cache, 0, 2 * h + kv, src.slot0, src.page,
                                    bar(full));
                    } else {
#pragma unroll
                        for (int b = 0; b < C::NBLK; ++b)
                            tma_load_4d(dst + b * C::BLK_BYTES + lane * box_rows * 128, &maps.cache, b * 64, 2 * h + kv, src.slot0,
                                        src.page, bar(full));
                    }
                }
            } else if (lane == 0) {
                if (QF8 && kv == 0) {  // the batch's own K codes, where a context block's raw rows land
                    tma_load_3d(dst + C::BLK_BYTES, &maps.new_k, 0, h, new_row0, bar(full));
                } else {
#pragma unroll
                    for (int b = 0; b < C::NBLK; ++b)
                        tma_load_3d(dst + b * C::BLK_BYTES, kv ? &maps.new_v : &maps.new_k, b * 64, h, new_row0, bar(full));
                }
            }
            return true;
        };
        // First key block of an item (bf16 cache), into stage 0 of region `dst` on barrier `kbar`:
        // of this item (the CTA's first) or, while this one still runs, of the next.
        auto load_k0 = [&](const TileCtx& of, uint32_t dst, uint32_t kbar) {
            if (a.ablation & kAblateLoads) {
                if (lane == 0) mbar_arrive(kbar);
                return;
            }
            if (of.n_ctx_blocks > 0) {
                const int pos = lane * box_rows;
                const bool sub_valid = lane < sub_blocks && pos < of.c;
                int page = 0;
                if (sub_valid) page = debug_read_page(a, of.pt_row[pos / ps]);
                const int n_sub_valid = __popc(__ballot_sync(0xffffffffu, sub_valid));
                if (lane == 0) mbar_arrive_expect_tx(kbar, (uint32_t)n_sub_valid * box_rows * D * 2);
                __syncwarp();
                if (sub_valid) {
#pragma unroll
                    for (int b = 0; b < C::NBLK; ++b)
                        tma_load_4d(dst + b * C::BLK_BYTES + lane * box_rows * 128, &maps.cache, b * 64, 2 * of.h, pos % ps, page, kbar);
                }
            } else if (lane == 0) {
                mbar_arrive_expect_tx(kbar, (uint32_t)C::TILE_BYTES);
#pragma unroll
                for (int b = 0; b < C::NBLK; ++b) tma_load_3d(dst + b * C::BLK_BYTES, &maps.new_k, b * 64, of.h, of.cu, kbar);
            }
        };
        if (!FP8 && k0_prefetched_for != iter) load_k0(it, k_region, bar(BAR_K0 + (iter & 1)));
        // The keys run one block ahead of the values: K(j+1) goes out before V(j).  A V stage is held
        // much longer than a K stage (until the PV product of its block, i.e. through that block's whole
        // softmax), and with the loads in block order the wait for a free V stage also held back the
        // next block's keys, whose stage had long been free.
        // (The loop is kept to what a block needs: this warp gets an issue slot every 60 cycles or so,
        // and on 16-slot pages a block is 32 boxes.)
        Src prev = source_of(0);
        if constexpr (FP8) {
            ok = fill(0, 0, prev);
        } else if (lane == 0) {
            // bf16 cache: block 0 is on its way already, on BAR_K0; stage 0's own barrier is moved past
            // its first phase, so that block 2k finds it in phase k as ever
            mbar_arrive(bar(BAR_KFULL + 0));
        }
        if (out_stores_pending) {  // the previous item's output tiles were parked in the V ring: before the first V block
            if (lane == 0) bulk_wait_read();
            __syncwarp();
            out_stores_pending = false;
        }
        for (int t = 1; t <= n_blocks && ok; ++t) {
            Src cur{0, 0, 0, false};
            if (t < n_blocks) {
                cur = source_of(t);
                ok = fill(t, 0, cur);
            }
            if (ok) ok = fill(t - 1, 1, prev);
            prev = cur;
        }
        // the next item's query tiles, into this item's K ring once its last score product has read it
        if (ok) ok = mbar_wait(bar(BAR_NEXT), iter & 1, abort_flag, a.status, 0x12);
        const volatile int* nxt = item_slots + ((iter + 1) & 1) * RAW_INTS;
        if (ok && nxt[RAW_ITEM] < n_items) {
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const int uses = (n_blocks + 1 - st) >> 1;  // key blocks of this item that went through stage st
                if (uses > 0) ok = ok && mbar_wait(bar(BAR_KEMPTY + st), (uses - 1) & 1, abort_flag, a.status, 0x13);
            }
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                if (lane == 0)
                    load_q(k_region, bar(BAR_Q + ((iter + 1) & 1)), nxt[RAW_NTOK], nxt[RAW_HEAD], nxt[RAW_CU] + nxt[RAW_TOK0]);
                q_prefetched_for = iter + 1;
                if constexpr (!FP8) {
                    // ... and its first key block, into this item's query region, which its last score
                    // product has read (the output tiles are parked in the V ring): the next item's
                    // first product then starts without the 1600 cycles a load takes to arrive
                    const TileCtx nx = tile_ctx_from_raw(a, nxt, kBlockN);
                    load_k0(nx, q_region, bar(BAR_K0 + ((iter + 1) & 1)));
                    k0_prefetched_for = iter + 1;
                }
            }
        }
        // The output tiles: the softmax groups park a full tile in the V ring (see the epilogue) and this
        // warp hands it to the copy engine, so that no softmax thread waits for the store to read its
        // tile out; the wait is taken before the next item's first V block instead.
        if (ok && !(a.ablation & kAblateCompute) && !(it.n_tok <= TQ && n_blocks >= 2)) {
            const int st_last = (n_blocks - 1) & 1;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                if ((x + 1) * TQ > it.n_tok) break;
                ok = mbar_wait(bar(BAR_EPI + x), 0, abort_flag, a.status, 0x36 + x);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t o_buf = smem_base + C::OFF_V + (x == 0 ? st_last ^ 1 : st_last) * C::TILE_BYTES;
#pragma unroll
                    for (int b = 0; b < C::NBLK; ++b)
                        tma_store_3d(&maps.out, o_buf + b * C::BLK_BYTES, b * 64, h * G, cu + it.q_tok0 + x * TQ);
                    bulk_commit();
                }
                out_stores_pending = true;
            }
        }
      } else if (warp == 1) {
        // ================================ MMA issuer ================================
        constexpr uint32_t idesc_qk = QF8 ? instr_desc_e4m3(128, kBlockN, 0, 0) : instr_desc_bf16(128, kBlockN, 0, 0);
        constexpr uint32_t idesc_pv = instr_desc_bf16(128, D, 0, 1);
        // Descriptors differ only in their 14-bit start-address field, so each product is issued
        // with one 32-bit add per operand: the issuing thread must not become the bottleneck.  For
        // the same reason the issuing lane is the one `elect.sync` names, not "lane 0": the branch
        // is then known to hold one lane of a converged warp, and issuing a product costs that
        // thread less (prefill 1160 -> 1190 TFLOP/s; the single-tile kernel, where the effect is
        // larger, elects per instruction).  Every wait's outcome is agreed on by the warp first, so
        // that the lanes are together at each election.
        constexpr uint32_t desc_hi = smem_desc_sw128_hi(1024);
        const uint32_t q_lo[2] = {smem_desc_sw128_lo(smem_base + q_off, 16), smem_desc_sw128_lo(smem_base + q_off + C::TILE_BYTES, 16)};
        // (FP8 scores: the key operand is the raw code rows, which sit in the second half of a K stage)
        const uint32_t k_lo = smem_desc_sw128_lo(smem_base + k_off + (QF8 ? C::BLK_BYTES : 0), 16);
        const uint32_t v_lo = smem_desc_sw128_lo(smem_base + C::OFF_V, C::BLK_BYTES);
        const bool no_compute = a.ablation & kAblateCompute;  // bench switch: commits without products
        auto issue_qk = [&](int x, int st) {  // S_x = Q_x K^T over d_k in steps of 16
            if (no_compute) return;
            const uint32_t kl = k_lo + st * (C::TILE_BYTES >> 4);
            if constexpr (QF8) {
#pragma unroll
                for (int ks = 0; ks < D / 32; ++ks)  // 32 code bytes of every row per product
                    umma_ss_f8(tm_s[x], make_desc(q_lo[x] + ks * 2, desc_hi), make_desc(kl + ks * 2, desc_hi), idesc_qk, ks > 0);
            } else {
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = ((ks / 4) * C::BLK_BYTES + (ks % 4) * 32) >> 4;
                    umma_ss(tm_s[x], make_desc(q_lo[x] + off, desc_hi), make_desc(kl + off, desc_hi), idesc_qk, ks > 0);
                }
            }
        };
        auto issue_pv = [&](int x, int st, bool first) {  // O_x (+)= P_x V over 128 positions in steps of 16
            if (no_compute) return;
            const uint32_t vl = v_lo + st * (C::TILE_BYTES >> 4);
#pragma unroll
            for (int kk = 0; kk < kBlockN / 16; ++kk)
                umma_ts(tm_o[x], tm_s[x] + kk * 8, make_desc(vl + kk * (2048 >> 4), desc_hi), idesc_pv, !(first && kk == 0));
        };
        // barrier that says block j's K (or V) operand is in place: with an FP8 cache a context
        // block is ready once the converter warps have expanded it, not when its bytes land
        auto k_ready = [&](int j) { return bar((FP8 && !QF8 && j < n_ctx_blocks ? BAR_KCONV : BAR_KFULL) + (j & 1)); };
        auto v_ready = [&](int j) { return bar((FP8 && j < n_ctx_blocks ? BAR_VCONV : BAR_VFULL) + (j & 1)); };
        const bool two_tiles = it.n_tok > TQ;  // a short item (at most TQ tokens) runs tile A only
        const bool split = !two_tiles && n_blocks >= 2;  // ... with its key blocks dealt to both accumulators
        bool ok = mbar_wait(bar(BAR_Q + (iter & 1)), (iter >> 1) & 1, abort_flag, a.status, 0x20);
        if constexpr (FP8) {
            ok = ok && mbar_wait(k_ready(0), 0, abort_flag, a.status, 0x21);
        } else {
            ok = ok && mbar_wait(bar(BAR_K0 + (iter & 1)), (iter >> 1) & 1, abort_flag, a.status, 0x21);
        }
        if (split) {
            // Block j uses score buffer, accumulator and K/V stage j & 1, all with tile A's queries.
            // Order of issue: S_0, S_1, then per block O_x += P_j V_j followed by S_(j+2).
            auto issue_qk_a = [&](int x, int st) {
                if (no_compute) return;
                const uint32_t kl = k_lo + st * (C::TILE_BYTES >> 4);
                if constexpr (QF8) {
#pragma unroll
                    for (int ks = 0; ks < D / 32; ++ks)
                        umma_ss_f8(tm_s[x], make_desc(q_lo[0] + ks * 2, desc_hi), make_desc(kl + ks * 2, desc_hi), idesc_qk, ks > 0);
                } else {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = ((ks / 4) * C::BLK_BYTES + (ks % 4) * 32) >> 4;
                        umma_ss(tm_s[x], make_desc(q_lo[0] + off, desc_hi), make_desc(kl + off, desc_hi), idesc_qk, ks > 0);
                    }
                }
            };
            if (ok) {
                tc_fence_after();
                if (elect_one()) {
                    issue_qk_a(0, 0);
                    tc_commit(bar(BAR_SFULL + 0));
                    tc_commit(bar(BAR_KEMPTY + 0));
                }
                __syncwarp();
                ok = mbar_wait(k_ready(1), 0, abort_flag, a.status, 0x26);
                if (ok) {
                    tc_fence_after();
                    if (elect_one()) {
                        issue_qk_a(1, 1);
                        tc_commit(bar(BAR_SFULL + 1));
                        tc_commit(bar(BAR_KEMPTY + 1));
                    }
                    __syncwarp();
                }
            }
            for (int j = 0; j < n_blocks && ok; ++j) {
                const int st = j & 1, ph = (j >> 1) & 1;
                ok = mbar_wait(v_ready(j), ph, abort_flag, a.status, 0x22);
                if (!ok) break;
                const bool ctx = j < n_ctx_blocks;
                const int n_valid = ctx ? min(kBlockN, c - j * kBlockN) : min(kBlockN, n_new_visible - (j - n_ctx_blocks) * kBlockN);
                if (n_valid < kBlockN) {  // zero the rows of V past the block's valid positions (see below)
                    uint8_t* v_s = smem + C::OFF_V + st * C::TILE_BYTES;
                    for (int idx = lane; idx < (kBlockN - n_valid) * C::NBLK * 8; idx += 32) {
                        const int r = n_valid + idx / (C::NBLK * 8), rem = idx % (C::NBLK * 8);
                        *reinterpret_cast<uint4*>(v_s + (rem / 8) * C::BLK_BYTES + r * 128 + (rem % 8) * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                }
                ok = mbar_wait(bar(BAR_PREADY + st), ph, abort_flag, a.status, 0x23);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    issue_pv(st, st, j < 2);
                    tc_commit(bar(BAR_ODONE + st));
                    tc_commit(bar(BAR_VEMPTY + st));
                    *progress = j + 1;
                }
                __syncwarp();
                if (j + 2 < n_blocks) {
                    ok = mbar_wait(k_ready(j + 2), ((j + 2) >> 1) & 1, abort_flag, a.status, 0x24);
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        issue_qk_a(st, st);
                        tc_commit(bar(BAR_SFULL + st));
                        tc_commit(bar(BAR_KEMPTY + st));
                    }
                    __syncwarp();
                }
            }
        } else {
        if (ok) {
            tc_fence_after();
            if (elect_one()) {
                issue_qk(0, 0);
                tc_commit(bar(BAR_SFULL + 0));
                if (two_tiles) {
                    issue_qk(1, 0);
                    tc_commit(bar(BAR_SFULL + 1));
                }
                tc_commit(bar(BAR_KEMPTY + 0));
            }
            __syncwarp();
        }
        for (int j = 0; j < n_blocks && ok; ++j) {
            const int st = j & 1, ph = (j >> 1) & 1;
            ok = mbar_wait(v_ready(j), ph, abort_flag, a.status, 0x22);
            if (!ok) break;
            // rows of V past the block's valid positions may hold stale or foreign data: make them
            // finite (zero) so that masked probabilities (exactly 0) cannot produce NaN
            const bool ctx = j < n_ctx_blocks;
            const int n_valid = ctx ? min(kBlockN, c - j * kBlockN) : min(kBlockN, n_new_visible - (j - n_ctx_blocks) * kBlockN);
            if (n_valid < kBlockN) {
                uint8_t* v_s = smem + C::OFF_V + st * C::TILE_BYTES;
                for (int idx = lane; idx < (kBlockN - n_valid) * C::NBLK * 8; idx += 32) {
                    const int r = n_valid + idx / (C::NBLK * 8), rem = idx % (C::NBLK * 8);
                    *reinterpret_cast<uint4*>(v_s + (rem / 8) * C::BLK_BYTES + r * 128 + (rem % 8) * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async_smem();
                __syncwarp();
            }
            const bool more = j + 1 < n_blocks;
            const int st1 = (j + 1) & 1, ph1 = ((j + 1) >> 1) & 1;
            ok = mbar_wait(bar(BAR_PREADY + 0), j & 1, abort_flag, a.status, 0x23);
            if (!ok) break;
            tc_fence_after();
            if (elect_one()) {
                issue_pv(0, st, j == 0);
                tc_commit(bar(BAR_ODONE + 0));
                *progress = j + 1;
            }
            __syncwarp();
            if (more) {
                ok = mbar_wait(k_ready(j + 1), ph1, abort_flag, a.status, 0x24);
                if (!ok) break;
                tc_fence_after();
                if (elect_one()) {
                    issue_qk(0, st1);
                    tc_commit(bar(BAR_SFULL + 0));
                }
                __syncwarp();
            }
            if (two_tiles) {
                ok = mbar_wait(bar(BAR_PREADY + 1), j & 1, abort_flag, a.status, 0x25);
                if (!ok) break;
                tc_fence_after();
            }
            if (elect_one()) {
                if (two_tiles) {
                    issue_pv(1, st, j == 0);
                    tc_commit(bar(BAR_ODONE + 1));
                }
                tc_commit(bar(BAR_VEMPTY + st));
                if (more) {
                    if (two_tiles) {
                        issue_qk(1, st1);
                        tc_commit(bar(BAR_SFULL + 1));
                    }
                    tc_commit(bar(BAR_KEMPTY + st1));
                }
            }
            __syncwarp();
        }
        }  // not split
      } else {
        // ================================ fused cache update ================================
        // One warp draws the next item and fetches its list entry and lengths while this item runs,
        // so that the next turn of the loop starts without that chain of loads - but not before the
        // item is within two key blocks of its end: a CTA that reserved its next item at the start
        // of a long one would keep it from the CTAs that fall idle in the meantime.  A short item
        // fetches first thing (the producer needs the entry to load the next query tiles in time),
        // a long one after its share of the update.
        auto fetch_next = [&]() {
            if (lane == 0) {
                const long long t0 = clock64();
                while (*progress < n_blocks - 2 && !*abort_flag && clock64() - t0 < 2000000000LL) __nanosleep(256);
            }
            __syncwarp();
            volatile int* nxt = item_slots + ((iter + 1) & 1) * RAW_INTS;
            draw_and_fetch_tile(a, persistent, n_items, nxt, lane);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(BAR_NEXT));  // the producer may now load the next item's query tiles
            // warm L2 with the next item's own tokens' K/V rows: the loads that open the next item
            // then find them there instead of in HBM
            if (nxt[RAW_ITEM] < n_items) {
                const int n_cu = nxt[RAW_CU], n_tok0 = nxt[RAW_TOK0], n_h = nxt[RAW_HEAD];
                if (lane < C::NBLK) {
                    tma_prefetch_3d(&maps.new_k, lane * 64, n_h, n_cu + n_tok0 / kBlockN * kBlockN);
                } else if (lane < 2 * C::NBLK) {
                    tma_prefetch_3d(&maps.new_v, (lane - C::NBLK) * 64, n_h, n_cu + n_tok0 / kBlockN * kBlockN);
                }
            }
        };
        const bool fetch_early = n_blocks <= 2;
        if (warp == 3 && fetch_early) fetch_next();
        if constexpr (FP8) {
            // FP8 cache: the item's own tokens were quantised and stored by the pass that ran before
            // this kernel.  These two warps expand the context blocks instead: a thread turns one raw
            // row (d_k code bytes, in the upper half of the stage) into its two 64-column halves of
            // the bf16 operand layout, every E4M3 value being exact in bf16.  The second half lands
            // on the raw row itself, which the thread has read by then.
            static_assert(!FP8 || D == 128, "raw rows of 128 bytes");
            const int t = tid - 64, box_rows = page_box_rows(ps, kBlockN);
            bool okc = true;
            for (int j = 0; j < n_ctx_blocks && okc; ++j) {
                const int st = j & 1, ph = (j >> 1) & 1;
                const int rows = min(kBlockN, (min(kBlockN, c - j * kBlockN) + box_rows - 1) / box_rows * box_rows);
#pragma unroll
                for (int kv = QF8 ? 1 : 0; kv < 2; ++kv) {  // (FP8 scores: the keys are used as they are)
                    okc = okc && mbar_wait(bar((kv ? BAR_VFULL : BAR_KFULL) + st), ph, abort_flag, a.status, 0x50 + kv);
                    if (!okc) break;
                    uint8_t* stage = smem + (kv ? (uint32_t)C::OFF_V : k_off) + st * C::TILE_BYTES;
                    for (int r = t; r < rows; r += 64) {
                        const uint8_t* raw = stage + C::BLK_BYTES + r * 128;
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint4 w[4];
#pragma unroll
                            for (int cch = 0; cch < 4; ++cch)
                                w[cch] = *reinterpret_cast<const uint4*>(raw + (((half * 4 + cch) ^ (r & 7)) << 4));
                            uint8_t* dst_row = stage + half * C::BLK_BYTES + r * 128;
#pragma unroll
                            for (int cch = 0; cch < 4; ++cch) {
                                uint4 lo, hi;
                                lo.x = e4m3x2_to_bf16x2(w[cch].x & 0xffffu);
                                lo.y = e4m3x2_to_bf16x2(w[cch].x >> 16);
                                lo.z = e4m3x2_to_bf16x2(w[cch].y & 0xffffu);
                                lo.w = e4m3x2_to_bf16x2(w[cch].y >> 16);
                                hi.x = e4m3x2_to_bf16x2(w[cch].z & 0xffffu);
                                hi.y = e4m3x2_to_bf16x2(w[cch].z >> 16);
                                hi.z = e4m3x2_to_bf16x2(w[cch].w & 0xffffu);
                                hi.w = e4m3x2_to_bf16x2(w[cch].w >> 16);
                                *reinterpret_cast<uint4*>(dst_row + (((2 * cch) ^ (r & 7)) << 4)) = lo;
                                *reinterpret_cast<uint4*>(dst_row + (((2 * cch + 1) ^ (r & 7)) << 4)) = hi;
                            }
                        }
                    }
                    fence_proxy_async_smem();
                    mbar_arrive(bar((kv ? BAR_VCONV : BAR_KCONV) + st));
                }
            }
        } else if (!(a.ablation & kAblateUpdate) && (it.flags & kFlagWriteKv)) {
            if constexpr (SHORT) {
                using U = TileUpdate<D>;
                tile_update_rounds_tma<D>(a, maps, it, (warp - 2) * U::TPW, 2 * U::TPW, lane, smem_base + C::OFF_UPD + (warp - 2) * U::WARP_BYTES,
                                          bar(BAR_UPD + warp - 2), upd_parity,
                                          [&](uint32_t b, uint32_t ph) { return mbar_wait(b, ph, abort_flag, a.status, 0x14); });
            } else {
                tile_update_cache<D>(a, it, warp - 2, lane, smem_base + C::OFF_UPD);
            }
        }
        if (warp == 3 && !fetch_early) fetch_next();
      }
      }  // item loop of the first warpgroup
      if (warp == 0 && lane == 0) bulk_wait_read();  // the last output tiles have left shared memory
    } else {
        // ================================ softmax warps ================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;\n");
        for (int iter = 0;; ++iter) {
        tc_fence_before();
        __syncthreads();  // everyone is done with the previous item
        if (*abort_flag) break;
        __syncthreads();  // item slot filled and mbarriers re-initialised by the first warpgroup
        tc_fence_after();
        const volatile int* slot = item_slots + (iter & 1) * RAW_INTS;
        if (slot[RAW_ITEM] >= n_items) break;
        const TileCtx it = tile_ctx_from_raw(a, slot, kBlockN);
      if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;  // (bounds-checked build: every thread of the CTA takes this exit together)
        const int h = it.h, cu = it.cu, q_r = it.q_r, L = it.L, c = it.c;
        const int n_ctx_blocks = it.n_ctx_blocks, n_new_visible = it.n_new_visible, n_blocks = it.n_blocks;
        const uint32_t q_off = (iter & 1) ? C::OFF_K : C::OFF_QA;  // this item's query region (see the producer)
        const int x = (warp - 4) >> 2;              // 0: tile A, 1: tile B
        const int quarter = warp & 3;               // TMEM lanes this warp may touch: 32*quarter ..
        const int row = quarter * 32 + lane;        // query row of this thread inside its tile
        const int tok_in_tile = row / G, g = row % G;
        // A short item (one tile of queries) with at least two key blocks is split by key blocks:
        // both softmax groups work on tile A's rows, group x takes the blocks j = x (mod 2) into its
        // own accumulator, and group 0 merges the two partial results in the epilogue.  The tensor
        // products of one half then overlap the softmax of the other, as with two query tiles.
        const bool split = it.n_tok <= TQ && n_blocks >= 2;
        const int xt = split ? 0 : x;                       // query tile of this thread's row
        const int tok = it.q_tok0 + xt * TQ + tok_in_tile;  // token index inside the sequence
        const bool row_valid = xt * TQ + tok_in_tile < it.n_tok;
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t s_addr = tm_s[x] + lane_sel, o_addr = tm_o[x] + lane_sel;
        int lim = a.causal ? c + min(tok, q_r - 1) : L - 1;  // last visible key position of this row
        int first = 0;                                       // first visible key position
        const bool packed = it.n_seqs > 1;
        if (packed) {  // a row sees the keys of its own sequence only
            const int k = packed_seq_of(it, min(tok, it.n_tok - 1));
            first = it.bounds[k];
            lim = a.causal ? min(tok, it.bounds[k + 1] - 1) : it.bounds[k + 1] - 1;
        }

        float m_ref = -INFINITY, l_sum = 0.f;
        bool ok = true;
        // tile B idles on a short item with a single key block
        const int my_blocks = split ? (n_blocks + 1 - x) >> 1 : (x == 1 && it.n_tok <= TQ) ? 0 : n_blocks;
        if (SHORT && a.short_items == 2 && n_blocks == 1 && n_new_visible <= kBlockN / 2 && my_blocks == 1 && !(a.ablation & kAblateCompute)) {
            // the item's only block is at most half full (no context then: positions 0 .. n_new_visible - 1)
            ok = mbar_wait(bar(BAR_SFULL + x), 0, abort_flag, a.status, 0x30 + x);
            if (ok) {
                tc_fence_after();
                const float2 ml = softmax_half_block(s_addr, min(n_new_visible, lim + 1), packed ? first : 0, a.scale_log2);
                m_ref = ml.x, l_sum = ml.y;
                tc_fence_before();
                mbar_arrive(bar(BAR_PREADY + x));
            }
        } else
        for (int jj = 0; jj < my_blocks; ++jj) {
            const int j = split ? 2 * jj + x : jj;  // key block; barrier phases count this group's own blocks
            ok = mbar_wait(bar(BAR_SFULL + x), jj & 1, abort_flag, a.status, 0x30 + x);
            if (!ok) break;
            tc_fence_after();
            if (a.ablation & kAblateCompute) {  // bench switch: hand over at once
                tc_fence_before();
                mbar_arrive(bar(BAR_PREADY + x));
                continue;
            }
            float s[kBlockN];
#pragma unroll
            for (int ch = 0; ch < kBlockN / 32; ++ch) {
                uint32_t r32[32];
                tmem_ld32(s_addr + ch * 32, r32);
#pragma unroll
                for (int i = 0; i < 32; ++i) s[ch * 32 + i] = __uint_as_float(r32[i]);
            }
            tc_wait_ld();
            // visible keys of this row inside the block: positions pos_base .. pos_base + n_vis - 1
            const bool ctx = j < n_ctx_blocks;
            const int pos_base = ctx ? j * kBlockN : c + (j - n_ctx_blocks) * kBlockN;
            const int n_valid = ctx ? min(kBlockN, c - pos_base) : min(kBlockN, c + n_new_visible - pos_base);
            const int n_vis = min(n_valid, lim - pos_base + 1);
            if (__any_sync(0xffffffffu, n_vis < kBlockN)) {
#pragma unroll
                for (int i = 0; i < kBlockN; ++i)
                    if (i >= n_vis) s[i] = -INFINITY;
            }
            if (packed) {
                const int n_before = first - pos_base;  // keys of earlier sequences in this block
#pragma unroll
                for (int i = 0; i < kBlockN; ++i)
                    if (i < n_before) s[i] = -INFINITY;
            }
            float mxp[8];  // independent partial maxima: no 128-long dependency chain
#pragma unroll
            for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(s[i], s[i + 8]);
#pragma unroll
            for (int i = 16; i < kBlockN; i += 16)
#pragma unroll
                for (int k = 0; k < 8; ++k) mxp[k] = max3(mxp[k], s[i + k], s[i + k + 8]);
            const float mx = fmaxf(max3(mxp[0], mxp[1], mxp[2]), max3(fmaxf(mxp[3], mxp[4]), max3(mxp[5], mxp[6], mxp[7]), -INFINITY));
            const float mx2 = mx * a.scale_log2;
            if (jj == 0) {
                m_ref = mx2;
            } else {
                const bool grow = mx2 - m_ref > kRescaleThreshold;
                if (__any_sync(0xffffffffu, grow)) {
                    // the previous PV product of this tile must have landed before O is touched
                    ok = mbar_wait(bar(BAR_ODONE + x), (jj - 1) & 1, abort_flag, a.status, 0x32 + x);
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
            float lp[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};  // independent partial sums, in pairs
#pragma unroll
            for (int ch = 0; ch < 2; ++ch) {
                uint32_t p32[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    // a pair of elements per instruction for the scaling and for the row sum (packed
                    // fp32 arithmetic): the softmax threads are bound by their own instruction count
                    float x0, x1;
                    fma2_bcast(x0, x1, s[ch * 64 + 2 * i], s[ch * 64 + 2 * i + 1], a.scale_log2, neg_m);
                    const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
                    add2(lp[2 * (i & 3)], lp[2 * (i & 3) + 1], p0, p1);
                    p32[i] = pack_bf16x2(p0, p1);
                }
                tmem_st32(s_addr + ch * 32, p32);
            }
            l_sum += ((lp[0] + lp[1]) + (lp[2] + lp[3])) + ((lp[4] + lp[5]) + (lp[6] + lp[7]));
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(bar(BAR_PREADY + x));
        }
        // ---- epilogue: O / l -> bf16 -> out ----
        if (ok && my_blocks > 0) ok = mbar_wait(bar(BAR_ODONE + x), (my_blocks - 1) & 1, abort_flag, a.status, 0x34 + x);
        float f_own = 1.f, f_other = 0.f;  // weights of the two halves of a split item
        if (a.ablation & kAblateCompute) ok = false;  // nothing to write
        if (ok && split) {
            // group 1 publishes its softmax state; group 0 waits for it (group 1's last product has
            // landed by then) and weighs the two accumulators
            float2* stats = reinterpret_cast<float2*>(smem + q_off + C::TILE_BYTES);  // the idle second query tile
            if (x == 1) {
                tc_fence_after();
                stats[row] = make_float2(m_ref, l_sum);
                tc_fence_before();
                mbar_arrive(bar(BAR_EPI + 1));
            } else {
                ok = mbar_wait(bar(BAR_EPI + 1), 0, abort_flag, a.status, 0x37);
                if (ok) {
                    const float2 other = stats[row];
                    const float m_all = fmaxf(m_ref, other.x);
                    f_own = fast_exp2(m_ref - m_all);
                    f_other = fast_exp2(other.x - m_all);
                    l_sum = l_sum * f_own + other.y * f_other;
                }
            }
        }
        if (ok && my_blocks > 0 && !(split && x == 1)) {
            tc_fence_after();
            const float inv = a.out_scale / l_sum;  // out_scale: 1, or v_scale of an FP8 cache
            if (split) {
                // merged output of a split item: rows go straight to global memory
                const float wa = f_own * inv, wb = f_other * inv;
                const uint32_t o_other = tm_o[1] + lane_sel;
                uint16_t* dst = a.out + (((int64_t)cu + tok) * a.h_q + h * G + g) * D;
#pragma unroll
                for (int ch = 0; ch < D / 32; ++ch) {
                    uint32_t r32[32], q32[32];
                    tmem_ld32(o_addr + ch * 32, r32);
                    tmem_ld32(o_other + ch * 32, q32);
                    tc_wait_ld();
                    if (row_valid) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            float v8[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                v8[e] = __uint_as_float(r32[8 * i + e]) * wa + __uint_as_float(q32[8 * i + e]) * wb;
                            uint4 v;
                            v.x = pack_bf16x2(v8[0], v8[1]);
                            v.y = pack_bf16x2(v8[2], v8[3]);
                            v.z = pack_bf16x2(v8[4], v8[5]);
                            v.w = pack_bf16x2(v8[6], v8[7]);
                            *reinterpret_cast<uint4*>(dst + ch * 32 + i * 8) = v;
                        }
                    }
                }
            } else if ((x + 1) * TQ <= it.n_tok) {
                // A full tile goes out through shared memory: each thread parks its row in the V
                // ring, in the swizzled layout of the tensor map, and the producer warp stores the
                // tile with the copy engine.  Row-per-thread stores to global would touch 32 lines per
                // instruction.  Tile A, done first, takes the stage the last key block did not use
                // (tile B's last PV product may still be reading that block's stage); tile B's own
                // last product is the last reader of the other.
                const int st_last = (n_blocks - 1) & 1;
                const uint32_t q_buf = smem_base + C::OFF_V + (x == 0 ? st_last ^ 1 : st_last) * C::TILE_BYTES;
#pragma unroll
                for (int ch = 0; ch < D / 32; ++ch) {
                    uint32_t r32[32];
                    tmem_ld32(o_addr + ch * 32, r32);
                    tc_wait_ld();
                    const uint32_t blk = q_buf + (ch / 2) * C::BLK_BYTES + row * 128;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const uint32_t dst_s = blk + ((((ch & 1) * 4 + i) ^ (row & 7)) << 4);
                        st_shared_v4(dst_s, pack_bf16x2(__uint_as_float(r32[8 * i + 0]) * inv, __uint_as_float(r32[8 * i + 1]) * inv),
                                     pack_bf16x2(__uint_as_float(r32[8 * i + 2]) * inv, __uint_as_float(r32[8 * i + 3]) * inv),
                                     pack_bf16x2(__uint_as_float(r32[8 * i + 4]) * inv, __uint_as_float(r32[8 * i + 5]) * inv),
                                     pack_bf16x2(__uint_as_float(r32[8 * i + 6]) * inv, __uint_as_float(r32[8 * i + 7]) * inv));
                    }
                }
                fence_proxy_async_smem();
                mbar_arrive(bar(BAR_EPI + x));
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
        }  // item loop of the softmax warpgroups
    }
    // ---- teardown: everyone arrives, then the allocating warp frees TMEM ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (tid == 0) {  // the last CTA to leave resets the counters for the next launch
        __threadfence();
        if (atomicAdd(a.tile_counters + 1, 1) == (int)gridDim.x - 1) {
            a.tile_counters[0] = 0;
            a.tile_counters[1] = 0;
        }
    }
}

// ---- host side -------------------------------------------------------------------------------

template <int D, int G, bool FP8>
cudaError_t launch_tile(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    constexpr bool kCanQF8 = FP8 && D == 128;
    if (a.q_fp8 && !kCanQF8) return cudaErrorInvalidValue;
    TileMaps maps;
    if (!cached_tile_maps(cache, a, token_rows, D, G, 128 / G, kBlockN, &maps)) return cudaErrorInvalidValue;
    if (FP8) {
        if (cudaError_t e = launch_quantise_new<D>(a, stream); e != cudaSuccess) return e;
    }
    const int grid = a.dev_counts ? a.num_tile_ctas : a.num_tile_ctas > 0 && a.num_tile_ctas < a.num_tile_items ? a.num_tile_ctas : a.num_tile_items;
    if constexpr (kCanQF8) {
        if (a.q_fp8) {
            rpa_tile_kernel<D, G, true, true><<<grid, kTileThreads, TileCfg<D>::SMEM, stream>>>(a, maps);
            return cudaGetLastError();
        }
    }
    if constexpr (!FP8) {
        if (a.short_items && !a.dev_counts) {
            rpa_tile_kernel<D, G, false, false, true><<<grid, kTileThreads, TileCfg<D>::SMEM, stream>>>(a, maps);
            return cudaGetLastError();
        }
    }
    rpa_tile_kernel<D, G, FP8, false><<<grid, kTileThreads, TileCfg<D>::SMEM, stream>>>(a, maps);
    return cudaGetLastError();
}

template <int D, int G, bool FP8>
cudaError_t prepare_tile() {
    if constexpr (FP8 && D == 128) {
        cudaError_t e = cudaFuncSetAttribute(rpa_tile_kernel<D, G, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<D>::SMEM);
        if (e != cudaSuccess) return e;
    }
    if constexpr (!FP8) {
        cudaError_t e = cudaFuncSetAttribute(rpa_tile_kernel<D, G, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<D>::SMEM);
        if (e != cudaSuccess) return e;
    }
    return cudaFuncSetAttribute(rpa_tile_kernel<D, G, FP8, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, TileCfg<D>::SMEM);
}

#define RPA_TILE_DISPATCH(D_, G_, F8_, FN, ...)                         \
    do {                                                                \
        if ((D_) == 128 && (F8_)) {                                     \
            switch (G_) {                                               \
                case 1: return FN<128, 1, true>(__VA_ARGS__);           \
                case 2: return FN<128, 2, true>(__VA_ARGS__);           \
                case 4: return FN<128, 4, true>(__VA_ARGS__);           \
                case 8: return FN<128, 8, true>(__VA_ARGS__);           \
                case 16: return FN<128, 16, true>(__VA_ARGS__);         \
            }                                                           \
        } else if ((D_) == 128) {                                       \
            switch (G_) {                                               \
                case 1: return FN<128, 1, false>(__VA_ARGS__);          \
                case 2: return FN<128, 2, false>(__VA_ARGS__);          \
                case 4: return FN<128, 4, false>(__VA_ARGS__);          \
                case 8: return FN<128, 8, false>(__VA_ARGS__);          \
                case 16: return FN<128, 16, false>(__VA_ARGS__);        \
            }                                                           \
        } else if ((D_) == 64 && !(F8_)) {                              \
            switch (G_) {                                               \
                case 1: return FN<64, 1, false>(__VA_ARGS__);           \
                case 2: return FN<64, 2, false>(__VA_ARGS__);           \
                case 4: return FN<64, 4, false>(__VA_ARGS__);           \
                case 8: return FN<64, 8, false>(__VA_ARGS__);           \
                case 16: return FN<64, 16, false>(__VA_ARGS__);         \
            }                                                           \
        }                                                               \
    } while (0)

}  // namespace

// One warp waits on an mbarrier that nothing ever arrives at, with a limit of about a millisecond:
// exercises the give-up path of the bounded waits (status word set, normal return) on demand.
__global__ void rpa_wait_selftest_kernel(uint32_t* status) {
    __shared__ __align__(8) unsigned long long barrier;
    __shared__ uint32_t abort_flag;
    const uint32_t bar = smem_u32(&barrier);
    if (threadIdx.x == 0) {
        abort_flag = 0u;
        mbar_init(bar, 1);
        fence_mbar_init();
    }
    __syncthreads();
    mbar_wait(bar, 0, &abort_flag, status, 0x7F, 2000000LL);
}

cudaError_t launch_wait_selftest(uint32_t* status, cudaStream_t stream) {
    rpa_wait_selftest_kernel<<<1, 32, 0, stream>>>(status);
    return cudaGetLastError();
}

bool tile_kernel_supported(int head_dim, int group) {
    return (head_dim == 64 || head_dim == 128) &&
           (group == 1 || group == 2 || group == 4 || group == 8 || group == 16);
}

bool tile_kernel_fp8_supported(int head_dim, int group) { return head_dim == 128 && tile_kernel_supported(head_dim, group); }

int tile_kernel_tokens(int group) { return 2 * (128 / group); }

cudaError_t tile_kernel_prepare(int head_dim, int group, bool fp8) {
    RPA_TILE_DISPATCH(head_dim, group, fp8, prepare_tile);
    return cudaErrorInvalidValue;
}

cudaError_t launch_tile_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    if (a.num_tile_items <= 0 && !a.dev_counts) return cudaSuccess;
    RPA_TILE_DISPATCH(a.head_dim, a.h_q / a.h_kv, a.kv_fp8 != 0, launch_tile, a, token_rows, cache, stream);
    return cudaErrorInvalidValue;
}

}  // namespace rpa
