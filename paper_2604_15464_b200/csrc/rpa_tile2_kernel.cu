// CTA-pair tile kernel: long-prefill attention on tcgen05 products of 256 rows (cta_group::2).
//
// Two CTAs on neighbouring SMs (a cluster of two) serve one TileItem of up to 4*TQ consecutive new
// tokens of one sequence for one KV head: CTA r takes tokens [2r*TQ, 2(r+1)*TQ) of the item as its
// query tiles A and B (rows = token*h_g + grouped head, Section 3.1.2), exactly as a CTA of the
// two-tile kernel does, with its own softmax warps, TMEM accumulators and output.  What the pair
// shares is the K/V operand: one product computes S (or O) for tile x of BOTH CTAs, 256 rows, and
// reads HALF of the key block (64 of its 128 positions for Q K^T, 64 of the d_k = 128 columns of V
// for P V) from each CTA's shared memory.  Per CTA that is 6 KB instead of 8 KB of shared-memory
// reads per score product and 2 KB instead of 4 KB per PV product - the score product of the
// two-tile kernel runs at the shared-memory read limit, not at the tensor pipe's rate - and every
// K/V byte crosses L2 -> SM once per 4 query tiles instead of once per 2.
//
// One thread of the pair's first CTA issues all products; completion is signalled to the barriers
// of both CTAs (tcgen05.commit to both).  Each CTA's producer warp loads its own halves with plain
// TMA loads into its own shared memory; the second CTA's warp 1 relays "my half has landed" to the
// first CTA's barriers, and its softmax warps arrive on the first CTA's "P ready" barriers.
//
// Items follow one another without a pause.  Nothing is re-initialised between items and no role
// waits for another at an item's end: every mbarrier keeps its phase from block to block across
// items (each role counts the blocks it has seen), the K/V rings run on into the next item's first
// blocks while the current item's last ones are still being consumed, the query tiles alternate
// between two buffers, and the score products of the next item's first block are issued right
// behind the last PV products of the running one - so the output epilogue of an item (TMEM ->
// shared memory -> bulk store) overlaps the next item's first products instead of idling the
// tensor pipe.  Items are drawn by one warp of the first CTA from the device-wide counter (the list
// is sorted heaviest first) a few key blocks before the running item ends, and handed to every
// role of both CTAs through a two-slot ring in shared memory.
//
// Algorithm 1's recurrences, the conditional rescale and the fused cache update ("Update U_kv")
// are those of the two-tile kernel.  Every wait is bounded; a CTA that gives up raises its
// partner's abort flag too, and neither leaves before both have arrived at the final cluster
// barrier.  bf16 cache, d_k = 128, host-made plans, items without packing; everything else runs
// on the two-tile kernel.
#include <cuda.h>
#include <cuda_bf16.h>

#include "rpa_kernels.h"
#include "rpa_ptx.cuh"
#include "rpa_sm100.cuh"
#include "rpa_tile_common.cuh"

#ifndef RPA_PAIR_POLY
#define RPA_PAIR_POLY 0
#endif

namespace rpa {

using namespace sm100;

namespace {

constexpr int kBlockN = 128;       // KV positions per block
constexpr int kHalfN = 64;         // ... of which each CTA of the pair stages this many keys
constexpr int kBoxN = 32;          // ... as two runs of 32: keys [32r, 32r+32) and [64+32r, 64+32r+32) for CTA r (see the MMA issuer)
constexpr int kPairThreads = 384;  // 12 warps = 3 warpgroups per CTA
constexpr int kPairWarps = 2 * (kPairThreads / 32);
constexpr uint32_t kTmemCols = 512;
constexpr float kRescaleThreshold = 8.f;  // log2 units
constexpr int kFetchAhead = 3;     // the next item is drawn when the running one has this many key blocks to go
constexpr int D = 128;

struct PairCfg {
    static constexpr int NBLK = D / 64;              // 64-element (128-byte) column blocks per row
    static constexpr int BLK_BYTES = 128 * 128;      // one column block of a 128-row tile
    static constexpr int TILE_BYTES = NBLK * BLK_BYTES;
    static constexpr int HALF_BLK = kHalfN * 128;    // one column block of this CTA's 64 keys
    static constexpr int K_STAGE = NBLK * HALF_BLK;  // 64 keys x d_k
    static constexpr int V_STAGE = BLK_BYTES;        // 128 positions x this CTA's 64 columns of V
    static constexpr int KS = 2, VS = 2;             // ring depths
    static constexpr int OFF_Q = 0;                  // two buffers (items alternate) of two query tiles
    static constexpr int OFF_K = 4 * TILE_BYTES;
    static constexpr int OFF_V = OFF_K + KS * K_STAGE;
    static constexpr int OFF_UPD = OFF_V + VS * V_STAGE;  // staging of the fused cache update
    static constexpr int OFF_BAR = OFF_UPD + TileUpdate<D>::STAGE_BYTES;
    static constexpr int OFF_FLAGS = OFF_BAR + 256;  // abort flag, TMEM address, progress
    static constexpr int OFF_SLOTS = OFF_FLAGS + 64; // two item slots of RAW_INTS ints
    static constexpr int SMEM = OFF_SLOTS + 2 * RAW_INTS * 4 + 1024;  // + slack for 1024-byte alignment
    static_assert(SMEM <= 232448, "shared memory budget");
};

// barrier slots (8 bytes each), two of each kind.  Every CTA has all of them at the same offsets;
// QPEER/KPEER/VPEER, PREADY, SCONS and ITEMFREE are used in the first CTA only.
enum { BAR_Q = 0, BAR_QPEER = 2, BAR_QFREE = 4, BAR_KFULL = 6, BAR_KEMPTY = 8, BAR_VFULL = 10, BAR_VEMPTY = 12, BAR_KPEER = 14,
       BAR_VPEER = 16, BAR_SFULL = 18, BAR_PREADY = 20, BAR_ODONE = 22, BAR_SCONS = 24, BAR_EPI = 26, BAR_ITEM = 28,
       BAR_ITEMFREE = 30, BAR_COUNT = 32 };
static_assert(8 * BAR_COUNT <= 256, "barrier block");

template <int G>
__global__ void __launch_bounds__(kPairThreads, 1)
rpa_tile2_kernel(const KernelArgs a, const __grid_constant__ TileMaps maps) {
    using C = PairCfg;
    constexpr int TQ = 128 / G;  // tokens per query tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    const uint32_t bars = smem_base + C::OFF_BAR;
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_FLAGS);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + C::OFF_FLAGS + 8);
    // key blocks (counted across items) whose first PV product has been issued; written by the MMA warp
    volatile int* progress = reinterpret_cast<volatile int*>(smem + C::OFF_FLAGS + 16);
    volatile int* item_slots = reinterpret_cast<volatile int*>(smem + C::OFF_SLOTS);
    auto bar = [&](int slot) { return bars + 8u * slot; };

    if (a.validated && (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput)) return;  // inputs were rejected
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();  // 0: the CTA that issues the pair's products
    const bool first_cta = rank == 0;
    const uint32_t peer_abort = map_to_cta(smem_u32(const_cast<uint32_t*>(abort_flag)), rank ^ 1u);
    auto wait = [&](int slot, uint32_t parity, uint32_t code) {
        return mbar_wait_pair(bar(slot), parity, abort_flag, peer_abort, a.status, code);
    };
    auto first_cta_bar = [&](int slot) { return map_to_cta(bar(slot), 0u); };
    const int ps = a.page_size;
    const int n_items = a.num_tile_items;
    if (tid == 0) {
        *abort_flag = 0u;
        *progress = 0;
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar(BAR_Q + s), 1);
            mbar_init(bar(BAR_QPEER + s), 1);
            mbar_init(bar(BAR_QFREE + s), 8);  // the softmax warps of this CTA, after an item's epilogue
            mbar_init(bar(BAR_KFULL + s), 1);
            mbar_init(bar(BAR_KEMPTY + s), 1);
            mbar_init(bar(BAR_VFULL + s), 1);
            mbar_init(bar(BAR_VEMPTY + s), 1);
            mbar_init(bar(BAR_KPEER + s), 1);
            mbar_init(bar(BAR_VPEER + s), 1);
            mbar_init(bar(BAR_SFULL + s), 1);
            mbar_init(bar(BAR_PREADY + s), 8);  // one arrival per softmax warp of the tile, both CTAs
            mbar_init(bar(BAR_ODONE + s), 1);
            mbar_init(bar(BAR_SCONS + s), 8);   // the tile's softmax warps of both CTAs have taken S into registers
            mbar_init(bar(BAR_EPI + s), 128);
            mbar_init(bar(BAR_ITEM + s), 1);
            mbar_init(bar(BAR_ITEMFREE + s), kPairWarps);  // every warp of both CTAs has read the slot
        }
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_s[2] = {tmem_base, tmem_base + 128u};
    const uint32_t tm_o[2] = {tmem_base + 256u, tmem_base + 256u + D};

    // Item n of this pair lives in slot n & 1.  A warp takes it (all lanes together): waits until the
    // drawing warp has published it, reads it, and tells the drawing warp that this warp is done with
    // the slot.  Returns false when the wait gave up.
    auto take_item = [&](int n, TileCtx& it, int& item) -> bool {
        const bool ok = wait(BAR_ITEM + (n & 1), (n >> 1) & 1, 0x60);
        if (!__all_sync(0xffffffffu, ok)) return false;
        const volatile int* slot = item_slots + (n & 1) * RAW_INTS;
        item = slot[RAW_ITEM];
        if (item < n_items) it = tile_ctx_from_raw(a, slot, kBlockN);
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(first_cta_bar(BAR_ITEMFREE + (n & 1)));
        return true;
    };
    // this CTA's share of an item: its two query tiles' tokens
    auto own_tokens = [&](const TileCtx& it) { return max(0, min(2 * TQ, it.n_tok - (int)rank * 2 * TQ)); };
    // valid positions of key block j of an item (the rest of the block is masked for every row)
    auto valid_in_block = [&](const TileCtx& it, int j) {
        return j < it.n_ctx_blocks ? min(kBlockN, it.c - j * kBlockN) : min(kBlockN, it.n_new_visible - (j - it.n_ctx_blocks) * kBlockN);
    };
    // rows of this CTA's V stage past the block's valid positions may hold stale or foreign
    // data: make them finite (zero) so that masked probabilities (exactly 0) cannot produce NaN
    auto zero_v_tail = [&](int n_valid, int st) {
        if (n_valid < kBlockN) {
            uint8_t* v_s = smem + C::OFF_V + st * C::V_STAGE;
            for (int idx = lane; idx < (kBlockN - n_valid) * 8; idx += 32)
                *reinterpret_cast<uint4*>(v_s + (n_valid + idx / 8) * 128 + (idx % 8) * 16) = make_uint4(0, 0, 0, 0);
            fence_proxy_async_smem();
            __syncwarp();
        }
    };

    if (warp < 4) {
      // first warpgroup: producer, MMA issuer / relay, cache update and item drawing; it needs few registers
      asm volatile("setmaxnreg.dec.sync.aligned.u32 56;\n");
      if (warp == 0) {
        // ================================ TMA producer (each CTA: its own halves) ================================
        if (lane == 0) {
            prefetch_tmap(&maps.q);
            prefetch_tmap(&maps.out);
            prefetch_tmap(&maps.cache);
            prefetch_tmap(&maps.new_k);
            prefetch_tmap(&maps.new_v);
        }
        const int box_rows = page_box_rows(ps, kBoxN);
        int gb = 0;  // key blocks of earlier items: block j of the running item is fill gb + j of either ring
        bool ok = true;
        for (int n = 0; ok; ++n) {
            TileCtx it;
            int item;
            ok = take_item(n, it, item);
            if (!ok || item >= n_items) break;
            if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;
            const int h = it.h, cu = it.cu, c = it.c, n_ctx_blocks = it.n_ctx_blocks, n_blocks = it.n_blocks;
            const int32_t* pt_row = it.pt_row;
            // the item's query tiles, into the buffer the item before the last one has left
            if (n >= 2) ok = wait(BAR_QFREE + (n & 1), ((n >> 1) - 1) & 1, 0x15);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (lane == 0) {
                const uint32_t region = smem_base + C::OFF_Q + (n & 1) * 2 * C::TILE_BYTES, q_bar = bar(BAR_Q + (n & 1));
                const int tok_row = cu + it.q_tok0 + (int)rank * 2 * TQ;
                if (a.ablation & kAblateLoads) {
                    mbar_arrive(q_bar);
                } else {
                    mbar_arrive_expect_tx(q_bar, 2 * C::TILE_BYTES);  // (rows past the tensors read as zero and count)
                    for (int x = 0; x < 2; ++x)
#pragma unroll
                        for (int b = 0; b < C::NBLK; ++b)
                            tma_load_3d(region + x * C::TILE_BYTES + b * C::BLK_BYTES, &maps.q, b * 64, h * G, tok_row + x * TQ, q_bar);
                }
            }
            // fills the next stage of the K (kv = 0) or V (kv = 1) ring with this CTA's half of block j:
            // keys [64 rank, 64 rank + 64) of the block with all of d_k, or all 128 positions of V with
            // columns [64 rank, 64 rank + 64)
            auto fill = [&](int j, int kv) -> bool {
                const bool ctx = j < n_ctx_blocks;
                const int f = gb + j, st = f & 1;
                if (!debug_stage_ok(a, st, C::KS)) return false;
                const int rows = kv ? kBlockN : kHalfN;            // rows of the block this CTA stages
                const int boxes = rows / box_rows;
                // row of the block that lands in row lr of the stage: V takes the block as it is; the keys of
                // CTA r are the runs [32r, 32r + 32) and [64 + 32r, 64 + 32r + 32)
                const int lr = lane * box_rows;
                const int blk_row = kv ? lr : (lr / kBoxN) * kHalfN + (int)rank * kBoxN + lr % kBoxN;
                int page = 0, slot0 = 0;
                bool sub_valid = false;
                if (ctx) {
                    const int pos = j * kBlockN + blk_row;
                    sub_valid = lane < boxes && pos < c;
                    if (sub_valid) {
                        page = debug_read_page(a, pt_row[pos / ps]);
                        slot0 = pos % ps;
                    }
                }
                const int n_sub_valid = __popc(__ballot_sync(0xffffffffu, sub_valid));
                const uint32_t bytes = ctx ? (uint32_t)n_sub_valid * box_rows * 128u * (kv ? 1u : (uint32_t)C::NBLK)
                                           : (uint32_t)(kv ? C::V_STAGE : C::K_STAGE);
                const int full = (kv ? BAR_VFULL : BAR_KFULL) + st, empty = (kv ? BAR_VEMPTY : BAR_KEMPTY) + st;
                bool good = true;
                if (f >= 2) good = wait(empty, ((f >> 1) - 1) & 1, 0x10 + kv);
                good = __all_sync(0xffffffffu, good);
                if (!good) return false;
                const uint32_t dst = smem_base + (kv ? C::OFF_V + st * C::V_STAGE : C::OFF_K + st * C::K_STAGE);
                if (a.ablation & kAblateLoads) {
                    if (lane == 0) mbar_arrive(bar(full));
                    return true;
                }
                if (lane == 0) mbar_arrive_expect_tx(bar(full), bytes);  // (0 bytes: completes at once)
                __syncwarp();
                if (ctx) {
                    if (sub_valid) {
                        if (kv) {
                            tma_load_4d(dst + lane * box_rows * 128, &maps.cache, (int)rank * 64, 2 * h + 1, slot0, page, bar(full));
                        } else {
#pragma unroll
                            for (int b = 0; b < C::NBLK; ++b)
                                tma_load_4d(dst + b * C::HALF_BLK + lane * box_rows * 128, &maps.cache, b * 64, 2 * h, slot0, page, bar(full));
                        }
                    }
                } else if (lane == 0) {
                    const int new_row0 = cu + (j - n_ctx_blocks) * kBlockN;
                    if (kv) {
#pragma unroll
                        for (int i = 0; i < kBlockN / kBoxN; ++i)
                            tma_load_3d(dst + i * kBoxN * 128, &maps.new_v, (int)rank * 64, h, new_row0 + i * kBoxN, bar(full));
                    } else {
#pragma unroll
                        for (int b = 0; b < C::NBLK; ++b)
#pragma unroll
                            for (int run = 0; run < 2; ++run)
                                tma_load_3d(dst + b * C::HALF_BLK + run * kBoxN * 128, &maps.new_k, b * 64, h,
                                            new_row0 + run * kHalfN + (int)rank * kBoxN, bar(full));
                    }
                }
                return true;
            };
            // the keys run one block ahead of the values (a V stage is held through its block's whole softmax)
            for (int t = 0; t <= n_blocks && ok; ++t) {
                if (t < n_blocks) ok = fill(t, 0);
                if (ok && t >= 1) ok = fill(t - 1, 1);
            }
            gb += n_blocks;
        }
        // every completion signal of the products has reached this CTA before it leaves
#pragma unroll
        for (int st = 0; st < 2; ++st) {
            const int uses = (gb + 1 - st) >> 1;  // fills that went through stage st
            if (uses > 0 && ok) ok = wait(BAR_KEMPTY + st, (uses - 1) & 1, 0x13);
            if (uses > 0 && ok) ok = wait(BAR_VEMPTY + st, (uses - 1) & 1, 0x14);
        }
      } else if (warp == 1 && !first_cta) {
        // ================================ second CTA: relay "my half has landed" ================================
        int gb = 0;
        bool ok = true;
        for (int n = 0; ok; ++n) {
            TileCtx it;
            int item;
            ok = take_item(n, it, item);
            if (!ok || item >= n_items) break;
            if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;
            const int n_blocks = it.n_blocks;
            ok = wait(BAR_Q + (n & 1), (n >> 1) & 1, 0x28);
            if (ok && lane == 0) mbar_arrive_cluster(first_cta_bar(BAR_QPEER + (n & 1)));
            for (int t = 0; t <= n_blocks && ok; ++t) {
                if (t < n_blocks) {
                    const int f = gb + t;
                    ok = wait(BAR_KFULL + (f & 1), (f >> 1) & 1, 0x29);
                    if (ok && lane == 0) mbar_arrive_cluster(first_cta_bar(BAR_KPEER + (f & 1)));
                }
                if (ok && t >= 1) {
                    const int f = gb + t - 1, n_valid = valid_in_block(it, t - 1);
                    ok = wait(BAR_VFULL + (f & 1), (f >> 1) & 1, 0x2A);
                    if (ok) {
                        zero_v_tail(n_valid, f & 1);
                        if (lane == 0) {
                            if (n_valid < kBlockN) {
                                mbar_arrive_cluster_release(first_cta_bar(BAR_VPEER + (f & 1)));  // the zeroed rows count
                            } else {
                                mbar_arrive_cluster(first_cta_bar(BAR_VPEER + (f & 1)));
                            }
                        }
                    }
                }
            }
            gb += n_blocks;
        }
      } else if (warp == 1) {
        // ================================ MMA issuer (first CTA, for the pair) ================================
        constexpr uint32_t idesc_qk = instr_desc_bf16(256, kBlockN / 2, 0, 0);
        constexpr uint32_t idesc_pv = instr_desc_bf16(256, D, 0, 1);
        constexpr uint32_t desc_hi = smem_desc_sw128_hi(1024);
        const uint32_t k_lo = smem_desc_sw128_lo(smem_base + C::OFF_K, 16);
        const uint32_t v_lo = smem_desc_sw128_lo(smem_base + C::OFF_V, C::BLK_BYTES);
        const bool no_compute = a.ablation & kAblateCompute;  // bench switch: commits without products
        // The scores of a block are made by two products of 64 keys each: columns [0, 64) of S ("low":
        // keys 0..63 of the block - run 0 of both CTAs' stages) and columns [64, 128) ("high").  The
        // probabilities of block j go into the HIGH columns, so the low product of block j+1 does not
        // have to wait for P_j V_j: it is issued as soon as the softmax warps have taken S_j into their
        // registers, and runs while they work; only the high product stands behind P_j V_j in the
        // tile's chain of dependencies (P ready -> PV -> scores -> softmax), 8 products of 64 keys
        // instead of 8 of 128.
        // S_x[:, 64 half ..] = Q_x K^T over d_k in steps of 16, tile x of both CTAs; queries of item n, keys in stage st
        auto issue_qk = [&](int n, int x, int st, int half) {
            if (no_compute) return;
            const uint32_t ql = smem_desc_sw128_lo(smem_base + C::OFF_Q + ((n & 1) * 2 + x) * C::TILE_BYTES, 16);
            const uint32_t kl = k_lo + ((st * C::K_STAGE + half * kBoxN * 128) >> 4);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint32_t q_off = ((ks / 4) * C::BLK_BYTES + (ks % 4) * 32) >> 4;
                const uint32_t k_off = ((ks / 4) * C::HALF_BLK + (ks % 4) * 32) >> 4;
                umma_ss_pair(tm_s[x] + half * 64, make_desc(ql + q_off, desc_hi), make_desc(kl + k_off, desc_hi), idesc_qk, ks > 0);
            }
        };
        auto issue_pv = [&](int x, int st, bool first) {  // O_x (+)= P_x V over 128 positions in steps of 16
            if (no_compute) return;
            const uint32_t vl = v_lo + st * (C::V_STAGE >> 4);
#pragma unroll
            for (int kk = 0; kk < kBlockN / 16; ++kk)
                umma_ts_pair(tm_o[x], tm_s[x] + 64 + kk * 8, make_desc(vl + kk * (2048 >> 4), desc_hi), idesc_pv, !(first && kk == 0));
        };
        auto q_landed = [&](int n) {
            return wait(BAR_Q + (n & 1), (n >> 1) & 1, 0x20) && wait(BAR_QPEER + (n & 1), (n >> 1) & 1, 0x21);
        };
        auto k_landed = [&](int f, uint32_t code) {  // fill f of the K ring, both halves
            return wait(BAR_KFULL + (f & 1), (f >> 1) & 1, code) && wait(BAR_KPEER + (f & 1), (f >> 1) & 1, code + 1);
        };
        int gb = 0;
        TileCtx it, nxt;
        int item, nxt_item = n_items;
        bool ok = take_item(0, it, item);
        if (ok && item < n_items && debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) {
            // the first item's first block; every later one is issued behind its predecessor's products
            ok = q_landed(0) && k_landed(0, 0x22);
            if (ok) {
                tc_fence_after();
                if (elect_one()) {
                    issue_qk(0, 0, 0, 0);
                    issue_qk(0, 0, 0, 1);
                    tc_commit_pair(bar(BAR_SFULL + 0));
                }
                __syncwarp();
                if (elect_one()) {
                    issue_qk(0, 1, 0, 0);
                    issue_qk(0, 1, 0, 1);
                    tc_commit_pair(bar(BAR_SFULL + 1));
                    tc_commit_pair(bar(BAR_KEMPTY + 0));
                }
                __syncwarp();
            }
            for (int n = 0; ok; ++n) {
                const int n_blocks = it.n_blocks;
                bool have_next = false, looked = false;
                for (int j = 0; j < n_blocks && ok; ++j) {
                    const int f = gb + j, st = f & 1, ph = (f >> 1) & 1;
                    ok = wait(BAR_VFULL + st, ph, 0x24);
                    if (!ok) break;
                    zero_v_tail(valid_in_block(it, j), st);
                    ok = wait(BAR_VPEER + st, ph, 0x25);
                    if (!ok) break;
                    const bool last = j + 1 == n_blocks;
                    if (last && !looked) {  // what follows this item?  (drawn by now: the drawing warp watches `progress`)
                        looked = true;
                        ok = take_item(n + 1, nxt, nxt_item);
                        if (!ok) break;
                        have_next = nxt_item < n_items && debug_rows_ok(a, (long long)nxt.cu + nxt.q_tok0, nxt.n_tok);
                    }
                    // the next score products: the item's next block, or the next item's first one
                    const bool more = !last || have_next;
                    const int f1 = f + 1, st1 = f1 & 1, n1 = last ? n + 1 : n;
                    if (more) {  // low half of tile A's next scores: S_A of this block is in the softmax warps' registers
                        if (last) ok = q_landed(n + 1);
                        ok = ok && k_landed(f1, 0x2C) && wait(BAR_SCONS + 0, f & 1, 0x2E);
                        if (!ok) break;
                        tc_fence_after();
                        if (elect_one()) issue_qk(n1, 0, st1, 0);
                        __syncwarp();
                    }
                    ok = wait(BAR_PREADY + 0, f & 1, 0x26);
                    if (!ok) break;
                        tc_fence_after();
                    if (elect_one()) {
                        issue_pv(0, st, j == 0);
                        tc_commit_pair(bar(BAR_ODONE + 0));
                        *progress = f + 1;
                        if (more) {
                            issue_qk(n1, 0, st1, 1);
                            tc_commit_pair(bar(BAR_SFULL + 0));
                        }
                    }
                    __syncwarp();
                    if (more) {  // low half of tile B's next scores
                        ok = wait(BAR_SCONS + 1, f & 1, 0x2F);
                        if (!ok) break;
                        tc_fence_after();
                        if (elect_one()) issue_qk(n1, 1, st1, 0);
                        __syncwarp();
                    }
                    ok = wait(BAR_PREADY + 1, f & 1, 0x27);
                    if (!ok) break;
                        tc_fence_after();
                    if (elect_one()) {
                        issue_pv(1, st, j == 0);
                        tc_commit_pair(bar(BAR_ODONE + 1));
                        tc_commit_pair(bar(BAR_VEMPTY + st));
                        if (more) {
                            issue_qk(n1, 1, st1, 1);
                            tc_commit_pair(bar(BAR_SFULL + 1));
                            tc_commit_pair(bar(BAR_KEMPTY + st1));
                        }
                    }
                    __syncwarp();
                }
                gb += n_blocks;
                if (!have_next) break;
                it = nxt;
            }
        }
      } else {
        // ================================ fused cache update (each CTA: its own tokens); item drawing ================================
        // Warp 3 of the first CTA draws the pair's items - the next one once the running one is within
        // a few key blocks of its end, so that no long item is reserved early - and writes each entry
        // into both CTAs' slots.
        auto publish = [&](int n, int fallback) {  // whole warp
            bool ok = true;
            if (n >= 2) ok = wait(BAR_ITEMFREE + (n & 1), ((n >> 1) - 1) & 1, 0x61);
            if (!__all_sync(0xffffffffu, ok)) return false;
            volatile int* slot = item_slots + (n & 1) * RAW_INTS;
            draw_and_fetch_tile(a, true, fallback, slot, lane);
            __syncwarp();
            if (lane == 0) {
                // the second CTA gets its copy from the copy engine, which counts the bytes at that CTA's
                // barrier (a releasing arrival across the pair costs as much as a device-wide fence)
                const uint32_t src = smem_u32(const_cast<int*>(slot)), remote_bar = map_to_cta(bar(BAR_ITEM + (n & 1)), 1u);
                fence_proxy_async_smem();
                mbar_arrive_expect_tx_cluster(remote_bar, RAW_INTS * 4);
                bulk_copy_to_cta(map_to_cta(src, 1u), src, RAW_INTS * 4, remote_bar);
                mbar_arrive(bar(BAR_ITEM + (n & 1)));
            }
            __syncwarp();
            return true;
        };
        const bool drawer = warp == 3 && first_cta;
        int gb = 0;
        bool ok = true;
        if (drawer) ok = publish(0, 0);
        for (int n = 0; ok; ++n) {
            TileCtx it;
            int item;
            ok = take_item(n, it, item);
            if (!ok || item >= n_items) break;
            if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;
            // a short item's successor is drawn before this warp's share of the update (which takes longer
            // than such an item runs), a long item's once it is within a few blocks of its end
            const bool draw_first = it.n_blocks <= kFetchAhead;
            if (drawer && draw_first) ok = publish(n + 1, n_items);
            if (ok && !(a.ablation & kAblateUpdate) && (it.flags & kFlagWriteKv)) {
                TileCtx own = it;
                own.q_tok0 = it.q_tok0 + (int)rank * 2 * TQ;
                own.n_tok = own_tokens(it);
                tile_update_cache<D>(a, own, warp - 2, lane, smem_base + C::OFF_UPD);
            }
            if (drawer && ok && !draw_first) {
                if (lane == 0) {
                    const long long t0 = clock64();
                    while (*progress < gb + it.n_blocks - kFetchAhead && !*abort_flag && clock64() - t0 < 4000000000LL) __nanosleep(256);
                }
                __syncwarp();
                ok = publish(n + 1, n_items);
            }
            gb += it.n_blocks;
        }
      }
    } else {
        // ================================ softmax warps ================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;\n");
        const int x = (warp - 4) >> 2;              // 0: tile A, 1: tile B
        const int quarter = warp & 3;               // TMEM lanes this warp may touch: 32*quarter ..
        const int row = quarter * 32 + lane;        // query row of this thread inside its tile
        const int tok_in_tile = row / G, g = row % G;
        const int tok_in_item = ((int)rank * 2 + x) * TQ + tok_in_tile;
        const uint32_t lane_sel = (uint32_t)(quarter * 32) << 16;
        const uint32_t s_addr = tm_s[x] + lane_sel, o_addr = tm_o[x] + lane_sel;
        const uint32_t pready = first_cta ? bar(BAR_PREADY + x) : first_cta_bar(BAR_PREADY + x);
        const uint32_t scons = first_cta ? bar(BAR_SCONS + x) : first_cta_bar(BAR_SCONS + x);
        int gb = 0, epi_uses = 0;
        bool ok = true;
        for (int n = 0; ok; ++n) {
        TileCtx it;
        int item;
        ok = take_item(n, it, item);
        if (!ok || item >= n_items) break;
        if (!debug_rows_ok(a, (long long)it.cu + it.q_tok0, it.n_tok)) break;
        const int h = it.h, cu = it.cu, q_r = it.q_r, L = it.L, c = it.c;
        const int n_ctx_blocks = it.n_ctx_blocks, n_new_visible = it.n_new_visible, n_blocks = it.n_blocks;
        const uint32_t q_region = smem_base + C::OFF_Q + (n & 1) * 2 * C::TILE_BYTES;
        const int tok = it.q_tok0 + tok_in_item;    // token index inside the sequence
        const bool row_valid = tok_in_item < it.n_tok;
        const int lim = a.causal ? c + min(tok, q_r - 1) : L - 1;  // last visible key position of this row

        float m_ref = -INFINITY, l_sum = 0.f;
        for (int j = 0; j < n_blocks; ++j) {
            const int f = gb + j;
            ok = wait(BAR_SFULL + x, f & 1, 0x30 + x);
            if (!ok) break;
            tc_fence_after();
            if (a.ablation & kAblateCompute) {  // bench switch: hand over at once
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_cluster(scons);
                    mbar_arrive_cluster(pready);
                }
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
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(scons);  // the low columns of S may be overwritten with the next block's scores
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
            float mxp[8];  // independent partial maxima: no 128-long dependency chain
#pragma unroll
            for (int i = 0; i < 8; ++i) mxp[i] = fmaxf(s[i], s[i + 8]);
#pragma unroll
            for (int i = 16; i < kBlockN; i += 16)
#pragma unroll
                for (int k = 0; k < 8; ++k) mxp[k] = max3(mxp[k], s[i + k], s[i + k + 8]);
            const float mx = fmaxf(max3(mxp[0], mxp[1], mxp[2]), max3(fmaxf(mxp[3], mxp[4]), max3(mxp[5], mxp[6], mxp[7]), -INFINITY));
            const float mx2 = mx * a.scale_log2;
            if (j == 0) {
                m_ref = mx2;
            } else {
                const bool grow = mx2 - m_ref > kRescaleThreshold;
                if (__any_sync(0xffffffffu, grow)) {
                    // the previous PV product of this tile must have landed before O is touched
                    ok = wait(BAR_ODONE + x, (f - 1) & 1, 0x32 + x);
                    if (!ok) break;
                    tc_fence_after();
                    const float fs = grow ? fast_exp2(m_ref - mx2) : 1.f;
#pragma unroll
                    for (int ch = 0; ch < D / 32; ++ch) {
                        uint32_t r32[32];
                        tmem_ld32(o_addr + ch * 32, r32);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r32[i] = __float_as_uint(__uint_as_float(r32[i]) * fs);
                        tmem_st32(o_addr + ch * 32, r32);
                    }
                    l_sum *= fs;
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
                    float x0, x1;
                    fma2_bcast(x0, x1, s[ch * 64 + 2 * i], s[ch * 64 + 2 * i + 1], a.scale_log2, neg_m);
                    const bool poly = RPA_PAIR_POLY && (i & 3) == 3;
                    const float p0 = poly ? poly_exp2(x0) : fast_exp2(x0), p1 = poly ? poly_exp2(x1) : fast_exp2(x1);
                    add2(lp[2 * (i & 3)], lp[2 * (i & 3) + 1], p0, p1);
                    p32[i] = pack_bf16x2(p0, p1);
                }
                tmem_st32(s_addr + 64 + ch * 32, p32);  // (the high columns: see the MMA issuer)
            }
            l_sum += ((lp[0] + lp[1]) + (lp[2] + lp[3])) + ((lp[4] + lp[5]) + (lp[6] + lp[7]));
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(pready);  // one arrival per warp, at the first CTA's barrier
        }
        // ---- epilogue: O / l -> bf16 -> out ----
        if (ok && n_blocks > 0) ok = wait(BAR_ODONE + x, (gb + n_blocks - 1) & 1, 0x34 + x);
        if (ok && n_blocks > 0 && !(a.ablation & kAblateCompute)) {
            tc_fence_after();
            const float inv = a.out_scale / l_sum;
            if (((int)rank * 2 + x + 1) * TQ <= it.n_tok) {
                // A full tile goes out through shared memory: each thread parks its row in the
                // tile's Q buffer (free since the item's last score product completed) in the swizzled
                // layout of the tensor map, and one thread stores the tile with the copy engine.
                const uint32_t q_buf = q_region + x * C::TILE_BYTES;
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
                if (row == 0) {
                    if (wait(BAR_EPI + x, epi_uses & 1, 0x36 + x)) {
#pragma unroll
                        for (int b = 0; b < C::NBLK; ++b)
                            tma_store_3d(&maps.out, q_buf + b * C::BLK_BYTES, b * 64, h * G, cu + it.q_tok0 + ((int)rank * 2 + x) * TQ);
                        bulk_commit();
                        bulk_wait_read();  // the Q buffer is loaded again two items later
                    }
                }
                ++epi_uses;
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
        // this warp is done with the item's query buffer (the producer loads the item after next into it)
        // and with the accumulator (the next item's first PV product overwrites it once this warp has
        // handed over that item's first probabilities)
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(BAR_QFREE + (n & 1)));
        gb += n_blocks;
        }  // item loop of the softmax warpgroups
    }
    // ---- teardown: both CTAs arrive, then each frees its half of the pair's TMEM allocation ----
    tc_fence_before();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
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

// launch configuration of `pairs` clusters of two CTAs
struct PairLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr;
    PairLaunch(int pairs, cudaStream_t stream) : cfg{}, attr{} {
        cfg.gridDim = dim3(2 * pairs, 1, 1);
        cfg.blockDim = dim3(kPairThreads, 1, 1);
        cfg.dynamicSmemBytes = PairCfg::SMEM;
        cfg.stream = stream;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
    }
    PairLaunch(const PairLaunch&) = delete;
};

// pairs the device can hold at once (an SM whose neighbour is taken cannot host half a pair)
template <int G>
int resident_pairs() {
    static int pairs = -1;
    if (pairs < 0) {
        PairLaunch l(148, nullptr);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, rpa_tile2_kernel<G>, &l.cfg) != cudaSuccess || n < 1) {
            (void)cudaGetLastError();
            n = 1;
        }
        pairs = n;
    }
    return pairs;
}

template <int G>
cudaError_t launch_tile2(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    TileMaps maps;
    if (!cached_tile_maps(cache, a, token_rows, D, G, 128 / G, kBoxN, &maps)) return cudaErrorInvalidValue;
    int pairs = resident_pairs<G>();
    if (a.num_tile_ctas > 0) pairs = min(pairs, max(1, a.num_tile_ctas / 2));
    pairs = min(pairs, a.num_tile_items);
    PairLaunch l(pairs, stream);
    return cudaLaunchKernelEx(&l.cfg, rpa_tile2_kernel<G>, a, maps);
}

template <int G>
cudaError_t prepare_tile2() {
    return cudaFuncSetAttribute(rpa_tile2_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg::SMEM);
}

#define RPA_TILE2_DISPATCH(G_, FN, ...)              \
    do {                                             \
        switch (G_) {                                \
            case 1: return FN<1>(__VA_ARGS__);       \
            case 2: return FN<2>(__VA_ARGS__);       \
            case 4: return FN<4>(__VA_ARGS__);       \
            case 8: return FN<8>(__VA_ARGS__);       \
            case 16: return FN<16>(__VA_ARGS__);     \
        }                                            \
    } while (0)

}  // namespace

bool tile2_kernel_supported(int head_dim, int group) {
    return head_dim == 128 && (group == 1 || group == 2 || group == 4 || group == 8 || group == 16);
}

int tile2_kernel_tokens(int group) { return 4 * (128 / group); }

cudaError_t tile2_kernel_prepare(int group) {
    RPA_TILE2_DISPATCH(group, prepare_tile2);
    return cudaErrorInvalidValue;
}

cudaError_t launch_tile2_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream) {
    if (a.num_tile_items <= 0) return cudaSuccess;
    if (a.dev_counts || a.kv_fp8 || a.head_dim != D) return cudaErrorInvalidValue;
    RPA_TILE2_DISPATCH(a.h_q / a.h_kv, launch_tile2, a, token_rows, cache, stream);
    return cudaErrorInvalidValue;
}

}  // namespace rpa
