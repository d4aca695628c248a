// Pieces shared by the tensor-core tile kernels: tensor maps, per-item context.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <string.h>

#include "rpa_fp8.cuh"
#include "rpa_kernels.h"
#include "rpa_ptx.cuh"
#include "rpa_sm100.cuh"

namespace rpa {

constexpr int kUpdBoxes = 6;  // slot counts 1, 2, ..., 32 of one store of the fused cache update

struct TileMaps {
    CUtensorMap q;      // (d, h_q, T)     box (64, G, query-tile tokens)
    CUtensorMap out;    // same geometry as q
    CUtensorMap new_k;  // (d, h_kv, T)    box (64, 1, key-block positions)
    CUtensorMap new_v;
    CUtensorMap cache;  // (d, 2h_kv, page_size, num_pages)  box (64, 1, page_box_rows(page_size, key-block positions), 1)
    // fused cache update of a bf16 cache (whole rows, no swizzle): see tile_update_rounds_tma
    CUtensorMap upd_k;  // (d, h_kv, T)    box (d, 1, TileUpdate<d>::TPW)
    CUtensorMap upd_v;
    CUtensorMap upd_cache[kUpdBoxes];  // (d, 2h_kv, page_size, num_pages)  box (d, 1, 1 << i, 1)
};

// Rows of one per-page TMA box of a context key block.  A block of block_n positions is fetched as
// block_n / rows boxes, each starting at a position that is a multiple of `rows`; `rows` divides
// both the page size and the block, so no box straddles a page whatever the page size is (48, 96,
// 192, ... included): the largest power of two that divides page_size, capped at the block.
__host__ __device__ __forceinline__ int page_box_rows(int page_size, int block_n) {
    const int pow2 = page_size & -page_size;
    return pow2 < block_n ? pow2 : block_n;
}

// Everything a role needs to know about one work item.
struct TileCtx {
    int seq, h, q_tok0, n_tok, flags;
    int cu, q_r, L, c;
    int n_ctx_blocks, n_new_visible, n_blocks;
    int n_seqs;                  // > 1: a packed item (several whole sequences without context)
    const volatile int* bounds;  // shared memory: token offsets of the item's sequences, bounds[0] = 0 .. bounds[n_seqs]
    const int32_t* pt_row;
};

// The item's list entry and its sequences' lengths, as one warp fetches them (a chain of two
// dependent global loads) and parks them in shared memory for the whole CTA.
enum { RAW_ITEM = 0, RAW_SEQ, RAW_HEAD, RAW_TOK0, RAW_NTOK, RAW_FLAGS, RAW_NSEQ, RAW_CU, RAW_L, RAW_BOUNDS = 16,
       RAW_INTS = 96 };
static_assert(RAW_BOUNDS + kMaxPackedSeqs + 1 <= RAW_INTS, "slot holds the bounds of a packed item");
constexpr int kTileBarBlockBytes = 256 + 2 * RAW_INTS * 4;  // mbarriers and flags, then two item slots

// Length of the tile item list: a launch argument, or, for lists planned on the device, a word the
// plan kernel of the same step wrote.
__device__ __forceinline__ int tile_item_count(const KernelArgs& a) {
    return a.dev_counts ? a.dev_counts[kDevCountTiles] : a.num_tile_items;
}

// Called by all 32 lanes of a warp with the same `item`.
__device__ __forceinline__ void fetch_tile_raw(const KernelArgs& a, int item, volatile int* slot, int lane) {
    if (lane == 0) slot[RAW_ITEM] = item;
    if (item >= tile_item_count(a)) return;
    const TileItem it = a.tile_items[item];
    const int m = (it.flags & kFlagPacked) ? it.n_seqs : 1;
    const int cu = a.cu_q_lens[it.seq];
    if (lane == 0) {
        slot[RAW_SEQ] = it.seq;
        slot[RAW_HEAD] = it.kv_head;
        slot[RAW_TOK0] = it.q_tok0;
        slot[RAW_NTOK] = it.n_tok;
        slot[RAW_FLAGS] = it.flags;
        slot[RAW_NSEQ] = m;
        slot[RAW_CU] = cu;
        slot[RAW_L] = a.kv_lens[it.seq];
    }
    for (int k = lane; k <= m; k += 32) slot[RAW_BOUNDS + k] = a.cu_q_lens[it.seq + k] - cu;
}

// Draws the next item (persistent CTAs: from the device-wide counter) and fetches it; whole warp.
__device__ __forceinline__ void draw_and_fetch_tile(const KernelArgs& a, bool persistent, int fallback_item, volatile int* slot,
                                                    int lane) {
    int item = fallback_item;
    if (persistent) {
        if (lane == 0) item = atomicAdd(a.tile_counters, 1);
        item = __shfl_sync(0xffffffffu, item, 0);
    }
    fetch_tile_raw(a, item, slot, lane);
}

__device__ __forceinline__ TileCtx tile_ctx_from_raw(const KernelArgs& a, const volatile int* slot, int block_n) {
    TileCtx t;
    t.seq = slot[RAW_SEQ];
    t.h = slot[RAW_HEAD];
    t.q_tok0 = slot[RAW_TOK0];
    t.n_tok = slot[RAW_NTOK];
    t.flags = slot[RAW_FLAGS];
    t.n_seqs = slot[RAW_NSEQ];
    t.bounds = slot + RAW_BOUNDS;
    t.cu = slot[RAW_CU];
    // a packed item looks like one sequence of n_tok new tokens without context; which keys a row
    // may see inside it is decided per row from `bounds`
    t.q_r = t.n_seqs > 1 ? t.n_tok : slot[RAW_BOUNDS + 1];
    t.L = t.n_seqs > 1 ? t.n_tok : slot[RAW_L];
    t.c = t.L - t.q_r;
    t.pt_row = a.page_table + (int64_t)t.seq * a.max_pages_per_seq;
    // key blocks: cached context [0, c), then the new tokens this item may see
    t.n_ctx_blocks = (t.c + block_n - 1) / block_n;
    t.n_new_visible = a.causal ? min(t.q_r, t.q_tok0 + t.n_tok) : t.q_r;
    t.n_blocks = t.n_ctx_blocks + (t.n_new_visible + block_n - 1) / block_n;
    return t;
}

// Sequence of a packed item that token `tok` (offset inside the item) belongs to.
__device__ __forceinline__ int packed_seq_of(const TileCtx& it, int tok) {
    int lo = 0, hi = it.n_seqs - 1;  // largest k with bounds[k] <= tok
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (it.bounds[mid] <= tok) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Fused cache update of an item ("Update U_kv" of Algorithm 1): the K and V rows of the item's own
// tokens for its KV head go into their cache slots, a round of TPW tokens at a time.  The rows of a
// round are fetched into shared memory with 16-byte asynchronous copies (one instruction moves 512
// bytes for the warp and does not block it), a token's K row and V row side by side as in a cache
// slot, and leave with one bulk store per token (lane t sends token t).  (An earlier version moved
// the rows in both directions with per-thread bulk copies: the copy engine takes such copies one
// thread at a time, about 60 cycles each - 192 of them per 64 tokens, which is what an item of a
// short prompt then cost; 16-byte stores on the way out cost a shuffle, a shared-memory load and a
// store per 512 bytes, more than the 32 bulk stores of a round.)  BUFS: staging buffers of
// WARP_BYTES each; with two, the next round's rows travel while this round's are written.
template <int D>
struct TileUpdate {
    static constexpr int ROW_BYTES = D * 2;                       // one K or V row of one head
    static constexpr int TPW = 8192 / ROW_BYTES < 32 ? 8192 / ROW_BYTES : 32;  // tokens per round
    static constexpr int WARP_BYTES = TPW * 2 * ROW_BYTES;
    static constexpr int STAGE_BYTES = 2 * WARP_BYTES;
};

// Rounds t_first, t_first + t_step, ... (token offsets inside the item) by one warp.  The warps of
// the first warpgroup get an issue slot every few cycles only (the softmax warps own the schedulers),
// so the loops below are kept to a handful of instructions per 512 bytes moved.
template <int D, int BUFS>
__device__ __forceinline__ void tile_update_rounds(const KernelArgs& a, const TileCtx& it, int t_first, int t_step, int lane, uint32_t stage) {
    using U = TileUpdate<D>;
    constexpr int ROW = U::ROW_BYTES, TPW = U::TPW, CPT = 2 * ROW / 16, HALF = CPT / 2;  // 16-byte pieces per token: K row, then V row
    constexpr int STEPS = TPW * CPT / 32;                                                // warp-wide instructions per full round
    static_assert(BUFS == 1 || BUFS == 2, "one or two staging buffers");
    static_assert((CPT & (CPT - 1)) == 0 && TPW * CPT % 32 == 0, "pieces per token: a power of two");
    const int ps = a.page_size;
    uint8_t* cache = reinterpret_cast<uint8_t*>(a.kv_cache);
    const int64_t tok_stride = (int64_t)a.h_kv * D;  // elements from one token's row to the next
    // writes a landed round out of its buffer; slot: this lane's token's cache slot in units of ROW
    // bytes (~0: none)
    auto write_out = [&](uint32_t buf, int nt, uint32_t slot) {
        __syncwarp();                    // every lane's pieces have landed (each waited for its own copies)
        sm100::fence_proxy_async_smem(); // ... and are visible to the copy engine
        if (lane < nt && slot != ~0u) sm100::bulk_store(cache + (int64_t)slot * ROW, buf + lane * 2 * ROW, 2 * ROW);
        sm100::bulk_commit();
        sm100::bulk_wait_read();         // the buffer may be refilled
        __syncwarp();
    };
    int r = 0, prev_nt = 0;
    uint32_t prev_slot = ~0u;
    for (int t0 = t_first;; t0 += t_step, ++r) {
        const bool have = t0 < it.n_tok;
        const uint32_t buf = stage + (r % BUFS) * U::WARP_BYTES;
        int nt = 0;
        uint32_t slot = ~0u;
        if (have) {
            nt = min(TPW, it.n_tok - t0);
            const bool act = lane < nt;
            const int tok = it.q_tok0 + t0 + lane;
            int pos = it.c + tok;
            const int32_t* pt_row = it.pt_row;
            if (it.n_seqs > 1 && act) {  // packed item: the token's own sequence, page-table row and position
                const int k = packed_seq_of(it, tok);
                pos = tok - it.bounds[k];
                pt_row += (int64_t)k * a.max_pages_per_seq;
            }
            const int page = act ? pt_row[pos / ps] : 0;
            if (act && debug_write_page_ok(a, page))  // (always true for a token of the round outside the bounds-checked build)
                slot = (uint32_t)(((int64_t)page * ps + pos % ps) * 2 * a.h_kv + 2 * it.h);
            const uint16_t* row0 = a.new_k + (((int64_t)it.cu + it.q_tok0 + t0) * a.h_kv + it.h) * D;  // token 0 of the round, K
            const int64_t v_minus_k = a.new_v - a.new_k;
#pragma unroll 4
            for (int s = 0; s < STEPS; ++s) {
                const int idx = s * 32 + lane, t = idx / CPT, piece = idx % CPT;
                const uint16_t* src = row0 + t * tok_stride + (piece % HALF) * 8 + (piece < HALF ? 0 : v_minus_k);
                if (t < nt) cp_async_16(buf + idx * 16, src, 16);
            }
            cp_async_commit();
        }
        if (BUFS == 1) {
            if (!have) break;
            cp_async_wait<0>();
            write_out(buf, nt, slot);
        } else {
            if (prev_nt > 0) {  // the round before has landed (all but the group just committed are complete)
                if (have) cp_async_wait<1>(); else cp_async_wait<0>();
                write_out(stage + ((r - 1) % BUFS) * U::WARP_BYTES, prev_nt, prev_slot);
            }
            if (!have) break;
            prev_nt = nt, prev_slot = slot;
        }
    }
}

// The same update with the copy engine doing all of it (bf16 cache): a round's K rows and V rows come
// in as two boxes of TPW rows each (dense, K rows at `stage`, V rows behind them) and leave as a few
// tiled stores.  The tokens of a round have consecutive positions, so they fall into runs that share
// a page; a run of n slots goes out as one store per set bit of n (the largest first), K and V
// apart - at a page size of 16, six to twelve stores a round where a store per token makes 32, and
// two loads where 16-byte copies make 32 instructions.  `bar`: this warp's mbarrier (one arrival),
// `parity` its running phase; `wait(bar, parity)` returns false when the kernel is being abandoned.
template <int D, class Wait>
__device__ __forceinline__ void tile_update_rounds_tma(const KernelArgs& a, const TileMaps& maps, const TileCtx& it, int t_first,
                                                       int t_step, int lane, uint32_t stage, uint32_t bar, uint32_t& parity, Wait&& wait) {
    using U = TileUpdate<D>;
    constexpr int ROW = U::ROW_BYTES, TPW = U::TPW;
    const int ps = a.page_size;
    for (int t0 = t_first; t0 < it.n_tok; t0 += t_step) {
        const int nt = min(TPW, it.n_tok - t0);
        if (lane == 0) {
            // (rows past the item's last token travel too and are not stored; past the tensor they read as zero)
            sm100::mbar_arrive_expect_tx(bar, 2 * TPW * ROW);
            sm100::tma_load_3d(stage, &maps.upd_k, 0, it.h, it.cu + it.q_tok0 + t0, bar);
            sm100::tma_load_3d(stage + TPW * ROW, &maps.upd_v, 0, it.h, it.cu + it.q_tok0 + t0, bar);
        }
        const bool act = lane < nt;
        const int tok = it.q_tok0 + t0 + lane;
        int pos = it.c + tok;
        const int32_t* pt_row = it.pt_row;
        if (it.n_seqs > 1 && act) {  // packed item: the token's own sequence, page-table row and position
            const int k = packed_seq_of(it, tok);
            pos = tok - it.bounds[k];
            pt_row += (int64_t)k * a.max_pages_per_seq;
        }
        const int page = act ? pt_row[pos / ps] : -1;
        const bool valid = act && debug_write_page_ok(a, page);  // (always true for a token of the round outside the bounds-checked build)
        // runs of tokens in one page: a run starts where the page changes (sequences share no page)
        const int page_before = __shfl_up_sync(0xffffffffu, page, 1);
        const bool valid_before = __shfl_up_sync(0xffffffffu, (int)valid, 1) != 0;
        const uint32_t starts = __ballot_sync(0xffffffffu, !valid || lane == 0 || !valid_before || page != page_before);
        int log_n = -1;  // this lane opens a store of 1 << log_n slots
        if (valid) {
            const int run0 = 31 - __clz(starts & (0xffffffffu >> (31 - lane)));
            const uint32_t above = lane == 31 ? 0u : starts >> (lane + 1);
            const int run_n = (above ? lane + __ffs(above) : 32) - run0;
            const int rest = run_n - (lane - run0);  // slots of the run from this one on
            const int hb = 31 - __clz(rest);
            if (rest == (run_n & ((2 << hb) - 1))) log_n = hb;
        }
        const bool ok = wait(bar, parity);
        parity ^= 1u;
        if (ok && log_n >= 0) {
            sm100::tma_store_4d(&maps.upd_cache[log_n], stage + lane * ROW, 0, 2 * it.h, pos % ps, page);
            sm100::tma_store_4d(&maps.upd_cache[log_n], stage + (TPW + lane) * ROW, 0, 2 * it.h + 1, pos % ps, page);
        }
        sm100::bulk_commit();
        sm100::bulk_wait_read();  // the buffer may be refilled
        __syncwarp();
        if (!ok) break;
    }
}

// The update of one item shared by two warps (`w` = 0 or 1), each with its own staging buffer at
// stage + w * WARP_BYTES: warp w takes every other round.
template <int D>
__device__ __forceinline__ void tile_update_cache(const KernelArgs& a, const TileCtx& it, int w, int lane, uint32_t stage) {
    using U = TileUpdate<D>;
    tile_update_rounds<D, 1>(a, it, w * U::TPW, 2 * U::TPW, lane, stage + w * U::WARP_BYTES);
}

// FP8 cache: the pass that runs before the tile kernel.  One CTA per tile item quantises the
// item's own K and V rows (Section 3.8: e4m3(x / scale), saturating), stores the codes in the
// cache - the cache update of Algorithm 1 for these tokens - and writes their values back as bf16
// into a scratch copy of new_k / new_v, from which the tile kernel takes its new-token key blocks:
// the batch attends its own tokens in quantised precision, as every later step will see them.
// Doing this once per token instead of once per (query tile, key block) inside the tile kernel is
// what keeps that kernel tensor-bound.
template <int D>
__global__ void __launch_bounds__(128) rpa_quantise_new_kernel(const KernelArgs a) {
    if ((a.validated || a.dev_counts) && (*reinterpret_cast<volatile uint32_t*>(a.status) & kStatusBadInput)) return;
    // a list planned on the device: fixed grid, CTAs stride over the items
    const int n_items = tile_item_count(a);
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const TileItem it = a.tile_items[item];
    const int cu = a.cu_q_lens[it.seq], q_r = a.cu_q_lens[it.seq + 1] - cu, c = a.kv_lens[it.seq] - q_r;
    const int32_t* pt_row = a.page_table + (int64_t)it.seq * a.max_pages_per_seq;
    constexpr int PPR = D / 16;  // 16-element pieces per row
    uint8_t* cache = reinterpret_cast<uint8_t*>(a.kv_cache);
    const int64_t slot_bytes = (int64_t)2 * a.h_kv * D;
    for (int idx = threadIdx.x; idx < it.n_tok * 2 * PPR; idx += blockDim.x) {
        const int jt = idx / (2 * PPR), kv = (idx / PPR) & 1, piece = idx % PPR;
        const int tok = it.q_tok0 + jt;
        int pos = c + tok;
        const int32_t* pt = pt_row;
        if (it.flags & kFlagPacked) {  // the token's own sequence inside the packed run (none of them has context)
            int lo = 0, hi = it.n_seqs - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (a.cu_q_lens[it.seq + mid] - cu <= tok) lo = mid; else hi = mid - 1;
            }
            pos = tok - (a.cu_q_lens[it.seq + lo] - cu);
            pt = pt_row + (int64_t)lo * a.max_pages_per_seq;
        }
        const int64_t src = (((int64_t)cu + tok) * a.h_kv + it.kv_head) * D + piece * 16;
        const uint4 codes = quantise16((kv ? a.new_v : a.new_k) + src, kv ? a.inv_v_scale : a.inv_k_scale);
        if (!kv && a.new_k_codes8) *reinterpret_cast<uint4*>(a.new_k_codes8 + src) = codes;  // for the FP8 score product
        if (!(a.ablation & kAblateUpdate)) {
            const int page = pt[pos / a.page_size];
            if (debug_write_page_ok(a, page))
                *reinterpret_cast<uint4*>(cache + ((int64_t)page * a.page_size + pos % a.page_size) * slot_bytes +
                                          (int64_t)(2 * it.kv_head + kv) * D + piece * 16) = codes;
        }
        uint4 lo, hi;
        lo.x = e4m3x2_to_bf16x2(codes.x & 0xffffu);
        lo.y = e4m3x2_to_bf16x2(codes.x >> 16);
        lo.z = e4m3x2_to_bf16x2(codes.y & 0xffffu);
        lo.w = e4m3x2_to_bf16x2(codes.y >> 16);
        hi.x = e4m3x2_to_bf16x2(codes.z & 0xffffu);
        hi.y = e4m3x2_to_bf16x2(codes.z >> 16);
        hi.z = e4m3x2_to_bf16x2(codes.w & 0xffffu);
        hi.w = e4m3x2_to_bf16x2(codes.w >> 16);
        uint16_t* dst = (kv ? a.new_v_codes : a.new_k_codes) + src;
        *reinterpret_cast<uint4*>(dst) = lo;
        *reinterpret_cast<uint4*>(dst + 8) = hi;
    }
    }
}

// (device-planned lists: eight CTAs per persistent tile CTA stride over the items)
template <int D>
inline cudaError_t launch_quantise_new(const KernelArgs& a, cudaStream_t stream) {
    rpa_quantise_new_kernel<D><<<a.dev_counts ? 8 * a.num_tile_ctas : a.num_tile_items, 128, 0, stream>>>(a);
    return cudaGetLastError();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// tensor map (bf16 and 128-byte swizzle unless told otherwise); dims/strides innermost first, strides in bytes for dims 1..
inline bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
              const uint32_t* box, CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
              CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gdim[5], gstr[5];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) {
        gdim[i] = dims[i];
        bx[i] = box[i];
        es[i] = 1;
        if (i > 0) gstr[i - 1] = strides_bytes[i - 1];
    }
    return fn(m, dtype, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr, bx, es,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The four maps of one launch.  q_tile_tokens: tokens per 128-row query tile (128 / h_g);
// block_n: key positions per block (the new-token box, and the cap of the per-page box).
inline bool build_tile_maps(const KernelArgs& a, int64_t token_rows, int D, int G, int q_tile_tokens, int block_n,
                            TileMaps* maps) {
    const uint64_t d = (uint64_t)D;
    {
        const uint64_t dims[3] = {d, (uint64_t)a.h_q, (uint64_t)token_rows};
        const uint64_t str[2] = {d * 2, d * 2 * a.h_q};
        const uint32_t box[3] = {64, (uint32_t)G, (uint32_t)q_tile_tokens};
        if (a.q_fp8) {  // code bytes: a row of 128 codes is one 128-byte swizzle span
            const uint64_t str8[2] = {d, d * a.h_q};
            const uint32_t box8[3] = {128, (uint32_t)G, (uint32_t)q_tile_tokens};
            if (D != 128 || !make_map(&maps->q, a.q_codes, 3, dims, str8, box8, CU_TENSOR_MAP_DATA_TYPE_UINT8)) return false;
        } else if (!make_map(&maps->q, a.q, 3, dims, str, box)) {
            return false;
        }
        if (!make_map(&maps->out, a.out, 3, dims, str, box)) return false;
    }
    {
        const uint64_t dims[3] = {d, (uint64_t)a.h_kv, (uint64_t)token_rows};
        const uint64_t str[2] = {d * 2, d * 2 * a.h_kv};
        const uint32_t box[3] = {64, 1, (uint32_t)block_n};
        // FP8 cache: the new-token key blocks come from the scratch copies that hold the quantised values
        if (a.q_fp8) {
            const uint64_t str8[2] = {d, d * a.h_kv};
            const uint32_t box8[3] = {128, 1, (uint32_t)block_n};
            if (!make_map(&maps->new_k, a.new_k_codes8, 3, dims, str8, box8, CU_TENSOR_MAP_DATA_TYPE_UINT8)) return false;
        } else if (!make_map(&maps->new_k, a.kv_fp8 ? a.new_k_codes : a.new_k, 3, dims, str, box)) {
            return false;
        }
        if (!make_map(&maps->new_v, a.kv_fp8 ? a.new_v_codes : a.new_v, 3, dims, str, box)) return false;
    }
    if (a.kv_fp8) {
        // one-byte elements: 128 codes are one 128-byte swizzle span (a row of d_k = 256 takes two boxes)
        const uint64_t dims[4] = {d, (uint64_t)2 * a.h_kv, (uint64_t)a.page_size, (uint64_t)a.num_pages};
        const uint64_t str[3] = {d, d * 2 * a.h_kv, d * 2 * a.h_kv * a.page_size};
        const uint32_t box[4] = {128, 1, (uint32_t)page_box_rows(a.page_size, block_n), 1};
        if (D % 128 || !make_map(&maps->cache, a.kv_cache, 4, dims, str, box, CU_TENSOR_MAP_DATA_TYPE_UINT8)) return false;
    } else {
        const uint64_t dims[4] = {d, (uint64_t)2 * a.h_kv, (uint64_t)a.page_size, (uint64_t)a.num_pages};
        const uint64_t str[3] = {d * 2, d * 2 * 2 * a.h_kv, d * 2 * 2 * a.h_kv * a.page_size};
        const uint32_t box[4] = {64, 1, (uint32_t)page_box_rows(a.page_size, block_n), 1};
        if (!make_map(&maps->cache, a.kv_cache, 4, dims, str, box)) return false;
        // the fused update's maps: whole rows as they lie in memory
        const int tpw = 8192 / (2 * D) < 32 ? 8192 / (2 * D) : 32;  // TileUpdate<D>::TPW
        const uint64_t ndims[3] = {d, (uint64_t)a.h_kv, (uint64_t)token_rows};
        const uint64_t nstr[2] = {d * 2, d * 2 * a.h_kv};
        const uint32_t nbox[3] = {(uint32_t)D, 1, (uint32_t)tpw};
        if (!make_map(&maps->upd_k, a.new_k, 3, ndims, nstr, nbox, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_NONE)) return false;
        if (!make_map(&maps->upd_v, a.new_v, 3, ndims, nstr, nbox, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_NONE)) return false;
        for (int i = 0; i < kUpdBoxes; ++i) {
            // (a store never leaves its page: a slot count above the page size or the round is never used)
            const int n = (1 << i) <= a.page_size && (1 << i) <= tpw ? 1 << i : 1;
            const uint32_t cbox[4] = {(uint32_t)D, 1, (uint32_t)n, 1};
            if (!make_map(&maps->upd_cache[i], a.kv_cache, 4, dims, str, cbox, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_NONE)) return false;
        }
    }
    return true;
}

// The same through a cache (see TileMapCache): returns the launch's maps, encoding them only when
// no entry was built from the same tensors.
inline bool cached_tile_maps(TileMapCache* cache, const KernelArgs& a, int64_t token_rows, int D, int G, int q_tile_tokens,
                             int block_n, TileMaps* maps) {
    static_assert(sizeof(TileMaps) == kTileMapBytes, "thirteen tensor maps");
    if (!cache) return build_tile_maps(a, token_rows, D, G, q_tile_tokens, block_n, maps);
    const void* nk = a.q_fp8 ? (const void*)a.new_k_codes8 : a.kv_fp8 ? (const void*)a.new_k_codes : (const void*)a.new_k;
    const void* qp = a.q_fp8 ? (const void*)a.q_codes : (const void*)a.q;
    const void* nv = a.kv_fp8 ? (const void*)a.new_v_codes : (const void*)a.new_v;
    for (auto& e : cache->entries) {
        if (e.valid && e.q == qp && e.q_fp8 == a.q_fp8 && e.out == a.out && e.new_k == nk && e.new_v == nv && e.kv_cache == a.kv_cache &&
            e.token_rows == token_rows && e.h_q == a.h_q && e.h_kv == a.h_kv && e.head_dim == D && e.page_size == a.page_size &&
            e.num_pages == a.num_pages && e.kv_fp8 == a.kv_fp8 && e.block_n == block_n && e.q_tile_tokens == q_tile_tokens) {
            memcpy(maps, e.maps, sizeof(TileMaps));
            return true;
        }
    }
    if (!build_tile_maps(a, token_rows, D, G, q_tile_tokens, block_n, maps)) return false;
    auto& e = cache->entries[cache->next];
    cache->next = (cache->next + 1) % TileMapCache::kEntries;
    e.valid = true;
    e.q = qp, e.q_fp8 = a.q_fp8, e.out = a.out, e.new_k = nk, e.new_v = nv, e.kv_cache = a.kv_cache;
    e.token_rows = token_rows;
    e.h_q = a.h_q, e.h_kv = a.h_kv, e.head_dim = D, e.page_size = a.page_size, e.num_pages = a.num_pages, e.kv_fp8 = a.kv_fp8;
    e.block_n = block_n, e.q_tile_tokens = q_tile_tokens;
    memcpy(e.maps, maps, sizeof(TileMaps));
    return true;
}

}  // namespace rpa
