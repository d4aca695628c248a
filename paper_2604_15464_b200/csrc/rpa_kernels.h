// Launch interface between the C-ABI layer and the CUDA kernels.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "rpa_types.h"

namespace rpa {

constexpr uint32_t kAblateUpdate = 1u;   // skip the fused cache update
constexpr uint32_t kAblateOverlap = 2u;  // mixed batches: run the two kernels one after the other
constexpr uint32_t kAblateCompute = 4u;  // no attention arithmetic: K/V movement and the cache update only (results undefined)
constexpr uint32_t kAblateLoads = 8u;    // no K/V loads: the arithmetic runs on whatever shared memory holds (results undefined)

struct KernelArgs {
    const uint16_t* q;        // bf16 bit patterns throughout
    const uint16_t* new_k;
    const uint16_t* new_v;
    uint16_t* kv_cache;
    uint16_t* new_k_codes;  // FP8 cache, tile path: scratch copies of new_k / new_v holding the values of
    uint16_t* new_v_codes;  // the quantised codes as bf16 (written by the pass before the tile kernel)
    // Quantised Q (a per-tensor scale for Q as well) on the d_k = 128 tile path: the score product runs
    // on the FP8 tensor-core format straight on code bytes - the E4M3 codes of the call's query rows and,
    // for the batch's own tokens, a scratch copy of their K codes (context keys are the cache's bytes).
    const uint8_t* q_codes;  // [T, h_q, d]
    uint8_t* new_k_codes8;   // [T, h_kv, d]
    int32_t q_fp8;           // 1: the tile kernel takes Q and K as E4M3 codes
    const int32_t* page_table;
    const int32_t* cu_q_lens;
    const int32_t* kv_lens;
    uint16_t* out;
    const RowItem* row_items;
    const TileItem* tile_items;
    const CombineGroup* groups;
    float* partial_o;   // [partials][16][d] unnormalised accumulators
    float* partial_ml;  // [partials][16][2] running max (log2 domain) and sum
    int32_t* group_counters;  // one arrival ticket per combine group (zero between calls); null: separate combine kernel
    int32_t* tile_counters;   // [0] next tile item to draw, [1] tile CTAs that have left, [2] CTAs of a dependent row kernel that have finished; all zero between launches
    uint32_t* status;   // device status word
    int32_t num_row_items;
    int32_t num_tile_items;
    int32_t num_tile_ctas;  // persistent CTAs of the tile kernel (each walks the item list with this stride)
    int32_t row_rows_max;   // most query rows (tokens x grouped heads) of any row item
    int32_t num_groups;
    int32_t h_q;
    int32_t h_kv;
    int32_t head_dim;
    int32_t page_size;
    int32_t max_pages_per_seq;
    int32_t num_pages;
    int32_t causal;
    float scale_log2;  // sm_scale * log2(e) (* k_scale for an FP8 cache)
    float out_scale;   // 1, or v_scale for an FP8 cache
    float inv_k_scale; // FP8 cache: fp32 reciprocals of the per-tensor scales, used when new rows are quantised
    float inv_v_scale;
    int32_t kv_fp8;    // cache elements are FP8 E4M3 bytes
    int32_t validated; // a validation kernel ran before this launch: leave at once if it flagged the inputs
    uint32_t ablation;
    int32_t short_items;  // two-tile kernel: 1 every tile item has at most two key blocks (chooses the instantiation built for such items), 2 each is one block at most half full
    // Lists planned on the device: the counts live in device memory (written by the plan kernel of the
    // same step) and take the place of num_row_items, num_tile_items, num_groups and num_tile_ctas.
    const int32_t* dev_counts;  // null: the counts above hold
    // Device-planned steps on a bf16 cache run the tile kernel and the row kernel on ONE stream as a
    // programmatic pair: the tile kernel's CTAs signal at their start (pdl_primary), so the row kernel's
    // CTAs follow them onto the SMs at once instead of waiting for the tile kernel to end, and the
    // row kernel's CTAs wait for the tile kernel's completion only when they leave (pdl_secondary),
    // which keeps the stream's order towards whatever comes next.
    int32_t pdl_primary;
    int32_t pdl_secondary;
    int32_t token_cap;  // rows of q / new_k / new_v / out the call may touch (checked by the RPA_DEBUG build)
};

enum { kDevCountRows = 0, kDevCountTiles = 1, kDevCountGroups = 2, kDevCountTileCtas = 3, kDevCountError = 4,
       kDevCountPartials = 5, kDevCountChunk = 6, kDevCountRowRows = 7, kDevCountInts = 8 };

// Arguments of the device-side planner (rpa_plan_kernel.cu): the lengths, the handle's policy and
// capacities, the lists to fill and its scratch.
struct DevPlanArgs {
    const int32_t* cu_q_lens;
    const int32_t* kv_lens;
    int32_t num_seqs;
    RowItem* rows;
    TileItem* tiles;
    CombineGroup* groups;
    int32_t* counts;       // [kDevCountInts]
    int32_t* seq_offsets;  // [4 * max_num_seqs]
    int32_t* hist;         // [2 * hist_len]
    uint32_t* status;
    int32_t hist_len;      // longest sequence the handle admits, in KV tiles, + 2
    int32_t h_q, h_kv, head_dim, page_size, max_pages_per_seq, max_num_seqs, causal;
    int32_t pack_short;     // pack runs of short sequences without context into shared tile items
    int32_t kv_elem_bytes;  // 2, or 1 for an FP8 cache (only the byte estimate behind the SM split uses it)
    int64_t max_num_tokens;
    int32_t num_slots_narrow;  // see PlanPolicy
    int32_t num_slots, kv_chunk_override, tile_min_q, tile_long_q, tile_long_kv, tile_tokens;
    int32_t max_row_items, max_tile_items, max_groups, max_partials, num_sms;
    double tile_tflops, row_gbs;
};
cudaError_t launch_plan_kernel(const DevPlanArgs& p, cudaStream_t stream);
// the row kernel for device-planned lists: a fixed grid whose CTAs stride over the item list
// (a.pdl_secondary: launched as the programmatic dependent of the kernel before it on `stream`)
cudaError_t launch_row_kernel_strided(const KernelArgs& a, int grid, cudaStream_t stream);
// narrow: the 8-row instantiation (a no-op for more than 8 grouped heads); a device-planned step launches both
cudaError_t launch_row_kernel_fp8_strided(const KernelArgs& a, int grid, bool narrow, cudaStream_t stream);

bool row_kernel_supported(int head_dim, int group);
int row_kernel_ctas_per_sm(int head_dim, int group);
cudaError_t row_kernel_prepare(int head_dim, int group);  // opts in to the dynamic shared memory it needs
cudaError_t launch_row_kernel(const KernelArgs& a, cudaStream_t stream);
cudaError_t launch_combine_kernel(const KernelArgs& a, cudaStream_t stream);
// the same row path on an FP8 E4M3 cache (rpa_row_kernel_fp8.cu)
int row_kernel_fp8_ctas_per_sm(int head_dim);
int row_kernel_fp8_narrow_ctas_per_sm(int head_dim);  // the 8-row instantiation, chosen when no row item has more rows
cudaError_t row_kernel_fp8_prepare(int head_dim, int group);
cudaError_t launch_row_kernel_fp8(const KernelArgs& a, cudaStream_t stream);
// per-tensor quantisation of Q (Section 3.8): q -> bf16 images of its E4M3 values and the raw codes; the rows are
// bounded by total_rows, or, when cu_q_lens (device) is given, by cu_q_lens[num_seqs] (at most max_rows)
cudaError_t launch_quantise_q(const uint16_t* q, uint16_t* q_img, uint8_t* q_codes, int64_t total_rows, const int32_t* cu_q_lens,
                              int32_t num_seqs, int64_t max_rows, int32_t row_elems, float inv_q_scale, const uint32_t* status,
                              bool check_status, cudaStream_t stream);

// The tensor maps of a tile-kernel launch, kept from launch to launch: encoding the five maps costs
// several microseconds of host time, and a serving loop passes the same tensors step after step.  An
// entry is reused when every tensor address and extent it was built from matches (a few entries, so
// that alternating staging buffers all hit); null: encode afresh.
constexpr int kTileMapBytes = 13 * 128;  // the CUtensorMap objects of one launch (128 bytes each)

struct TileMapCache {
    static constexpr int kEntries = 4;
    struct Entry {
        bool valid = false;
        const void *q = nullptr, *out = nullptr, *new_k = nullptr, *new_v = nullptr, *kv_cache = nullptr;
        int64_t token_rows = 0;
        int32_t h_q = 0, h_kv = 0, head_dim = 0, page_size = 0, num_pages = 0, kv_fp8 = 0, q_fp8 = 0, block_n = 0, q_tile_tokens = 0;
        alignas(64) unsigned char maps[kTileMapBytes];
    } entries[kEntries];
    int next = 0;
};

bool tile_kernel_supported(int head_dim, int group);       // d_k = 256 does not fit its TMEM budget
int tile_kernel_tokens(int group);                         // new tokens one tile item covers
bool tile_kernel_fp8_supported(int head_dim, int group);   // the same kernel on an FP8 E4M3 cache
cudaError_t tile_kernel_prepare(int head_dim, int group, bool fp8);  // opts in to its dynamic shared memory
// token_rows: rows of q / new_k / new_v the call may touch (tensor-map extent; rows past it read as zero)
cudaError_t launch_tile_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream);

// single-tile variant with double-buffered scores (rpa_tile1_kernel.cu): d_k = 256
bool tile1_kernel_supported(int head_dim, int group);
cudaError_t tile1_kernel_prepare(int head_dim, int group);
cudaError_t launch_tile1_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream);

// CTA-pair variant for long prefill (rpa_tile2_kernel.cu): d_k = 128, bf16 cache, host-made plans;
// an item covers twice the tokens of a two-tile item, half of them per CTA of the pair
bool tile2_kernel_supported(int head_dim, int group);
int tile2_kernel_tokens(int group);
cudaError_t tile2_kernel_prepare(int group);
cudaError_t launch_tile2_kernel(const KernelArgs& a, int64_t token_rows, TileMapCache* cache, cudaStream_t stream);

// Checks the device copies of the lengths against the plan and every page id a sequence maps
// against the pool size; a violation sets bit 29 of the status word (low bits: the sequence).
cudaError_t launch_validate_kernel(const KernelArgs& a, int32_t num_seqs, const int32_t* plan_kv_lens, cudaStream_t stream);
constexpr uint32_t kStatusBadInput = 1u << 29;

// The bounds-checked build (-DRPA_DEBUG: a library of its own, see build.py) checks every page id
// the kernels take from the page table, the token rows of every work item and the ring-stage
// addresses they form, BEFORE the access.  The first violation of a call is recorded in the status
// word - bit 27, the kind in bits 24..26, the offending value (page id, token row, stage index) in
// the low 24 bits - and the access is skipped (a read goes to page 0 instead, a write is dropped, an
// item with bad rows is not run): the stand-in for a memory checker where none may be run.  Never
// traps.  In the normal build the helpers compile to nothing.
constexpr uint32_t kStatusDebug = 1u << 27;
enum { kDebugPageId = 1, kDebugTokenRow = 2, kDebugStage = 3 };
#if defined(__CUDACC__)
__device__ __forceinline__ void debug_record(const KernelArgs& a, int kind, int value) {
    atomicCAS(a.status, 0u, kStatusDebug | ((uint32_t)kind << 24) | ((uint32_t)value & 0xFFFFFFu));  // the first one stays
}
// page id for a read: the id itself, or page 0 after recording an id outside the pool
__device__ __forceinline__ int debug_read_page(const KernelArgs& a, int page) {
#ifdef RPA_DEBUG
    if ((unsigned)page >= (unsigned)a.num_pages) {
        debug_record(a, kDebugPageId, page);
        return 0;
    }
#endif
    return page;
}
// may this page id be written through?
__device__ __forceinline__ bool debug_write_page_ok(const KernelArgs& a, int page) {
#ifdef RPA_DEBUG
    if ((unsigned)page >= (unsigned)a.num_pages) {
        debug_record(a, kDebugPageId, page);
        return false;
    }
#endif
    return true;
}
// do token rows [row0, row0 + n) lie inside the tensors?
__device__ __forceinline__ bool debug_rows_ok(const KernelArgs& a, long long row0, int n) {
#ifdef RPA_DEBUG
    if (row0 < 0 || n < 0 || row0 + n > a.token_cap) {
        debug_record(a, kDebugTokenRow, (int)(row0 + n));
        return false;
    }
#endif
    return true;
}
// is ring stage `index` one of the `stages` the ring has?
__device__ __forceinline__ bool debug_stage_ok(const KernelArgs& a, int index, int stages) {
#ifdef RPA_DEBUG
    if ((unsigned)index >= (unsigned)stages) {
        debug_record(a, kDebugStage, index);
        return false;
    }
#endif
    return true;
}
#endif

// Launches one warp whose bounded wait must give up (nothing arrives): sets the status word.
cudaError_t launch_wait_selftest(uint32_t* status, cudaStream_t stream);

}  // namespace rpa
