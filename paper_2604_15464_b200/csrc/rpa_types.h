// Internal types shared by the host planner and the CUDA kernels of the library.
#pragma once
#include <stdint.h>

namespace rpa {

constexpr int kRowTileRows = 16;  // query rows (tokens x grouped heads) one row-kernel item covers
constexpr int kKvTile = 16;       // KV positions per pipeline stage of the row kernel
constexpr int kChunkDivisor = 2;  // split-KV: no row item longer than 1/kChunkDivisor of a resident CTA's average share
// Small batches (fewer than kRefineWaves waves of row items): the chunk is varied around its default
// by these factors (in sixteenths) and the one with the lowest estimated makespan wins; the estimate
// is waves x (mean fixed cost of an item, in keys' worth of streaming time, + mean keys per item).
constexpr int kRefineWaves = 6;
constexpr int kRefineFactors[8] = {8, 10, 12, 14, 18, 20, 24, 32};
constexpr int kItemFixedKeys = 192;       // measured: about 4 us per item
constexpr int kSplitItemFixedKeys = 400;  // an item of a split sequence also writes its partial, and one of them merges the group
constexpr long long kTileGlobalOrderBytes = 72ll << 20;  // K/V of the tile-routed sequences up to which tile items are ordered across heads
// Sequences with a few query rows more than one row item holds go to the tile kernel when their context
// is long and their pages have at least this many slots (with 16-slot pages the tile kernel's per-page
// TMA boxes are too small for it to beat two row items; from 32 slots on it streams at 6.1 TB/s against 5.0)
constexpr int kTileLongPage = 32;
constexpr int kQTile = 128;       // query rows per tile-kernel item (tcgen05 M)

constexpr int kFlagWriteKv = 1;   // this item copies its new tokens' K/V rows into the cache
constexpr int kFlagPacked = 2;    // tile item that packs several whole sequences without context (see TileItem)
constexpr int kFlagGroupShift = 8;  // flags >> 8 = 1 + index of the item's combine group (0: not split)
constexpr int kMaxPackedSeqs = 64;  // sequences one packed tile item may hold

// One unit of work for the split-KV row kernel: up to 16 query rows = n_tok consecutive new
// tokens x the h_g query heads of one KV head, against KV positions [kv_begin, kv_end).
struct RowItem {
    int32_t seq;
    int32_t kv_head;
    int32_t q_tok0;    // index of the first token inside its sequence
    int32_t n_tok;
    int32_t kv_begin;  // multiple of kKvTile
    int32_t kv_end;
    int32_t partial;   // workspace slot for the (o, m, l) partial, or -1: write out directly
    int32_t flags;
};

// One unit of work for the tensor-core tile kernel: a tile of query tokens of one sequence for
// one KV head (all h_g grouped query heads), against every key the tile may see.
// A packed item (kFlagPacked) holds n_seqs consecutive sequences, each without cached context
// (kv_len == q_len): seq is the first of them, q_tok0 is 0 and n_tok the sum of their lengths.  Their
// tokens are neighbours on the flattened token axis, so queries, keys and values of the whole group
// are one contiguous range of rows; a row attends only to keys of its own sequence.
struct TileItem {
    int32_t seq;
    int32_t kv_head;
    int32_t q_tok0;
    int32_t n_tok;
    int32_t flags;
    int32_t n_seqs;  // packed items only
    int32_t reserved[2];
};

// A (query block, KV head) whose KV range was split: combine partials [first, first+n).
struct CombineGroup {
    int32_t out_tok0;  // row of the flattened token axis
    int32_t n_tok;
    int32_t kv_head;
    int32_t first_partial;
    int32_t n_partials;
    int32_t reserved[3];
};

static_assert(sizeof(RowItem) == 32 && sizeof(TileItem) == 32 && sizeof(CombineGroup) == 32, "8 int32 each");

}  // namespace rpa
