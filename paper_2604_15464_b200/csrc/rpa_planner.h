// Host-side planner: classifies the batch and builds the device work lists.
//
// This plays the role of the paper's distribution-aware dispatch (Section 3.5): instead of sorting
// the batch into decode / fixed-chunk prefill / mixed ranges and compiling one kernel per range, the
// planner routes every sequence to the kernel specialised for its class and emits explicit work
// items, so the caller may pass requests in any order.
#pragma once
#include <stdint.h>

#include <vector>

#include "../../include/rpa.h"
#include "rpa_types.h"

namespace rpa {

struct PlanPolicy {
    int num_slots = 296;        // CTAs of the row kernel resident on the device at once
    int num_slots_narrow = 0;   // > 0: the same when no row item has more than 8 query rows (a leaner instantiation runs)
    int kv_chunk_override = 0;  // > 0: split-KV chunk length in tokens (multiple of kKvTile)
    int tile_min_q = 0;         // sequences with q_len >= this go to the tile kernel; 0 = none
    int tile_long_q = 0;        // > 0: sequences with q_len >= this also go to the tile kernel when their
                                // context is long (>= kTileLongKv tokens) and pages are not small (>= kTileLongPage slots)
    int tile_tokens = 0;        // query tokens per tile item
    bool pack_short = false;    // pack runs of short sequences without context into one tile item
    int max_row_items = 0;      // capacities of the device lists
    int max_tile_items = 0;
    int max_groups = 0;
    int max_partials = 0;
    bool fused_combine = false;  // the row kernel combines split groups itself (no combine launch)
    int num_sms = 148;
    double tile_tflops = 750.0;   // planning estimates of what each kernel sustains on the whole device
    double row_gbs = 6500.0;
};

constexpr int kTileLongKv = 1024;

struct Plan {
    std::vector<RowItem> rows;
    std::vector<TileItem> tiles;
    std::vector<CombineGroup> groups;
    std::vector<uint32_t> sort_keys;   // scratch
    std::vector<RowItem> sort_scratch; // scratch
    std::vector<uint32_t> sort_count;  // scratch
    std::vector<int32_t> pack_len;     // scratch: sequences in the packed run that starts here (0: none; -1: inside a run)
    rpa_plan_info_t info{};
    int num_partials = 0;
    int row_rows_max = 0;  // most query rows (tokens x grouped heads) of any row item
    int tile_ctas = 0;  // SMs given to the tile kernel (all of them unless row items run beside it)
    bool valid = false;
};

// Does the planner route a sequence of these lengths to the tile kernel?
bool sequence_routed_to_tile(const rpa_config_t& cfg, const PlanPolicy& policy, int64_t q_len, int64_t kv_len);

// Validates the lengths against `cfg` and fills `plan`.  No CUDA call.
rpa_status_t build_plan(const rpa_config_t& cfg, const PlanPolicy& policy, const int32_t* cu_q_lens,
                        const int32_t* kv_lens, int32_t num_seqs, Plan& plan);

}  // namespace rpa
