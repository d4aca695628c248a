// C-ABI layer: argument checks, plan staging and kernel launches.  See include/rpa.h.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <new>
#include <string>
#include <vector>

#include "../../include/rpa.h"
#include "rpa_kernels.h"
#include "rpa_planner.h"

using namespace rpa;

struct rpa_handle {
    rpa_config_t cfg{};
    int device = -1;
    bool plan_only = false;
    int num_sms = 148;
    PlanPolicy policy;
    Plan plan;
    int planned_num_seqs = -1;
    uint32_t ablation = 0;
    int tile_pair_mode = 2;  // tile items of host-made plans: 0 two-tile kernel, 1 CTA-pair kernel, 2 the pair kernel where every tile-routed sequence is long
    bool plan_pair = false;  // the current host-made plan's tile items are pair items
    int plan_short = 0;      // ... or all have at most two key blocks (1), at most half a block (2): see short_items_only
    std::string last_error;

    // Device work lists, [row items | tile items | combine groups | kv_lens | cu_q_lens], in a ring of
    // kPlanRing buffers so that the copy of the next plans (on an internal stream) overlaps the kernels
    // of the current one.  A host-made plan is packed tightly (the offsets of its sections are kept per
    // buffer) and travels in one copy; off_tiles / off_groups / off_kvlens are the offsets at full
    // capacity, used for the buffers' size and by the device-side planner.
    static constexpr int kPlanRing = 4;
    uint8_t* d_lists[kPlanRing] = {};
    uint8_t* h_lists[kPlanRing] = {};  // pinned mirrors
    size_t buf_off_tiles[kPlanRing] = {}, buf_off_groups[kPlanRing] = {}, buf_off_kvlens[kPlanRing] = {}, buf_off_cu[kPlanRing] = {};
    size_t off_tiles = 0, off_groups = 0, lists_bytes = 0;
    TileMapCache tile_maps;  // tensor maps of the tile kernels, keyed by the tensors they describe
    cudaStream_t copy_stream = nullptr;
    cudaStream_t aux_stream = nullptr;  // the tile kernel of a mixed batch runs here, beside the row kernel
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
    cudaStream_t aux2_stream = nullptr;  // device-planned FP8 steps: the row kernel instantiation the list may not need
    cudaEvent_t ev_fork2 = nullptr, ev_join2 = nullptr;
    cudaEvent_t ev_copied[kPlanRing] = {};    // plan copy into buffer b finished
    cudaEvent_t ev_consumed[kPlanRing] = {};  // last forward that read buffer b finished
    bool copied_pending[kPlanRing] = {};
    bool consumed_pending[kPlanRing] = {};
    int cur = 0;  // buffer holding the current plan
    bool validate = false;        // run the input validation kernel before the attention kernels
    size_t off_kvlens = 0;        // the plan's kv_lens travel with the lists (for the validation kernel)
    std::vector<int32_t> plan_kv_lens;
    int32_t* d_group_counters = nullptr;

    // lists planned on the device (rpa_plan_device): their own buffer, counts and scratch
    bool device_planned = false;
    // (two sets, so that the plan of step i+1 may be written on one stream while the kernels of step i
    // still read theirs on another; events order a set's writer and readers)
    uint8_t* d_dev_lists_buf[2] = {nullptr, nullptr};
    int32_t* d_dev_counts_buf[2] = {nullptr, nullptr};
    int dev_cur = 0;                    // set holding the latest device-made plan
    uint8_t* d_dev_lists = nullptr;     // = d_dev_lists_buf[dev_cur]
    int32_t* d_dev_counts = nullptr;    // = d_dev_counts_buf[dev_cur]
    cudaEvent_t ev_dev_planned[2] = {nullptr, nullptr};   // plan kernel writing set b finished
    cudaEvent_t ev_dev_consumed[2] = {nullptr, nullptr};  // last forward reading set b finished
    bool dev_planned_pending[2] = {false, false};
    bool dev_consumed_pending[2] = {false, false};
    int32_t* d_dev_scratch = nullptr;
    int32_t dev_hist_len = 0;
    uint16_t* d_new_codes = nullptr;  // FP8 cache with a tile path: bf16 copies of new_k | new_v after quantisation
    uint16_t* d_q_img = nullptr;      // quantised Q (q_scale > 0): the E4M3 values of the call's query rows as bf16 ...
    uint8_t* d_q_codes = nullptr;     // ... and their codes
    uint8_t* d_new_k_codes8 = nullptr;  // ... and, for the FP8 score product of the tile kernel, the K codes of the call's own tokens
    float* d_partial_o = nullptr;
    float* d_partial_ml = nullptr;
    uint32_t* d_status = nullptr;

    // optional per-kernel timing: event pairs recorded around each launch (0 row, 1 tile, 2 combine)
    bool timing = false;
    std::vector<cudaEvent_t> ev[3];  // start, stop, start, stop, ...
    size_t ev_used[3] = {0, 0, 0};

    // staging for rpa_forward_host and its submit/wait halves (allocated on first use): two slots, so
    // that the copies of one step run beside the kernels of its neighbours
    uint8_t* d_host_stage[2] = {nullptr, nullptr};
    size_t hs_q = 0, hs_k = 0, hs_v = 0, hs_out = 0, hs_pt = 0, hs_cu = 0, hs_kl = 0, hs_bytes = 0;
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    cudaEvent_t ev_in[2] = {nullptr, nullptr}, ev_ran[2] = {nullptr, nullptr}, ev_out[2] = {nullptr, nullptr};
    uint64_t hs_submitted = 0, hs_waited = 0;
};

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

rpa_status_t cuda_fail(rpa_handle* h, cudaError_t e, const char* what) {
    if (h) h->last_error = std::string(what) + ": " + cudaGetErrorString(e);
    return RPA_ERR_CUDA;
}

#define RPA_CUDA(h, call)                                       \
    do {                                                        \
        cudaError_t e_ = (call);                                \
        if (e_ != cudaSuccess) return cuda_fail(h, e_, #call);  \
    } while (0)

bool valid_config(const rpa_config_t& c, rpa_status_t* why) {
    *why = RPA_ERR_INVALID_ARG;
    if (c.num_q_heads <= 0 || c.num_kv_heads <= 0 || c.num_q_heads % c.num_kv_heads) return false;
    if (c.head_dim <= 0 || c.page_size <= 0 || c.num_pages <= 0 || c.max_pages_per_seq <= 0) return false;
    if (c.max_num_seqs <= 0 || c.max_num_tokens <= 0 || !(c.sm_scale >= 0.f)) return false;
    if (c.kv_dtype != RPA_KV_BF16 && c.kv_dtype != RPA_KV_FP8_E4M3) return false;
    if (c.kv_dtype == RPA_KV_FP8_E4M3 && !(c.k_scale > 0.f && c.v_scale > 0.f)) return false;
    if (!(c.q_scale >= 0.f) || (c.q_scale > 0.f && c.kv_dtype != RPA_KV_FP8_E4M3)) return false;  // a scale for Q goes with an FP8 cache
    *why = RPA_ERR_UNSUPPORTED;
    if (!row_kernel_supported(c.head_dim, c.num_q_heads / c.num_kv_heads)) return false;
    if (c.page_size % kKvTile) return false;
    return true;
}

void free_all(rpa_handle* h) {
    if (!h->plan_only) {
        for (int b = 0; b < rpa_handle::kPlanRing; ++b) {
            cudaFree(h->d_lists[b]);
            if (h->h_lists[b]) cudaFreeHost(h->h_lists[b]);
            if (h->ev_copied[b]) cudaEventDestroy(h->ev_copied[b]);
            if (h->ev_consumed[b]) cudaEventDestroy(h->ev_consumed[b]);
        }
        if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
        if (h->aux_stream) cudaStreamDestroy(h->aux_stream);
        if (h->aux2_stream) cudaStreamDestroy(h->aux2_stream);
        if (h->ev_fork2) cudaEventDestroy(h->ev_fork2);
        if (h->ev_join2) cudaEventDestroy(h->ev_join2);
        if (h->ev_fork) cudaEventDestroy(h->ev_fork);
        if (h->ev_join) cudaEventDestroy(h->ev_join);
        cudaFree(h->d_group_counters);
        cudaFree(h->d_partial_o);
        cudaFree(h->d_new_codes);
        cudaFree(h->d_q_img);
        cudaFree(h->d_q_codes);
        cudaFree(h->d_new_k_codes8);
        for (int b = 0; b < 2; ++b) {
            cudaFree(h->d_dev_lists_buf[b]);
            cudaFree(h->d_dev_counts_buf[b]);
            if (h->ev_dev_planned[b]) cudaEventDestroy(h->ev_dev_planned[b]);
            if (h->ev_dev_consumed[b]) cudaEventDestroy(h->ev_dev_consumed[b]);
        }
        cudaFree(h->d_dev_scratch);
        cudaFree(h->d_partial_ml);
        cudaFree(h->d_status);
        for (int b = 0; b < 2; ++b) {
            cudaFree(h->d_host_stage[b]);
            if (h->ev_in[b]) cudaEventDestroy(h->ev_in[b]);
            if (h->ev_ran[b]) cudaEventDestroy(h->ev_ran[b]);
            if (h->ev_out[b]) cudaEventDestroy(h->ev_out[b]);
        }
        if (h->h2d_stream) cudaStreamDestroy(h->h2d_stream);
        if (h->d2h_stream) cudaStreamDestroy(h->d2h_stream);
        for (auto& v : h->ev)
            for (cudaEvent_t e : v) cudaEventDestroy(e);
    }
}

rpa_status_t ensure_device(rpa_handle* h) {
    int cur = -1;
    RPA_CUDA(h, cudaGetDevice(&cur));
    if (cur != h->device) RPA_CUDA(h, cudaSetDevice(h->device));
    return RPA_OK;
}

constexpr size_t kMaxTimedLaunches = 8192;

// Records an event on `s` for kernel kind `k`; creates events on demand, stops silently when full.
void timing_mark(rpa_handle* h, int k, cudaStream_t s) {
    if (!h->timing || h->ev_used[k] >= 2 * kMaxTimedLaunches) return;
    if (h->ev_used[k] == h->ev[k].size()) {
        cudaEvent_t e;
        if (cudaEventCreate(&e) != cudaSuccess) return;
        h->ev[k].push_back(e);
    }
    cudaEventRecord(h->ev[k][h->ev_used[k]++], s);
}

// Sequences whose query rows (tokens x heads of a group) fill more than two row items go to the
// tile kernel: from three row items on, the row kernel re-reads the context once per item and falls
// behind the tile kernel even though most of a 128-row tile stays empty.
int default_tile_min_q(int h_g) { return std::max(2, 2 * kRowTileRows / h_g + 1); }

// Is there a tensor-core tile kernel for this shape and cache type?
bool tile_path_available(const rpa_config_t& c) {
    const int h_g = c.num_q_heads / c.num_kv_heads;
    // (the single-tile kernel has an FP8 instantiation for every shape it supports)
    if (c.kv_dtype == RPA_KV_FP8_E4M3) return tile_kernel_fp8_supported(c.head_dim, h_g) || tile1_kernel_supported(c.head_dim, h_g);
    return tile_kernel_supported(c.head_dim, h_g) || tile1_kernel_supported(c.head_dim, h_g);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// RPA_LOG=1 in the environment (read once): every rpa_plan prints one line to stderr that says what
// it made of the batch - its class, how the sequences were routed, the work lists, the split-KV
// chunk, the SM split of a mixed batch, the algorithmic work.
bool plan_log_enabled() {
    static const bool on = [] {
        const char* v = getenv("RPA_LOG");
        return v && *v && strcmp(v, "0") != 0;
    }();
    return on;
}

void log_plan(const rpa_handle* h) {
    static const char* const kCase[] = {"empty", "decode", "prefill", "mixed"};
    const rpa_plan_info_t& i = h->plan.info;
    fprintf(stderr,
            "[rpa] plan: %s batch, %d seqs (%d decode, %d prefill), %d new tokens; row kernel %d items (largest %d rows, "
            "split chunk %d tokens, %d combine groups, %d partials), %s kernel %d items on %d CTAs; %d launches, %.3f GB, "
            "%.3f GFLOP (row %.3f GB, tile %.3f GFLOP)\n",
            kCase[i.batch_case & 3], i.num_seqs, i.num_decode_seqs, i.num_prefill_seqs, i.num_tokens, i.num_row_items,
            h->plan.row_rows_max, i.kv_chunk_tokens, i.num_combine_groups, h->plan.num_partials,
            i.tile_kernel == 3 ? "pair" : i.tile_kernel == 2 ? "single-tile" : i.tile_short_items ? "tile (short-item)" : "tile", i.num_tile_items,
            h->plan.tile_ctas > 0 ? h->plan.tile_ctas : (i.num_tile_items > 0 ? std::min(i.num_tile_items, h->num_sms) : 0),
            i.gpu_launches, i.algorithmic_bytes / 1e9, i.algorithmic_flops / 1e9, i.row_bytes / 1e9, i.tile_flops / 1e9);
}

// Do this batch's tile items run on the CTA-pair kernel?  It wants items of four full query tiles:
// a shorter item leaves the pair's second CTA (or half of each CTA) without rows.  So, unless told
// otherwise, it is chosen for pure long-prefill batches - every sequence goes to the tile kernel and
// brings at least two full pair items of new tokens - and left alone for small-q steps over long
// contexts, for short prompts (which the two-tile kernel splits by key blocks or packs) and for mixed
// batches, where the tile kernel shares the device with the row kernel (measured: 1024-token chunks
// beside 192 decode rows run 0.5-1 % slower on pairs, which need two neighbouring SMs each).
bool pair_kernel_wanted(const rpa_handle* h, const int32_t* cu_q_lens, const int32_t* kv_lens, int32_t num_seqs) {
    const rpa_config_t& c = h->cfg;
    const int h_g = c.num_q_heads / c.num_kv_heads;
    if (h->tile_pair_mode == 0 || h->policy.tile_min_q <= 0 || c.kv_dtype != RPA_KV_BF16 || !tile2_kernel_supported(c.head_dim, h_g))
        return false;
    if (h->plan_only && h->tile_pair_mode != 1) return false;  // (no device: plan what every device can run)
    if (h->tile_pair_mode == 1) return true;
    if (!cu_q_lens || !kv_lens) return false;
    const int64_t per_item = tile2_kernel_tokens(h_g), long_q = 2 * per_item;
    int64_t items = 0;
    for (int32_t r = 0; r < num_seqs; ++r) {
        const int64_t q = (int64_t)cu_q_lens[r + 1] - cu_q_lens[r];
        if (q == 0) continue;
        if (!sequence_routed_to_tile(c, h->policy, q, kv_lens[r]) || q < long_q) return false;
        items += (int64_t)c.num_kv_heads * ((q + per_item - 1) / per_item);
    }
    // ... and when there are enough items to keep every pair busy for a few rounds (one prompt of 2048
    // tokens, 128 pair items on 74 pairs, ran 7 % slower than its 256 items on the two-tile kernel)
    return items >= 2 * (int64_t)h->num_sms;
}

// The two-tile kernel has an instantiation for batches whose tile items all have one or two key blocks
// (many short prompts without much context): there the per-item chain of latencies is everything, and
// the cache update by the copy engine and the softmax function for a half-full block pay; on items
// that stream many key blocks the same code costs 2-5 % (small-q steps over 4096 tokens of context on
// 16-slot pages: 445 us with it, 426 without), so those keep the plain instantiation.
// Returns 0 (plain instantiation), 1 (short items) or 2 (short items that are all of one, at most
// half-full key block: only then does the half-block softmax pay - in a batch that mixes such items
// with full blocks, 1024 prompts of 128 tokens, it made the step 5-8 % slower).
int short_items_only(const rpa_handle* h, const int32_t* cu_q_lens, const int32_t* kv_lens, int32_t num_seqs) {
    const rpa_config_t& c = h->cfg;
    if (c.kv_dtype != RPA_KV_BF16 || !cu_q_lens || !kv_lens) return 0;
    int32_t longest = 0;
    for (int32_t r = 0; r < num_seqs; ++r) {
        const int64_t q = (int64_t)cu_q_lens[r + 1] - cu_q_lens[r];
        if (q == 0 || !sequence_routed_to_tile(c, h->policy, q, kv_lens[r])) continue;
        longest = std::max(longest, kv_lens[r]);
    }
    return longest == 0 || longest > 2 * kQTile ? 0 : longest <= kQTile / 2 ? 2 : 1;
}

// Events recorded outside a capture cannot be waited for inside one (and the other way round): while
// a stream is being captured into a graph, the capture's own order stands in for the handle's events.
bool stream_is_capturing(cudaStream_t s) {
    cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
    return cudaStreamIsCapturing(s, &st) == cudaSuccess && st != cudaStreamCaptureStatusNone;
}

}  // namespace

extern "C" {

rpa_status_t rpa_create(const rpa_config_t* cfg, int device, rpa_handle_t** out) {
    if (out) *out = nullptr;
    if (!cfg || !out) return RPA_ERR_INVALID_ARG;
    rpa_status_t why;
    if (!valid_config(*cfg, &why)) return why;
    rpa_handle* h = new (std::nothrow) rpa_handle();
    if (!h) return RPA_ERR_CUDA;
    h->cfg = *cfg;
    if (h->cfg.sm_scale == 0.f) h->cfg.sm_scale = 1.f / sqrtf((float)cfg->head_dim);
    h->device = device;
    h->plan_only = device < 0;
    const int h_g = cfg->num_q_heads / cfg->num_kv_heads;

    if (!h->plan_only) {
        cudaError_t e = cudaSetDevice(device);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, device);
        if (e == cudaSuccess)
            e = cfg->kv_dtype == RPA_KV_FP8_E4M3 ? row_kernel_fp8_prepare(cfg->head_dim, h_g) : row_kernel_prepare(cfg->head_dim, h_g);
        if (e == cudaSuccess && cfg->kv_dtype == RPA_KV_BF16 && tile_kernel_supported(cfg->head_dim, h_g))
            e = tile_kernel_prepare(cfg->head_dim, h_g, false);
        if (e == cudaSuccess && cfg->kv_dtype == RPA_KV_FP8_E4M3 && tile_kernel_fp8_supported(cfg->head_dim, h_g))
            e = tile_kernel_prepare(cfg->head_dim, h_g, true);
        if (e == cudaSuccess && tile1_kernel_supported(cfg->head_dim, h_g)) e = tile1_kernel_prepare(cfg->head_dim, h_g);
        if (e == cudaSuccess && cfg->kv_dtype == RPA_KV_BF16 && tile2_kernel_supported(cfg->head_dim, h_g)) e = tile2_kernel_prepare(h_g);
        if (e != cudaSuccess) {
            delete h;
            return RPA_ERR_CUDA;
        }
    }
    PlanPolicy& p = h->policy;
    p.num_slots = h->num_sms * (cfg->kv_dtype == RPA_KV_FP8_E4M3 ? row_kernel_fp8_ctas_per_sm(cfg->head_dim)
                                                                   : row_kernel_ctas_per_sm(cfg->head_dim, h_g));
    if (cfg->kv_dtype == RPA_KV_FP8_E4M3 && h_g <= 8) p.num_slots_narrow = h->num_sms * row_kernel_fp8_narrow_ctas_per_sm(cfg->head_dim);
    const int tpi = kRowTileRows / h_g;
    const int64_t base_units = (int64_t)cfg->num_kv_heads * ((cfg->max_num_tokens + tpi - 1) / tpi + cfg->max_num_seqs);
    p.max_partials = std::max(16 * std::max(p.num_slots, p.num_slots_narrow), 4096);
    p.max_groups = p.max_partials / 2;
    p.max_row_items = (int)std::min<int64_t>(base_units + p.max_partials, 1 << 28);
    p.fused_combine = true;
    p.num_sms = h->num_sms;
    // d_k = 256 runs the single-tile variant: an item is one query tile
    const bool single_tile = tile1_kernel_supported(cfg->head_dim, h_g);
    p.tile_tokens = single_tile ? 128 / h_g : tile_kernel_tokens(h_g);
    p.tile_min_q = default_tile_min_q(h_g);
    p.tile_long_q = std::max(2, kRowTileRows / h_g + 1);
    if (!tile_path_available(*cfg)) p.tile_min_q = p.tile_long_q = 0;  // rows only
    // runs of short sequences without context share one tile item (two-tile kernel)
    p.pack_short = p.tile_min_q > 0 && !single_tile;
    p.max_tile_items = (int)std::min<int64_t>(
        (int64_t)cfg->num_kv_heads * ((cfg->max_num_tokens + p.tile_tokens - 1) / p.tile_tokens + cfg->max_num_seqs), 1 << 28);
    h->plan.rows.reserve(p.max_row_items);
    h->plan.sort_scratch.reserve(p.max_row_items);
    h->plan.sort_keys.reserve(p.max_row_items);
    h->plan.groups.reserve(p.max_groups);
    h->plan.tiles.reserve(std::max(p.max_tile_items, 1));

    h->off_tiles = align_up((size_t)p.max_row_items * sizeof(RowItem), 256);
    h->off_groups = h->off_tiles + align_up((size_t)std::max(p.max_tile_items, 1) * sizeof(TileItem), 256);
    h->off_kvlens = h->off_groups + align_up((size_t)p.max_groups * sizeof(CombineGroup), 256);
    h->lists_bytes = h->off_kvlens + align_up((size_t)cfg->max_num_seqs * sizeof(int32_t), 256) +
                     align_up(((size_t)cfg->max_num_seqs + 1) * sizeof(int32_t), 256);

    if (!h->plan_only) {
        cudaError_t e = cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking);
        int prio_lo = 0, prio_hi = 0;
        if (e == cudaSuccess) e = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi);
        if (e == cudaSuccess) e = cudaStreamCreateWithPriority(&h->aux_stream, cudaStreamNonBlocking, prio_hi);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->aux2_stream, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_fork2, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_join2, cudaEventDisableTiming);
        for (int b = 0; b < rpa_handle::kPlanRing && e == cudaSuccess; ++b) {
            e = cudaMalloc(&h->d_lists[b], h->lists_bytes);
            if (e == cudaSuccess) e = cudaMallocHost(&h->h_lists[b], h->lists_bytes);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_copied[b], cudaEventDisableTiming);
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&h->ev_consumed[b], cudaEventDisableTiming);
        }
        if (e == cudaSuccess && cfg->kv_dtype == RPA_KV_FP8_E4M3 && p.tile_min_q > 0)
            e = cudaMalloc(&h->d_new_codes, (size_t)2 * cfg->max_num_tokens * cfg->num_kv_heads * cfg->head_dim * sizeof(uint16_t));
        if (e == cudaSuccess && cfg->q_scale > 0.f) {
            const size_t q_elems = (size_t)cfg->max_num_tokens * cfg->num_q_heads * cfg->head_dim;
            e = cudaMalloc(&h->d_q_img, q_elems * sizeof(uint16_t));
            if (e == cudaSuccess) e = cudaMalloc(&h->d_q_codes, q_elems);
            if (e == cudaSuccess && cfg->head_dim == 128 && p.tile_min_q > 0)
                e = cudaMalloc(&h->d_new_k_codes8, (size_t)cfg->max_num_tokens * cfg->num_kv_heads * cfg->head_dim);
        }
        if (e == cudaSuccess) e = cudaMalloc(&h->d_group_counters, (size_t)p.max_groups * sizeof(int32_t));
        if (e == cudaSuccess) e = cudaMemset(h->d_group_counters, 0, (size_t)p.max_groups * sizeof(int32_t));
        if (e == cudaSuccess)
            e = cudaMalloc(&h->d_partial_o, (size_t)p.max_partials * kRowTileRows * cfg->head_dim * sizeof(float));
        if (e == cudaSuccess) e = cudaMalloc(&h->d_partial_ml, (size_t)p.max_partials * kRowTileRows * 2 * sizeof(float));
        if (e == cudaSuccess) e = cudaMalloc(&h->d_status, 256);
        if (e == cudaSuccess) e = cudaMemset(h->d_status, 0, 256);
        if (e != cudaSuccess) {
            free_all(h);
            delete h;
            return RPA_ERR_CUDA;
        }
    }
    *out = h;
    return RPA_OK;
}

void rpa_destroy(rpa_handle_t* h) {
    if (!h) return;
    free_all(h);
    delete h;
}

rpa_status_t rpa_plan(rpa_handle_t* h, const int32_t* cu_q_lens_host, const int32_t* kv_lens_host, int32_t num_seqs,
                      void* stream) {
    if (!h) return RPA_ERR_INVALID_ARG;
    h->planned_num_seqs = -1;
    h->device_planned = false;
    const bool pair = pair_kernel_wanted(h, cu_q_lens_host, kv_lens_host, num_seqs);
    PlanPolicy pol = h->policy;
    if (pair) {  // pair items: twice the tokens, never packed
        pol.tile_tokens = tile2_kernel_tokens(h->cfg.num_q_heads / h->cfg.num_kv_heads);
        pol.pack_short = false;
    }
    rpa_status_t st = build_plan(h->cfg, pol, cu_q_lens_host, kv_lens_host, num_seqs, h->plan);
    if (st != RPA_OK) return st;
    h->plan_pair = pair;
    h->plan_short = pair ? 0 : short_items_only(h, cu_q_lens_host, kv_lens_host, num_seqs);
    h->plan.info.tile_kernel = h->plan.tiles.empty() ? 0
                               : pair ? 3
                               : tile1_kernel_supported(h->cfg.head_dim, h->cfg.num_q_heads / h->cfg.num_kv_heads) ? 2 : 1;
    if (h->plan.info.tile_kernel != 1) h->plan_short = 0;
    h->plan.info.tile_short_items = h->plan_short;
    if (plan_log_enabled()) log_plan(h);
    if (!h->plan_only) {
        st = ensure_device(h);
        if (st != RPA_OK) return st;
        // The copy goes into the next buffer of the ring, on the internal stream: it may run while the
        // kernels of earlier rpa_forward calls are still in flight.  The host waits only if the pinned
        // mirror of that buffer still feeds the copy of the plan made kPlanRing calls ago (the caller is
        // that many plans ahead of the device).
        const int b = (h->cur + 1) % rpa_handle::kPlanRing;
        if (h->copied_pending[b]) {
            if (cudaEventQuery(h->ev_copied[b]) != cudaSuccess) RPA_CUDA(h, cudaEventSynchronize(h->ev_copied[b]));
            h->copied_pending[b] = false;
        }
        if (h->consumed_pending[b]) {  // kernels of an older rpa_forward may still read the device buffer
            RPA_CUDA(h, cudaStreamWaitEvent(h->copy_stream, h->ev_consumed[b], 0));
            h->consumed_pending[b] = false;
        }
        // one tightly packed block, one copy: [row items | tile items | groups | kv_lens | cu_q_lens]
        const size_t nb_rows = h->plan.rows.size() * sizeof(RowItem);
        const size_t nb_tiles = h->plan.tiles.size() * sizeof(TileItem);
        const size_t nb_groups = h->plan.groups.size() * sizeof(CombineGroup);
        const size_t n = (size_t)std::max(num_seqs, 0);
        h->buf_off_tiles[b] = align_up(nb_rows, 256);
        h->buf_off_groups[b] = h->buf_off_tiles[b] + align_up(nb_tiles, 256);
        h->buf_off_kvlens[b] = h->buf_off_groups[b] + align_up(nb_groups, 256);
        h->buf_off_cu[b] = h->buf_off_kvlens[b] + align_up(n * sizeof(int32_t), 256);
        const size_t total = h->buf_off_cu[b] + (n + 1) * sizeof(int32_t);
        uint8_t* m = h->h_lists[b];
        if (nb_rows) memcpy(m, h->plan.rows.data(), nb_rows);
        if (nb_tiles) memcpy(m + h->buf_off_tiles[b], h->plan.tiles.data(), nb_tiles);
        if (nb_groups) memcpy(m + h->buf_off_groups[b], h->plan.groups.data(), nb_groups);
        if (n) memcpy(m + h->buf_off_kvlens[b], kv_lens_host, n * sizeof(int32_t));
        if (n) memcpy(m + h->buf_off_cu[b], cu_q_lens_host, (n + 1) * sizeof(int32_t));
        RPA_CUDA(h, cudaMemcpyAsync(h->d_lists[b], m, total, cudaMemcpyHostToDevice, h->copy_stream));
        RPA_CUDA(h, cudaEventRecord(h->ev_copied[b], h->copy_stream));
        h->copied_pending[b] = true;
        h->cur = b;
    }
    h->planned_num_seqs = num_seqs;
    return RPA_OK;
}

// The kernel arguments every launch of a call shares: tensors, shape, scales; `lists` is the device
// buffer holding [row items | tile items | combine groups].  Counts are filled in by the caller.
static KernelArgs common_kernel_args(const rpa_handle* h, uint8_t* lists, size_t off_tiles, size_t off_groups, const void* q, const void* new_k, const void* new_v,
                                     void* kv_cache, const int32_t* page_table, const int32_t* cu_q_lens,
                                     const int32_t* kv_lens, void* out) {
    const rpa_config_t& c = h->cfg;
    KernelArgs a{};
    // with a scale for Q the kernels read the quantised image the pass before them has made
    a.q = c.q_scale > 0.f ? h->d_q_img : static_cast<const uint16_t*>(q);
    a.new_k = static_cast<const uint16_t*>(new_k);
    a.new_v = static_cast<const uint16_t*>(new_v);
    a.kv_cache = static_cast<uint16_t*>(kv_cache);
    a.q_codes = h->d_q_codes;
    a.new_k_codes8 = h->d_new_k_codes8;
    a.q_fp8 = h->d_new_k_codes8 != nullptr && !(h->ablation & 16u) ? 1 : 0;  // (ablation bit 4: bf16 score products on the images instead)
    a.new_k_codes = h->d_new_codes;
    a.new_v_codes = h->d_new_codes ? h->d_new_codes + (size_t)c.max_num_tokens * c.num_kv_heads * c.head_dim : nullptr;
    a.page_table = page_table;
    a.cu_q_lens = cu_q_lens;
    a.kv_lens = kv_lens;
    a.out = static_cast<uint16_t*>(out);
    a.row_items = reinterpret_cast<const RowItem*>(lists);
    a.tile_items = reinterpret_cast<const TileItem*>(lists + off_tiles);
    a.groups = reinterpret_cast<const CombineGroup*>(lists + off_groups);
    a.partial_o = h->d_partial_o;
    a.partial_ml = h->d_partial_ml;
    a.status = h->d_status;
    a.tile_counters = reinterpret_cast<int32_t*>(h->d_status) + 16;  // same zero-initialised block as the status word
    a.h_q = c.num_q_heads;
    a.h_kv = c.num_kv_heads;
    a.head_dim = c.head_dim;
    a.page_size = c.page_size;
    a.max_pages_per_seq = c.max_pages_per_seq;
    a.num_pages = c.num_pages;
    a.causal = c.causal ? 1 : 0;
    const bool fp8 = c.kv_dtype == RPA_KV_FP8_E4M3;
    a.kv_fp8 = fp8 ? 1 : 0;
    a.scale_log2 = c.sm_scale * 1.4426950408889634f * (fp8 ? c.k_scale : 1.f) * (c.q_scale > 0.f ? c.q_scale : 1.f);
    a.out_scale = fp8 ? c.v_scale : 1.f;
    a.inv_k_scale = fp8 ? 1.0f / c.k_scale : 1.f;
    a.inv_v_scale = fp8 ? 1.0f / c.v_scale : 1.f;
    a.ablation = h->ablation;
    a.token_cap = c.max_num_tokens;
    return a;
}

// The attention kernels of a step whose lists were planned on the device.  The host knows neither
// the batch's class nor its item counts, so both kernels are launched with fixed grids, side by
// side: the tile kernel as one CTA per SM (the CTAs beyond the planner's share leave at once), the
// row kernel as a fixed number of CTAs striding over the list.  Nothing here depends on the
// lengths, so the sequence [rpa_plan_device, rpa_forward] can be captured in a CUDA graph.
static rpa_status_t forward_device_planned(rpa_handle* h, const void* q, const void* new_k, const void* new_v,
                                           void* kv_cache, const int32_t* page_table, const int32_t* cu_q_lens,
                                           const int32_t* kv_lens, void* out, void* stream) {
    if (!q || !new_k || !new_v || !kv_cache || !page_table || !cu_q_lens || !kv_lens || !out) return RPA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(new_k) || !aligned16(new_v) || !aligned16(kv_cache) || !aligned16(out))
        return RPA_ERR_INVALID_ARG;
    const rpa_config_t& c = h->cfg;
    KernelArgs a = common_kernel_args(h, h->d_dev_lists, h->off_tiles, h->off_groups, q, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens, out);
    a.group_counters = h->d_group_counters;
    a.dev_counts = h->d_dev_counts;
    a.num_tile_ctas = h->num_sms;
    const bool fp8 = c.kv_dtype == RPA_KV_FP8_E4M3;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int b = h->dev_cur;
    const bool capturing = stream_is_capturing(s);
    if (!capturing && h->dev_planned_pending[b]) RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_dev_planned[b], 0));  // the plan may come from another stream
    if (c.q_scale > 0.f)  // (T is known on the device only: the pass bounds its rows by cu_q_lens[num_seqs])
        RPA_CUDA(h, launch_quantise_q(static_cast<const uint16_t*>(q), h->d_q_img, h->d_q_codes, 0, cu_q_lens, h->planned_num_seqs,
                                      c.max_num_tokens, c.num_q_heads * c.head_dim, 1.0f / c.q_scale, h->d_status, true, s));
    const bool tiles = h->policy.tile_min_q > 0;
    const bool single_tile = tile1_kernel_supported(c.head_dim, c.num_q_heads / c.num_kv_heads);
    // eight waves of resident CTAs: short lists get one item per CTA (placed dynamically by the
    // hardware, as with a host-made plan), long ones are strided
    const int grid = (int)std::min<int64_t>(h->policy.max_row_items, (int64_t)8 * h->policy.num_slots);
    if (!fp8) {
        // One stream, two kernels as a programmatic pair.  The tile kernel goes first and gets its SMs
        // first (a CTA of it needs an SM to itself even to find that the list holds nothing for it);
        // its CTAs signal at their start, and the row kernel's CTAs follow them onto the device without
        // waiting for the tile kernel to end.  A decode step thus pays for a grid of CTAs that leave at
        // once, not for a kernel that can only start as the row kernel drains.  (Events recorded
        // between the two launches, when per-kernel timing is on, serialise the pair.)
        if (tiles) {
            a.pdl_primary = 1;
            timing_mark(h, 1, s);
            RPA_CUDA(h, single_tile ? launch_tile1_kernel(a, c.max_num_tokens, &h->tile_maps, s)
                                    : launch_tile_kernel(a, c.max_num_tokens, &h->tile_maps, s));
            timing_mark(h, 1, s);
            a.pdl_primary = 0;
            a.pdl_secondary = 1;
        }
        timing_mark(h, 0, s);
        RPA_CUDA(h, launch_row_kernel_strided(a, grid, s));
        timing_mark(h, 0, s);
    } else {
        if (tiles) {
            RPA_CUDA(h, cudaEventRecord(h->ev_fork, s));
            RPA_CUDA(h, cudaStreamWaitEvent(h->aux_stream, h->ev_fork, 0));
            timing_mark(h, 1, h->aux_stream);
            RPA_CUDA(h, single_tile ? launch_tile1_kernel(a, c.max_num_tokens, &h->tile_maps, h->aux_stream)
                                    : launch_tile_kernel(a, c.max_num_tokens, &h->tile_maps, h->aux_stream));
            timing_mark(h, 1, h->aux_stream);
            RPA_CUDA(h, cudaEventRecord(h->ev_join, h->aux_stream));
        }
        timing_mark(h, 0, s);
        // Two instantiations, of which the list needs one (known on the device only): side by side, so
        // that the idle one's CTAs leave while the other one already works.
        const bool both = c.num_q_heads / c.num_kv_heads <= 8;
        if (both) {
            RPA_CUDA(h, cudaEventRecord(h->ev_fork2, s));
            RPA_CUDA(h, cudaStreamWaitEvent(h->aux2_stream, h->ev_fork2, 0));
            RPA_CUDA(h, launch_row_kernel_fp8_strided(a, grid, false, h->aux2_stream));
            RPA_CUDA(h, cudaEventRecord(h->ev_join2, h->aux2_stream));
            RPA_CUDA(h, launch_row_kernel_fp8_strided(a, grid, true, s));
            RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_join2, 0));
        } else {
            RPA_CUDA(h, launch_row_kernel_fp8_strided(a, grid, false, s));
        }
        timing_mark(h, 0, s);
        if (tiles) RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_join, 0));
    }
    if (!capturing) {
        RPA_CUDA(h, cudaEventRecord(h->ev_dev_consumed[b], s));
        h->dev_consumed_pending[b] = true;
    }
    return RPA_OK;
}

rpa_status_t rpa_plan_device(rpa_handle_t* h, const int32_t* cu_q_lens, const int32_t* kv_lens, int32_t num_seqs,
                             void* stream) {
    if (!h || !cu_q_lens || !kv_lens || num_seqs < 0) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) {
        h->last_error = "handle was created without a CUDA device";
        return RPA_ERR_CUDA;
    }
    if (num_seqs > h->cfg.max_num_seqs) return RPA_ERR_CAPACITY;
    rpa_status_t st = ensure_device(h);
    if (st != RPA_OK) return st;
    const rpa_config_t& c = h->cfg;
    if (!h->d_dev_scratch) {  // first use: the only allocations of this path (call once before capturing a graph)
        h->dev_hist_len = (int32_t)std::min<int64_t>((int64_t)c.max_pages_per_seq * c.page_size / kKvTile + 2, 1 << 24);
        for (int b = 0; b < 2; ++b) {
            if (!h->d_dev_lists_buf[b]) RPA_CUDA(h, cudaMalloc(&h->d_dev_lists_buf[b], h->lists_bytes));
            if (!h->d_dev_counts_buf[b]) {
                RPA_CUDA(h, cudaMalloc(&h->d_dev_counts_buf[b], kDevCountInts * sizeof(int32_t)));
                RPA_CUDA(h, cudaMemset(h->d_dev_counts_buf[b], 0, kDevCountInts * sizeof(int32_t)));
            }
            if (!h->ev_dev_planned[b]) RPA_CUDA(h, cudaEventCreateWithFlags(&h->ev_dev_planned[b], cudaEventDisableTiming));
            if (!h->ev_dev_consumed[b]) RPA_CUDA(h, cudaEventCreateWithFlags(&h->ev_dev_consumed[b], cudaEventDisableTiming));
        }
        RPA_CUDA(h, cudaMalloc(&h->d_dev_scratch, ((size_t)4 * c.max_num_seqs + (size_t)2 * h->dev_hist_len) * sizeof(int32_t)));
    }
    // The plan goes into the set the latest plan does not use: kernels of the previous step may still
    // read that one.  Inside a stream capture the set never changes (a replayed graph keeps the
    // addresses it was captured with) and the capture's order replaces the events.
    cudaStream_t ps = static_cast<cudaStream_t>(stream);
    const bool capturing = stream_is_capturing(ps);
    const int b = capturing ? h->dev_cur : h->dev_cur ^ 1;
    if (!capturing && h->dev_consumed_pending[b]) {
        RPA_CUDA(h, cudaStreamWaitEvent(ps, h->ev_dev_consumed[b], 0));
        h->dev_consumed_pending[b] = false;
    }
    h->dev_cur = b;
    h->d_dev_lists = h->d_dev_lists_buf[b];
    h->d_dev_counts = h->d_dev_counts_buf[b];
    DevPlanArgs p{};
    p.cu_q_lens = cu_q_lens;
    p.kv_lens = kv_lens;
    p.num_seqs = num_seqs;
    p.rows = reinterpret_cast<RowItem*>(h->d_dev_lists);
    p.tiles = reinterpret_cast<TileItem*>(h->d_dev_lists + h->off_tiles);
    p.groups = reinterpret_cast<CombineGroup*>(h->d_dev_lists + h->off_groups);
    p.counts = h->d_dev_counts;
    p.seq_offsets = h->d_dev_scratch;
    p.hist = h->d_dev_scratch + (size_t)4 * c.max_num_seqs;
    p.status = h->d_status;
    p.hist_len = h->dev_hist_len;
    p.h_q = c.num_q_heads;
    p.h_kv = c.num_kv_heads;
    p.head_dim = c.head_dim;
    p.page_size = c.page_size;
    p.max_pages_per_seq = c.max_pages_per_seq;
    p.max_num_seqs = c.max_num_seqs;
    p.causal = c.causal ? 1 : 0;
    p.kv_elem_bytes = c.kv_dtype == RPA_KV_FP8_E4M3 ? 1 : 2;
    p.max_num_tokens = c.max_num_tokens;
    const PlanPolicy& pol = h->policy;
    p.num_slots = pol.num_slots;
    p.num_slots_narrow = pol.num_slots_narrow;
    p.kv_chunk_override = pol.kv_chunk_override;
    p.tile_min_q = pol.tile_min_q;
    p.tile_long_q = pol.tile_long_q;
    p.tile_long_kv = kTileLongKv;
    p.tile_tokens = pol.tile_tokens;
    p.pack_short = pol.pack_short ? 1 : 0;
    p.max_row_items = pol.max_row_items;
    p.max_tile_items = pol.max_tile_items;
    p.max_groups = pol.max_groups;
    p.max_partials = pol.max_partials;
    p.num_sms = pol.num_sms;
    p.tile_tflops = pol.tile_tflops;
    p.row_gbs = pol.row_gbs;
    RPA_CUDA(h, launch_plan_kernel(p, ps));
    h->dev_planned_pending[b] = false;
    if (!capturing) {
        RPA_CUDA(h, cudaEventRecord(h->ev_dev_planned[b], ps));
        h->dev_planned_pending[b] = true;
    }
    h->device_planned = true;
    h->plan.valid = false;
    h->planned_num_seqs = num_seqs;
    return RPA_OK;
}

rpa_status_t rpa_plan_device_dump(rpa_handle_t* h, int32_t* counts, int32_t* row_items, int32_t row_capacity,
                                  int32_t* tile_items, int32_t tile_capacity, int32_t* combine_groups,
                                  int32_t group_capacity) {
    if (!h || !counts) return RPA_ERR_INVALID_ARG;
    if (!h->device_planned || !h->d_dev_lists) return RPA_ERR_PLAN_MISMATCH;
    RPA_CUDA(h, cudaDeviceSynchronize());
    RPA_CUDA(h, cudaMemcpy(counts, h->d_dev_counts, kDevCountInts * sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (row_items) {
        if (row_capacity < counts[kDevCountRows]) return RPA_ERR_CAPACITY;
        RPA_CUDA(h, cudaMemcpy(row_items, h->d_dev_lists, (size_t)counts[kDevCountRows] * sizeof(RowItem), cudaMemcpyDeviceToHost));
    }
    if (tile_items) {
        if (tile_capacity < counts[kDevCountTiles]) return RPA_ERR_CAPACITY;
        RPA_CUDA(h, cudaMemcpy(tile_items, h->d_dev_lists + h->off_tiles, (size_t)counts[kDevCountTiles] * sizeof(TileItem),
                               cudaMemcpyDeviceToHost));
    }
    if (combine_groups) {
        if (group_capacity < counts[kDevCountGroups]) return RPA_ERR_CAPACITY;
        RPA_CUDA(h, cudaMemcpy(combine_groups, h->d_dev_lists + h->off_groups,
                               (size_t)counts[kDevCountGroups] * sizeof(CombineGroup), cudaMemcpyDeviceToHost));
    }
    return RPA_OK;
}

rpa_status_t rpa_forward(rpa_handle_t* h, const void* q, const void* new_k, const void* new_v, void* kv_cache,
                         const int32_t* page_table, const int32_t* cu_q_lens, const int32_t* kv_lens,
                         int32_t num_seqs, void* out, void* stream) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) {
        h->last_error = "handle was created without a CUDA device";
        return RPA_ERR_CUDA;
    }
    if (h->device_planned) {
        if (h->planned_num_seqs != num_seqs) return RPA_ERR_PLAN_MISMATCH;
        return forward_device_planned(h, q, new_k, new_v, kv_cache, page_table, cu_q_lens, kv_lens, out, stream);
    }
    if (!h->plan.valid || h->planned_num_seqs < 0 || h->planned_num_seqs != num_seqs) return RPA_ERR_PLAN_MISMATCH;
    if (h->plan.info.num_tokens == 0) return RPA_OK;
    if (!q || !new_k || !new_v || !kv_cache || !page_table || !cu_q_lens || !kv_lens || !out) return RPA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(new_k) || !aligned16(new_v) || !aligned16(kv_cache) || !aligned16(out))
        return RPA_ERR_INVALID_ARG;
    rpa_status_t st = ensure_device(h);
    if (st != RPA_OK) return st;

    uint8_t* lists = h->d_lists[h->cur];
    KernelArgs a = common_kernel_args(h, lists, h->buf_off_tiles[h->cur], h->buf_off_groups[h->cur], q, new_k, new_v, kv_cache, page_table,
                                      cu_q_lens, kv_lens, out);
    a.group_counters = h->policy.fused_combine ? h->d_group_counters : nullptr;
    a.num_row_items = (int32_t)h->plan.rows.size();
    a.num_tile_items = (int32_t)h->plan.tiles.size();
    a.num_tile_ctas = h->plan.tile_ctas;
    a.short_items = h->plan_short;
    a.row_rows_max = h->plan.row_rows_max;
    a.num_groups = (int32_t)h->plan.groups.size();
    const bool fp8 = h->cfg.kv_dtype == RPA_KV_FP8_E4M3;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_copied[h->cur], 0));  // the plan's lists have landed
    if (h->validate) {
        a.validated = 1;
        RPA_CUDA(h, launch_validate_kernel(a, num_seqs, reinterpret_cast<const int32_t*>(lists + h->buf_off_kvlens[h->cur]), s));
    }
    if (h->cfg.q_scale > 0.f)
        RPA_CUDA(h, launch_quantise_q(static_cast<const uint16_t*>(q), h->d_q_img, h->d_q_codes, h->plan.info.num_tokens, nullptr, 0,
                                      h->cfg.max_num_tokens, h->cfg.num_q_heads * h->cfg.head_dim, 1.0f / h->cfg.q_scale, h->d_status,
                                      h->validate, s));
    const bool single_tile = tile1_kernel_supported(h->cfg.head_dim, h->cfg.num_q_heads / h->cfg.num_kv_heads);
    const bool side_by_side = a.num_row_items > 0 && a.num_tile_items > 0 && !(h->ablation & kAblateOverlap);
    if (side_by_side) {
        // Mixed batch: the persistent tile kernel takes its share of the SMs on a second stream
        // (submitted first, higher priority), the row items stream through the remaining SMs.
        RPA_CUDA(h, cudaEventRecord(h->ev_fork, s));
        RPA_CUDA(h, cudaStreamWaitEvent(h->aux_stream, h->ev_fork, 0));
        timing_mark(h, 1, h->aux_stream);
        RPA_CUDA(h, h->plan_pair   ? launch_tile2_kernel(a, h->plan.info.num_tokens, &h->tile_maps, h->aux_stream)
                    : single_tile ? launch_tile1_kernel(a, h->plan.info.num_tokens, &h->tile_maps, h->aux_stream)
                                  : launch_tile_kernel(a, h->plan.info.num_tokens, &h->tile_maps, h->aux_stream));
        timing_mark(h, 1, h->aux_stream);
        RPA_CUDA(h, cudaEventRecord(h->ev_join, h->aux_stream));
        timing_mark(h, 0, s);
        RPA_CUDA(h, fp8 ? launch_row_kernel_fp8(a, s) : launch_row_kernel(a, s));
        timing_mark(h, 0, s);
        RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_join, 0));
    } else {
        if (a.num_row_items > 0) {
            timing_mark(h, 0, s);
            RPA_CUDA(h, fp8 ? launch_row_kernel_fp8(a, s) : launch_row_kernel(a, s));
            timing_mark(h, 0, s);
        }
        if (a.num_tile_items > 0) {
            a.num_tile_ctas = h->num_sms;  // one after the other: the whole device each, one persistent CTA per SM
            timing_mark(h, 1, s);
            RPA_CUDA(h, h->plan_pair   ? launch_tile2_kernel(a, h->plan.info.num_tokens, &h->tile_maps, s)
                        : single_tile ? launch_tile1_kernel(a, h->plan.info.num_tokens, &h->tile_maps, s)
                                      : launch_tile_kernel(a, h->plan.info.num_tokens, &h->tile_maps, s));
            timing_mark(h, 1, s);
        }
    }
    if (a.num_groups > 0 && a.group_counters == nullptr) {
        timing_mark(h, 2, s);
        RPA_CUDA(h, launch_combine_kernel(a, s));
        timing_mark(h, 2, s);
    }
    RPA_CUDA(h, cudaEventRecord(h->ev_consumed[h->cur], s));
    h->consumed_pending[h->cur] = true;
    return RPA_OK;
}

rpa_status_t rpa_forward_host_submit(rpa_handle_t* h, const void* q_host, const void* new_k_host,
                                     const void* new_v_host, void* kv_cache, const int32_t* page_table_host,
                                     const int32_t* cu_q_lens_host, const int32_t* kv_lens_host, int32_t num_seqs,
                                     void* out_host, void* stream) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) {
        h->last_error = "handle was created without a CUDA device";
        return RPA_ERR_CUDA;
    }
    rpa_status_t st = rpa_plan(h, cu_q_lens_host, kv_lens_host, num_seqs, stream);
    if (st != RPA_OK) return st;
    const rpa_config_t& c = h->cfg;
    if (!h->d_host_stage[1]) {  // (the last thing the set-up creates)
        const size_t qb = (size_t)c.max_num_tokens * c.num_q_heads * c.head_dim * 2;
        const size_t kb = (size_t)c.max_num_tokens * c.num_kv_heads * c.head_dim * 2;
        h->hs_q = 0;
        h->hs_k = align_up(h->hs_q + qb, 256);
        h->hs_v = align_up(h->hs_k + kb, 256);
        h->hs_out = align_up(h->hs_v + kb, 256);
        h->hs_pt = align_up(h->hs_out + qb, 256);
        h->hs_cu = align_up(h->hs_pt + (size_t)c.max_num_seqs * c.max_pages_per_seq * 4, 256);
        h->hs_kl = align_up(h->hs_cu + ((size_t)c.max_num_seqs + 1) * 4, 256);
        h->hs_bytes = align_up(h->hs_kl + (size_t)c.max_num_seqs * 4, 256);
        if (!h->h2d_stream) RPA_CUDA(h, cudaStreamCreateWithFlags(&h->h2d_stream, cudaStreamNonBlocking));
        if (!h->d2h_stream) RPA_CUDA(h, cudaStreamCreateWithFlags(&h->d2h_stream, cudaStreamNonBlocking));
        for (int b = 0; b < 2; ++b) {
            if (!h->ev_in[b]) RPA_CUDA(h, cudaEventCreateWithFlags(&h->ev_in[b], cudaEventDisableTiming));
            if (!h->ev_ran[b]) RPA_CUDA(h, cudaEventCreateWithFlags(&h->ev_ran[b], cudaEventDisableTiming));
            if (!h->ev_out[b]) RPA_CUDA(h, cudaEventCreateWithFlags(&h->ev_out[b], cudaEventDisableTiming));
            if (!h->d_host_stage[b]) RPA_CUDA(h, cudaMalloc(&h->d_host_stage[b], h->hs_bytes));
        }
    }
    const int64_t T = h->plan.info.num_tokens;
    const bool empty = T == 0 || num_seqs == 0;
    if (!empty && (!q_host || !new_k_host || !new_v_host || !page_table_host || !out_host || !kv_cache)) return RPA_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int slot = (int)(h->hs_submitted & 1);
    uint8_t* d = h->d_host_stage[slot];
    // The slot's previous step (two submits ago) must have delivered its output before the slot's
    // buffers are overwritten; an event that was never recorded counts as complete.
    RPA_CUDA(h, cudaStreamWaitEvent(h->h2d_stream, h->ev_out[slot], 0));
    if (!empty) {
        const size_t q_row = (size_t)c.num_q_heads * c.head_dim * 2, k_row = (size_t)c.num_kv_heads * c.head_dim * 2;
        RPA_CUDA(h, cudaMemcpyAsync(d + h->hs_q, q_host, T * q_row, cudaMemcpyHostToDevice, h->h2d_stream));
        RPA_CUDA(h, cudaMemcpyAsync(d + h->hs_k, new_k_host, T * k_row, cudaMemcpyHostToDevice, h->h2d_stream));
        RPA_CUDA(h, cudaMemcpyAsync(d + h->hs_v, new_v_host, T * k_row, cudaMemcpyHostToDevice, h->h2d_stream));
        RPA_CUDA(h, cudaMemcpyAsync(d + h->hs_pt, page_table_host, (size_t)num_seqs * c.max_pages_per_seq * 4,
                                    cudaMemcpyHostToDevice, h->h2d_stream));
        // (the lengths travel with the plan's lists: one copy less each)
    }
    RPA_CUDA(h, cudaEventRecord(h->ev_in[slot], h->h2d_stream));
    RPA_CUDA(h, cudaStreamWaitEvent(s, h->ev_in[slot], 0));
    if (!empty) {
        const uint8_t* lists = h->d_lists[h->cur];
        st = rpa_forward(h, d + h->hs_q, d + h->hs_k, d + h->hs_v, kv_cache, reinterpret_cast<const int32_t*>(d + h->hs_pt),
                         reinterpret_cast<const int32_t*>(lists + h->buf_off_cu[h->cur]),
                         reinterpret_cast<const int32_t*>(lists + h->buf_off_kvlens[h->cur]), num_seqs, d + h->hs_out, stream);
        if (st != RPA_OK) return st;
    }
    RPA_CUDA(h, cudaEventRecord(h->ev_ran[slot], s));
    RPA_CUDA(h, cudaStreamWaitEvent(h->d2h_stream, h->ev_ran[slot], 0));
    if (!empty) {
        const size_t q_row = (size_t)c.num_q_heads * c.head_dim * 2;
        RPA_CUDA(h, cudaMemcpyAsync(out_host, d + h->hs_out, T * q_row, cudaMemcpyDeviceToHost, h->d2h_stream));
    }
    RPA_CUDA(h, cudaEventRecord(h->ev_out[slot], h->d2h_stream));
    ++h->hs_submitted;
    return RPA_OK;
}

rpa_status_t rpa_forward_host_wait(rpa_handle_t* h) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) {
        h->last_error = "handle was created without a CUDA device";
        return RPA_ERR_CUDA;
    }
    if (h->hs_waited == h->hs_submitted) return RPA_OK;  // nothing outstanding
    // (with more than two steps outstanding the slot's event belongs to a later step, whose end implies this one's)
    RPA_CUDA(h, cudaEventSynchronize(h->ev_out[h->hs_waited & 1]));
    ++h->hs_waited;
    return RPA_OK;
}

rpa_status_t rpa_forward_host(rpa_handle_t* h, const void* q_host, const void* new_k_host, const void* new_v_host,
                              void* kv_cache, const int32_t* page_table_host, const int32_t* cu_q_lens_host,
                              const int32_t* kv_lens_host, int32_t num_seqs, void* out_host, void* stream) {
    rpa_status_t st = rpa_forward_host_submit(h, q_host, new_k_host, new_v_host, kv_cache, page_table_host, cu_q_lens_host,
                                              kv_lens_host, num_seqs, out_host, stream);
    if (st != RPA_OK) return st;
    while (h->hs_waited < h->hs_submitted) {  // this step and any submitted before it
        st = rpa_forward_host_wait(h);
        if (st != RPA_OK) return st;
    }
    return RPA_OK;
}

rpa_status_t rpa_plan_info(const rpa_handle_t* h, rpa_plan_info_t* info) {
    if (!h || !info) return RPA_ERR_INVALID_ARG;
    if (!h->plan.valid) return RPA_ERR_PLAN_MISMATCH;
    *info = h->plan.info;
    return RPA_OK;
}

rpa_status_t rpa_plan_dump(const rpa_handle_t* h, int32_t* row_items, int32_t row_capacity, int32_t* tile_items,
                           int32_t tile_capacity, int32_t* combine_groups, int32_t group_capacity) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (!h->plan.valid) return RPA_ERR_PLAN_MISMATCH;
    if (row_items) {
        if ((size_t)row_capacity < h->plan.rows.size()) return RPA_ERR_CAPACITY;
        memcpy(row_items, h->plan.rows.data(), h->plan.rows.size() * sizeof(RowItem));
    }
    if (tile_items) {
        if ((size_t)tile_capacity < h->plan.tiles.size()) return RPA_ERR_CAPACITY;
        memcpy(tile_items, h->plan.tiles.data(), h->plan.tiles.size() * sizeof(TileItem));
    }
    if (combine_groups) {
        if ((size_t)group_capacity < h->plan.groups.size()) return RPA_ERR_CAPACITY;
        memcpy(combine_groups, h->plan.groups.data(), h->plan.groups.size() * sizeof(CombineGroup));
    }
    return RPA_OK;
}

rpa_status_t rpa_poll_status(rpa_handle_t* h, void* stream, uint32_t* detail) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) return RPA_ERR_CUDA;
    uint32_t word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RPA_CUDA(h, cudaMemcpyAsync(&word, h->d_status, sizeof word, cudaMemcpyDeviceToHost, s));
    RPA_CUDA(h, cudaStreamSynchronize(s));
    if (detail) *detail = word;
    if (word == 0) return RPA_OK;
    RPA_CUDA(h, cudaMemsetAsync(h->d_status, 0, sizeof word, s));  // reported once
    RPA_CUDA(h, cudaStreamSynchronize(s));
    return (word & (1u << 28)) ? RPA_ERR_TIMEOUT : RPA_ERR_INVALID_ARG;
}

rpa_status_t rpa_selftest_bounded_wait(rpa_handle_t* h, void* stream) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) return RPA_ERR_CUDA;
    rpa_status_t st = ensure_device(h);
    if (st != RPA_OK) return st;
    RPA_CUDA(h, launch_wait_selftest(h->d_status, static_cast<cudaStream_t>(stream)));
    return RPA_OK;
}

rpa_status_t rpa_set_validation(rpa_handle_t* h, int32_t enable) {
    if (!h) return RPA_ERR_INVALID_ARG;
    h->validate = enable != 0;
    return RPA_OK;
}

rpa_status_t rpa_set_ablation(rpa_handle_t* h, uint32_t mask) {
    if (!h) return RPA_ERR_INVALID_ARG;
    h->ablation = mask;
    return RPA_OK;
}

rpa_status_t rpa_set_kernel_timing(rpa_handle_t* h, int32_t enable) {
    if (!h) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) return RPA_ERR_CUDA;
    h->timing = enable != 0;
    for (size_t& u : h->ev_used) u = 0;
    return RPA_OK;
}

rpa_status_t rpa_get_kernel_timing(rpa_handle_t* h, float* total_ms, int32_t* launches) {
    if (!h || !total_ms || !launches) return RPA_ERR_INVALID_ARG;
    if (h->plan_only) return RPA_ERR_CUDA;
    for (int k = 0; k < 3; ++k) {
        total_ms[k] = 0.f;
        launches[k] = 0;
        const size_t pairs = h->ev_used[k] / 2;
        if (pairs) RPA_CUDA(h, cudaEventSynchronize(h->ev[k][2 * pairs - 1]));
        for (size_t i = 0; i < pairs; ++i) {
            float ms = 0.f;
            RPA_CUDA(h, cudaEventElapsedTime(&ms, h->ev[k][2 * i], h->ev[k][2 * i + 1]));
            total_ms[k] += ms;
            launches[k]++;
        }
    }
    return RPA_OK;
}

rpa_status_t rpa_set_tile_min_q(rpa_handle_t* h, int32_t tokens) {
    if (!h || tokens < 0) return RPA_ERR_INVALID_ARG;
    const int h_g = h->cfg.num_q_heads / h->cfg.num_kv_heads;
    h->policy.tile_min_q = tokens == 0 ? default_tile_min_q(h_g) : tokens;
    h->policy.tile_long_q = tokens == 0 ? std::max(2, kRowTileRows / h_g + 1) : 0;  // an explicit threshold is the only rule
    if (!tile_path_available(h->cfg)) h->policy.tile_min_q = h->policy.tile_long_q = 0;
    h->policy.pack_short = tokens == 0 && h->policy.tile_min_q > 0 && !tile1_kernel_supported(h->cfg.head_dim, h_g);
    h->plan.valid = false;
    h->planned_num_seqs = -1;
    return RPA_OK;
}

rpa_status_t rpa_set_tile_pair(rpa_handle_t* h, int32_t mode) {
    if (!h || mode < 0 || mode > 2) return RPA_ERR_INVALID_ARG;
    const int h_g = h->cfg.num_q_heads / h->cfg.num_kv_heads;
    if (mode == 1 && (h->cfg.kv_dtype != RPA_KV_BF16 || !tile2_kernel_supported(h->cfg.head_dim, h_g))) return RPA_ERR_UNSUPPORTED;
    h->tile_pair_mode = mode;
    h->plan.valid = false;
    h->planned_num_seqs = -1;
    return RPA_OK;
}

rpa_status_t rpa_set_kv_chunk(rpa_handle_t* h, int32_t tokens) {
    if (!h || tokens < 0) return RPA_ERR_INVALID_ARG;
    h->policy.kv_chunk_override = tokens;
    h->plan.valid = false;
    h->planned_num_seqs = -1;
    return RPA_OK;
}

const char* rpa_status_string(rpa_status_t s) {
    switch (s) {
        case RPA_OK: return "ok";
        case RPA_ERR_INVALID_ARG: return "invalid argument";
        case RPA_ERR_UNSUPPORTED: return "unsupported shape";
        case RPA_ERR_CAPACITY: return "capacity exceeded";
        case RPA_ERR_PLAN_MISMATCH: return "no matching plan";
        case RPA_ERR_CUDA: return "CUDA error";
        case RPA_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

const char* rpa_last_cuda_error(const rpa_handle_t* h) { return h ? h->last_error.c_str() : ""; }

}  // extern "C"
