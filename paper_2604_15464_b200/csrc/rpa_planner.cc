#include "rpa_planner.h"

#include <algorithm>
#include <limits.h>

namespace rpa {

namespace {

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up(int64_t a, int64_t b) { return ceil_div(a, b) * b; }

// Stable counting sort of the row items by KV tiles, longest first: the hardware dispatches CTAs
// in index order, so this is longest-processing-time-first list scheduling over the SM slots.
void sort_longest_first(Plan& plan) {
    const size_t n = plan.rows.size();
    if (n < 2) return;
    uint32_t max_tiles = 0;
    plan.sort_keys.resize(n);
    for (size_t i = 0; i < n; ++i) {
        const RowItem& it = plan.rows[i];
        uint32_t tiles = (uint32_t)ceil_div(it.kv_end - it.kv_begin, kKvTile);
        plan.sort_keys[i] = tiles;
        max_tiles = std::max(max_tiles, tiles);
    }
    plan.sort_count.assign((size_t)max_tiles + 2, 0);
    for (size_t i = 0; i < n; ++i) plan.sort_count[max_tiles - plan.sort_keys[i] + 1]++;
    for (size_t b = 1; b < plan.sort_count.size(); ++b) plan.sort_count[b] += plan.sort_count[b - 1];
    plan.sort_scratch.resize(n);
    for (size_t i = 0; i < n; ++i) plan.sort_scratch[plan.sort_count[max_tiles - plan.sort_keys[i]]++] = plan.rows[i];
    plan.rows.swap(plan.sort_scratch);
}

// Which kernel serves a sequence.  From three row items' worth of query rows on, the tile kernel
// wins everywhere.  With two row items' worth it wins only where it streams keys faster than two row
// items re-reading them: long contexts on pages of at least 64 slots (one TMA box per page; with
// small pages the number of boxes, not HBM, paces it).
inline bool routed_to_tile(const rpa_config_t& cfg, const PlanPolicy& policy, int64_t q_r, int64_t L_r) {
    if (policy.tile_min_q <= 0) return false;
    if (q_r >= policy.tile_min_q) return true;
    return policy.tile_long_q > 0 && q_r >= policy.tile_long_q && L_r >= kTileLongKv && cfg.page_size >= kTileLongPage;
}

}  // namespace

bool sequence_routed_to_tile(const rpa_config_t& cfg, const PlanPolicy& policy, int64_t q_len, int64_t kv_len) {
    return routed_to_tile(cfg, policy, q_len, kv_len);
}

rpa_status_t build_plan(const rpa_config_t& cfg, const PlanPolicy& policy, const int32_t* cu_q_lens,
                        const int32_t* kv_lens, int32_t num_seqs, Plan& plan) {
    plan.valid = false;
    plan.rows.clear();
    plan.tiles.clear();
    plan.groups.clear();
    plan.num_partials = 0;
    plan.row_rows_max = 0;
    plan.info = rpa_plan_info_t{};
    if (!cu_q_lens || !kv_lens || num_seqs < 0) return RPA_ERR_INVALID_ARG;
    if (num_seqs > cfg.max_num_seqs) return RPA_ERR_CAPACITY;
    if (cu_q_lens[0] != 0) return RPA_ERR_INVALID_ARG;

    const int h_g = cfg.num_q_heads / cfg.num_kv_heads;
    const int tpi = kRowTileRows / h_g;  // tokens per row item
    const int ps = cfg.page_size;
    const bool causal = cfg.causal != 0;

    // pass 0: validate the lengths
    for (int r = 0; r < num_seqs; ++r) {
        const int64_t q_r = (int64_t)cu_q_lens[r + 1] - cu_q_lens[r];
        const int64_t L_r = kv_lens[r];
        if (q_r < 0 || L_r < q_r) return RPA_ERR_INVALID_ARG;
        if (ceil_div(L_r, ps) > cfg.max_pages_per_seq) return RPA_ERR_CAPACITY;
    }
    // Short-sequence packing (the remedy Section 5 of the paper names for short sequences): a run
    // of consecutive sequences without cached context whose tokens fit one tile item becomes a
    // single item instead of one mostly empty item each.
    plan.pack_len.assign((size_t)num_seqs, 0);
    if (policy.pack_short && policy.tile_min_q > 0) {
        for (int r = 0; r < num_seqs;) {
            int m = 0;
            int64_t tokens = 0;
            while (r + m < num_seqs && m < kMaxPackedSeqs) {
                const int64_t q = (int64_t)cu_q_lens[r + m + 1] - cu_q_lens[r + m];
                if (q < 1 || kv_lens[r + m] != q || tokens + q > policy.tile_tokens) break;
                tokens += q;
                ++m;
            }
            if (m >= 2) {
                plan.pack_len[r] = m;
                for (int k = 1; k < m; ++k) plan.pack_len[r + k] = -1;
                r += m;
            } else {
                ++r;
            }
        }
    }

    // pass 1: classify, count work
    int64_t bytes = 0, pairs = 0, row_tokens = 0, row_bytes = 0, tile_pairs = 0, tile_kv_bytes = 0;
    int n_decode = 0, n_prefill = 0;
    int64_t row_rows = 0;  // most query rows of any row item
    for (int r = 0; r < num_seqs; ++r) {
        const int64_t q_r = (int64_t)cu_q_lens[r + 1] - cu_q_lens[r];
        const int64_t L_r = kv_lens[r];
        if (q_r == 0) continue;
        if (q_r == 1) ++n_decode; else ++n_prefill;
        const int64_t kv_elem_bytes = cfg.kv_dtype == RPA_KV_FP8_E4M3 ? 1 : 2;
        const int64_t seq_bytes = (L_r + q_r) * 2 * cfg.num_kv_heads * cfg.head_dim * kv_elem_bytes +
                                  q_r * 2 * cfg.num_q_heads * cfg.head_dim * 2;
        const int64_t seq_pairs = causal ? q_r * (L_r - q_r) + q_r * (q_r + 1) / 2 : q_r * L_r;
        bytes += seq_bytes;
        pairs += seq_pairs;
        const bool to_tile = plan.pack_len[r] != 0 || routed_to_tile(cfg, policy, q_r, L_r);
        if (to_tile) {
            tile_pairs += seq_pairs;
            tile_kv_bytes += L_r * 2 * cfg.num_kv_heads * cfg.head_dim * kv_elem_bytes;
        } else {
            row_bytes += seq_bytes;
            row_rows = std::max(row_rows, std::min<int64_t>(tpi, q_r) * h_g);
            for (int64_t t0 = 0; t0 < q_r; t0 += tpi) {
                const int64_t nt = std::min<int64_t>(tpi, q_r - t0);
                row_tokens += (causal ? L_r - q_r + t0 + nt : L_r) * cfg.num_kv_heads;
            }
        }
    }
    const int64_t T = cu_q_lens[num_seqs];
    if (T > cfg.max_num_tokens) return RPA_ERR_CAPACITY;

    // split-KV chunk: no item longer than half (1 / kChunkDivisor) of a slot's average share, never below 256
    const int num_slots = policy.num_slots_narrow > 0 && row_rows <= 8 ? policy.num_slots_narrow : policy.num_slots;
    int64_t chunk = policy.kv_chunk_override;
    if (chunk <= 0) {
        const int64_t per_slot = row_tokens / std::max(num_slots, 1);
        chunk = std::max<int64_t>(256, round_up(per_slot / kChunkDivisor, 64));
    }
    chunk = round_up(chunk, kKvTile);
    if (chunk > INT_MAX / 2) chunk = INT_MAX / 2 / kKvTile * kKvTile;
    if (policy.kv_chunk_override <= 0 && row_tokens > 0) {
        // A small batch runs in a few waves of CTAs, and a last wave that is nearly empty costs as
        // much as a full one: try chunks around the default and keep the best estimate.
        const int64_t slots = std::max(num_slots, 1);
        int64_t split_items = 0;  // of the last count_items call
        auto count_items = [&](int64_t c) {
            int64_t items = 0;
            split_items = 0;
            for (int r = 0; r < num_seqs; ++r) {
                const int64_t q_r = (int64_t)cu_q_lens[r + 1] - cu_q_lens[r], L_r = kv_lens[r];
                if (q_r == 0 || plan.pack_len[r] != 0 || routed_to_tile(cfg, policy, q_r, L_r)) continue;
                for (int64_t t0 = 0; t0 < q_r; t0 += tpi) {
                    const int64_t ve = causal ? L_r - q_r + t0 + std::min<int64_t>(tpi, q_r - t0) : L_r;
                    const int64_t ns = ceil_div(ve, c), part = round_up(ceil_div(ve, ns), kKvTile);
                    const int64_t emitted = std::min(ns, ceil_div(ve, part));
                    items += emitted * cfg.num_kv_heads;
                    if (emitted > 1) split_items += emitted * cfg.num_kv_heads;
                }
            }
            return items;
        };
        auto estimate = [&](int64_t items) {  // uses split_items of the count that produced `items`
            const int64_t fixed = kItemFixedKeys * (items - split_items) + kSplitItemFixedKeys * split_items;
            return ceil_div(items, slots) * ((fixed + row_tokens) / items);
        };
        const int64_t base_items = count_items(chunk);
        if (base_items < kRefineWaves * slots) {
            int64_t best = chunk, best_cost = estimate(base_items);
            for (int f : kRefineFactors) {
                const int64_t c = std::max<int64_t>(256, round_up(chunk * f / 16, kKvTile));
                const int64_t cost = estimate(count_items(c));
                if (cost * 100 < best_cost * 97) {
                    best = c;
                    best_cost = cost;
                }
            }
            chunk = best;
        }
    }

    // pass 2: emit items
    for (int r = 0; r < num_seqs; ++r) {
        const int q_r = cu_q_lens[r + 1] - cu_q_lens[r];
        const int L_r = kv_lens[r];
        if (q_r == 0) continue;
        const int c_r = L_r - q_r;
        if (plan.pack_len[r] < 0) continue;  // inside a packed run: its item was emitted at the run's first sequence
        if (plan.pack_len[r] > 0) {
            const int m = plan.pack_len[r];
            for (int h = 0; h < cfg.num_kv_heads; ++h) {
                if ((int)plan.tiles.size() >= policy.max_tile_items) return RPA_ERR_CAPACITY;
                TileItem it{};
                it.seq = r;
                it.kv_head = h;
                it.q_tok0 = 0;
                it.n_tok = cu_q_lens[r + m] - cu_q_lens[r];
                it.flags = kFlagWriteKv | kFlagPacked;
                it.n_seqs = m;
                plan.tiles.push_back(it);
            }
            continue;
        }
        const bool to_tile = routed_to_tile(cfg, policy, q_r, L_r);
        if (to_tile) {
            // One KV head after the other, latest (heaviest) query tile first inside a head: CTAs that
            // run together walk the same K/V stream, which then stays in L2 (16 MB per head at 32K
            // tokens), and the lightest items of the last head come last.
            const int tt = policy.tile_tokens;
            for (int h = 0; h < cfg.num_kv_heads; ++h) {
                for (int t0 = (q_r - 1) / tt * tt; t0 >= 0; t0 -= tt) {
                    if ((int)plan.tiles.size() >= policy.max_tile_items) return RPA_ERR_CAPACITY;
                    TileItem it{};
                    it.seq = r;
                    it.kv_head = h;
                    it.q_tok0 = t0;
                    it.n_tok = std::min(tt, q_r - t0);
                    it.flags = kFlagWriteKv;
                    plan.tiles.push_back(it);
                }
            }
            continue;
        }
        for (int t0 = 0; t0 < q_r; t0 += tpi) {
            const int nt = std::min(tpi, q_r - t0);
            const int visible_end = causal ? c_r + t0 + nt : L_r;
            const int n_split = (int)ceil_div(visible_end, chunk);
            // equal parts, boundaries on KV tiles
            const int part = (int)round_up(ceil_div(visible_end, n_split), kKvTile);
            for (int h = 0; h < cfg.num_kv_heads; ++h) {
                int first_partial = -1;
                if (n_split > 1) {
                    if ((int)plan.groups.size() >= policy.max_groups) return RPA_ERR_CAPACITY;
                    if (plan.num_partials + n_split > policy.max_partials) return RPA_ERR_CAPACITY;
                    first_partial = plan.num_partials;
                    plan.num_partials += n_split;
                }
                int emitted = 0;
                for (int k = 0; k < n_split; ++k) {
                    const int b = k * part;
                    const int e = std::min(visible_end, b + part);
                    if (b >= e) continue;  // rounding can leave the last part empty
                    if ((int)plan.rows.size() >= policy.max_row_items) return RPA_ERR_CAPACITY;
                    RowItem it{};
                    it.seq = r;
                    it.kv_head = h;
                    it.q_tok0 = t0;
                    it.n_tok = nt;
                    it.kv_begin = b;
                    it.kv_end = e;
                    it.partial = n_split > 1 ? first_partial + emitted : -1;
                    it.flags = e == visible_end ? kFlagWriteKv : 0;
                    if (n_split > 1) it.flags |= (int32_t)(plan.groups.size() + 1) << kFlagGroupShift;
                    plan.rows.push_back(it);
                    plan.row_rows_max = std::max(plan.row_rows_max, nt * h_g);
                    ++emitted;
                }
                if (n_split > 1) {
                    if (emitted == 1) {  // degenerate: nothing left to combine
                        plan.rows.back().partial = -1;
                        plan.rows.back().flags &= (1 << kFlagGroupShift) - 1;
                        plan.num_partials -= n_split;
                    } else {
                        plan.num_partials -= n_split - emitted;
                        CombineGroup g{};
                        g.out_tok0 = cu_q_lens[r] + t0;
                        g.n_tok = nt;
                        g.kv_head = h;
                        g.first_partial = first_partial;
                        g.n_partials = emitted;
                        plan.groups.push_back(g);
                    }
                }
            }
        }
    }
    sort_longest_first(plan);

    // Tile items come one KV head after the other so that CTAs running together share a K/V stream
    // in L2.  When the K/V of all tile-routed sequences fits L2 several times over anyway, that
    // order only delays the heavy items of the later heads: then the items are put heaviest first
    // across heads (stable, so equal items keep the head order).
    if (!plan.tiles.empty() && tile_kv_bytes <= kTileGlobalOrderBytes) {
        auto blocks_of = [&](const TileItem& it) {
            if (it.flags & kFlagPacked) return 1;
            const int q = cu_q_lens[it.seq + 1] - cu_q_lens[it.seq], ctx = kv_lens[it.seq] - q;
            return (ctx + kQTile - 1) / kQTile + ((causal ? std::min(q, it.q_tok0 + it.n_tok) : q) + kQTile - 1) / kQTile;
        };
        std::stable_sort(plan.tiles.begin(), plan.tiles.end(),
                         [&](const TileItem& x, const TileItem& y) { return blocks_of(x) > blocks_of(y); });
    }

    rpa_plan_info_t& info = plan.info;
    info.num_seqs = num_seqs;
    info.num_tokens = (int32_t)T;
    info.num_decode_seqs = n_decode;
    info.num_prefill_seqs = n_prefill;
    info.batch_case = (n_decode && n_prefill) ? RPA_CASE_MIXED
                      : n_decode              ? RPA_CASE_DECODE
                      : n_prefill             ? RPA_CASE_PREFILL
                                              : RPA_CASE_EMPTY;
    info.num_row_items = (int32_t)plan.rows.size();
    info.num_tile_items = (int32_t)plan.tiles.size();
    info.num_combine_groups = (int32_t)plan.groups.size();
    info.kv_chunk_tokens = (int32_t)std::min<int64_t>(chunk, INT_MAX);
    // (an FP8 cache adds the quantising pass that runs before the tile kernel)
    info.gpu_launches = (plan.rows.empty() ? 0 : 1) + (plan.tiles.empty() ? 0 : cfg.kv_dtype == RPA_KV_FP8_E4M3 ? 2 : 1) +
                        ((plan.groups.empty() || policy.fused_combine) ? 0 : 1) +
                        ((cfg.q_scale > 0.f && T > 0) ? 1 : 0);  // the pass that quantises Q
    info.algorithmic_bytes = bytes;
    info.algorithmic_flops = 4 * (int64_t)cfg.num_q_heads * cfg.head_dim * pairs;
    // SM split for mixed batches: the tile kernel is persistent on tile_ctas SMs while row items
    // stream through the others (the two kernels cannot share an SM: their shared memory adds up
    // to more than an SM has).  Give the tensor-bound part just enough SMs to finish together with
    // the HBM-bound part, which keeps its bandwidth as long as about half the SMs remain.
    plan.tile_ctas = 0;  // 0: one CTA per item, scheduled by the hardware over the whole device
    if (!plan.rows.empty() && !plan.tiles.empty()) {
        const double t_tile = 4.0 * cfg.num_q_heads * cfg.head_dim * (double)tile_pairs / (policy.tile_tflops * 1e12);
        const double t_row = (double)row_bytes / (policy.row_gbs * 1e9);
        int n = (int)(policy.num_sms * t_tile / std::max(t_row, 1e-9) + 0.5);
        plan.tile_ctas = std::min(std::max(n, policy.num_sms / 8), policy.num_sms * 5 / 8);
        plan.tile_ctas = std::min<int>(plan.tile_ctas, (int)plan.tiles.size());
    }
    info.row_bytes = row_bytes;
    info.tile_flops = 4 * (int64_t)cfg.num_q_heads * cfg.head_dim * tile_pairs;
    info.workspace_bytes =
        (int64_t)plan.num_partials * kRowTileRows * ((int64_t)cfg.head_dim * 4 + 8);
    plan.valid = true;
    return RPA_OK;
}

}  // namespace rpa
