// Device-side planner: builds the work lists of a batch from the device copies of its lengths, so
// that a step (plan + attention) needs no host round trip and can be captured in a CUDA graph and
// replayed with new lengths.  It applies the same rules as the host planner (routing, split-KV
// chunking, combine groups, longest items first); batches of more than 1024
// sequences are not searched for runs of short sequences to pack, and the order among row items of
// equal length is whatever the atomics give.
//
// One CTA.  Phases, separated by CTA-wide barriers:
//   1. per sequence: validate, route, count the keys the row items will stream  -> split-KV chunk
//   2. per sequence: count row items, tile items, combine groups, split partials -> exclusive scans
//   3. histogram of the row items' lengths (in KV tiles)                          -> bucket starts
//   4. emit: row items into their length bucket, tile items and groups at their scanned offsets
//   5. counts, SM split between the two kernels, error word
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "rpa_kernels.h"
#include "rpa_types.h"

namespace rpa {

__device__ constexpr int kRefineFactorsDev[8] = {8, 10, 12, 14, 18, 20, 24, 32};
static_assert(kRefineFactorsDev[0] == kRefineFactors[0] && kRefineFactorsDev[7] == kRefineFactors[7], "same factors as the host planner");

namespace {

constexpr int kPlanThreads = 1024;
constexpr int kSmemSeqs = 1024;
constexpr int kSmemBuckets = 4096;  // row-item length buckets kept in shared memory

__device__ __forceinline__ int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
__device__ __forceinline__ int64_t round_up64(int64_t a, int64_t b) { return ceil_div64(a, b) * b; }

__device__ __forceinline__ bool dev_routed_to_tile(const DevPlanArgs& p, int64_t q_r, int64_t L_r) {
    if (p.tile_min_q <= 0) return false;
    if (q_r >= p.tile_min_q) return true;
    return p.tile_long_q > 0 && q_r >= p.tile_long_q && L_r >= p.tile_long_kv && p.page_size >= kTileLongPage;
}

// The split of one row unit (up to tpi tokens of one sequence starting at t0), as the host planner
// computes it: `emitted` non-empty parts of `part` keys each (the last one shorter).
struct UnitSplit {
    int nt, visible_end, part, emitted;
};
__device__ __forceinline__ UnitSplit split_unit(const DevPlanArgs& p, int q_r, int c_r, int L_r, int t0, int tpi, int64_t chunk) {
    UnitSplit u;
    u.nt = min(tpi, q_r - t0);
    u.visible_end = p.causal ? c_r + t0 + u.nt : L_r;
    // 32-bit arithmetic: visible_end < 2^31 and chunk <= 2^30 (64-bit division is a long subroutine)
    const uint32_t ve = (uint32_t)u.visible_end, ch = (uint32_t)chunk;
    const uint32_t n_split = (ve + ch - 1) / ch;
    const uint32_t part = ((ve + n_split - 1) / n_split + kKvTile - 1) / kKvTile * kKvTile;
    u.part = (int)part;
    u.emitted = (int)min(n_split, (ve + part - 1) / part);
    return u;
}

// Exclusive scan of one int per thread across the CTA; returns this thread's prefix, `total` for all.
__device__ int block_exclusive_scan(int v, int* smem_warp, int& total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += n;
    }
    __syncthreads();  // smem_warp may still be read from a previous call
    if (lane == 31) smem_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = smem_warp[lane];
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int n = __shfl_up_sync(0xffffffffu, wi, d);
            if (lane >= d) wi += n;
        }
        smem_warp[lane] = wi - w;       // exclusive prefix of the warp totals
        if (lane == 31) smem_warp[32] = wi;
    }
    __syncthreads();
    total = smem_warp[32];
    return smem_warp[warp] + incl - v;
}

__device__ int64_t block_sum64(int64_t v, int64_t* smem64) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) smem64[threadIdx.x >> 5] = v;
    __syncthreads();
    int64_t t = 0;
    for (int w = 0; w < kPlanThreads / 32; ++w) t += smem64[w];
    return t;
}

}  // namespace

__global__ void __launch_bounds__(kPlanThreads, 1) rpa_plan_kernel(const DevPlanArgs p) {
    __shared__ int s_warp[33];
    __shared__ int64_t s_64[kPlanThreads / 32];
    __shared__ int s_error;
    __shared__ int s_row_rows;  // most query rows of any row item
    __shared__ int s_carry[4];
    __shared__ int s_off_tile[kSmemSeqs], s_q_len[kSmemSeqs];  // per-sequence data of small batches, for the tile emit
    const int tid = threadIdx.x;
    const int n = p.num_seqs;
    const int h_g = p.h_q / p.h_kv;
    const int tpi = kRowTileRows / h_g;
    const int ps = p.page_size;
    int* off_row = p.seq_offsets;  // four arrays of max_num_seqs ints: where each sequence's entries start
    int* off_tile = off_row + p.max_num_seqs;
    int* off_group = off_tile + p.max_num_seqs;
    int* off_part = off_group + p.max_num_seqs;

    if (tid == 0) s_error = s_row_rows = 0;
    // ---- phase 0: short-sequence packing (batches of up to kSmemSeqs sequences), the host planner's
    // greedy walk made parallel: every thread finds where a group that starts at its sequence would
    // end; then one thread per maximal run of packable sequences hops from group to group.
    // s_pack[r] = sequences in the group that starts at r, -1 inside a group, 0 otherwise ----
    __shared__ signed char s_pack[kSmemSeqs], s_group_len[kSmemSeqs];
    const bool packing = p.pack_short && p.tile_min_q > 0 && n <= kSmemSeqs;
    if (packing) {
        for (int r = tid; r < n; r += kPlanThreads) {
            const int q = p.cu_q_lens[r + 1] - p.cu_q_lens[r];
            s_q_len[r] = (q >= 1 && q <= p.tile_tokens && p.kv_lens[r] == q) ? q : 0;  // 0: cannot be packed
            s_pack[r] = 0;
        }
        __syncthreads();
        for (int r = tid; r < n; r += kPlanThreads) {
            int m = 0, tokens = 0;
            while (r + m < n && m < kMaxPackedSeqs && s_q_len[r + m] > 0 && tokens + s_q_len[r + m] <= p.tile_tokens) {
                tokens += s_q_len[r + m];
                ++m;
            }
            s_group_len[r] = (signed char)m;
        }
        __syncthreads();
        for (int r = tid; r < n; r += kPlanThreads) {
            if (s_q_len[r] == 0 || (r > 0 && s_q_len[r - 1] > 0)) continue;  // not the first of a run
            for (int i = r; i < n && s_q_len[i] > 0;) {
                const int m = s_group_len[i];
                if (m >= 2) {
                    s_pack[i] = (signed char)m;
                    for (int k = 1; k < m; ++k) s_pack[i + k] = -1;
                    i += m;
                } else {
                    ++i;
                }
            }
        }
    }
    __syncthreads();
    auto to_tile = [&](int r, int64_t q_r, int64_t L_r) {
        return (packing && s_pack[r] != 0) || dev_routed_to_tile(p, q_r, L_r);
    };

    // ---- phase 1: validate, route, count streamed keys ----
    int64_t row_tokens = 0, row_bytes = 0, tile_pairs = 0;
    for (int r = tid; r < n; r += kPlanThreads) {
        const int64_t q_r = (int64_t)p.cu_q_lens[r + 1] - p.cu_q_lens[r];
        const int64_t L_r = p.kv_lens[r];
        if (q_r < 0 || q_r > p.max_num_tokens || L_r < q_r || ceil_div64(L_r, ps) > p.max_pages_per_seq ||
            (r == 0 && p.cu_q_lens[0] != 0)) {
            atomicOr(&s_error, 1);
            continue;
        }
        if (q_r == 0) continue;
        const int64_t seq_pairs = p.causal ? q_r * (L_r - q_r) + q_r * (q_r + 1) / 2 : q_r * L_r;
        if (to_tile(r, q_r, L_r)) {
            tile_pairs += seq_pairs;
        } else {
            row_bytes += (L_r + q_r) * 2 * p.h_kv * p.head_dim * p.kv_elem_bytes + q_r * 2 * p.h_q * p.head_dim * 2;
            atomicMax(&s_row_rows, (int)min((int64_t)tpi, q_r) * (p.h_q / p.h_kv));
            for (int64_t t0 = 0; t0 < q_r; t0 += tpi) {
                const int64_t nt = min((int64_t)tpi, q_r - t0);
                row_tokens += (p.causal ? L_r - q_r + t0 + nt : L_r) * p.h_kv;
            }
        }
    }
    if (n > 0 && tid == 0 && (int64_t)p.cu_q_lens[n] > p.max_num_tokens) atomicOr(&s_error, 2);
    row_tokens = block_sum64(row_tokens, s_64);
    row_bytes = block_sum64(row_bytes, s_64);
    tile_pairs = block_sum64(tile_pairs, s_64);
    __syncthreads();
    const bool bad = s_error != 0;

    int64_t chunk = p.kv_chunk_override;
    const int num_slots = p.num_slots_narrow > 0 && s_row_rows <= 8 ? p.num_slots_narrow : p.num_slots;
    if (chunk <= 0) chunk = max((int64_t)256, round_up64(row_tokens / max(num_slots, 1) / kChunkDivisor, 64));
    chunk = round_up64(chunk, kKvTile);
    if (chunk > INT_MAX / 2) chunk = INT_MAX / 2 / kKvTile * kKvTile;

    if (p.kv_chunk_override <= 0 && row_tokens > 0 && !bad) {
        // small batches: pick the chunk with the lowest estimated makespan among a few around the
        // default (same rule and integer arithmetic as the host planner)
        __shared__ int s_items[9], s_split[9];
        int64_t cand[9];
        cand[0] = chunk;
#pragma unroll
        for (int i = 0; i < 8; ++i) cand[i + 1] = max((int64_t)256, round_up64(chunk * kRefineFactorsDev[i] / 16, kKvTile));
        if (tid < 9) s_items[tid] = s_split[tid] = 0;
        __syncthreads();
        int items[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0}, split[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
        for (int r = tid; r < n; r += kPlanThreads) {
            const int q_r = p.cu_q_lens[r + 1] - p.cu_q_lens[r], L_r = p.kv_lens[r];
            if (q_r == 0 || to_tile(r, q_r, L_r)) continue;
            for (int t0 = 0; t0 < q_r; t0 += tpi) {
#pragma unroll
                for (int i = 0; i < 9; ++i) {
                    const int emitted = split_unit(p, q_r, L_r - q_r, L_r, t0, tpi, cand[i]).emitted;
                    items[i] += emitted * p.h_kv;
                    if (emitted > 1) split[i] += emitted * p.h_kv;
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 9; ++i) {
            int v = items[i];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if ((tid & 31) == 0 && v) atomicAdd(&s_items[i], v);
            int w = split[i];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) w += __shfl_xor_sync(0xffffffffu, w, d);
            if ((tid & 31) == 0 && w) atomicAdd(&s_split[i], w);
        }
        __syncthreads();
        // nine threads price the nine candidates (64-bit divisions are long subroutines: not for
        // all 1024 threads), one thread picks
        __shared__ long long s_cost[9], s_chunk;
        const int64_t slots = max(num_slots, 1);
        if (tid < 9) {
            const int64_t items_i = max(s_items[tid], 1), split_i = s_split[tid];
            const int64_t fixed = kItemFixedKeys * (items_i - split_i) + kSplitItemFixedKeys * split_i;
            s_cost[tid] = ceil_div64(items_i, slots) * ((fixed + row_tokens) / items_i);
        }
        __syncthreads();
        if (tid == 0) {
            int64_t best = chunk;
            if ((int64_t)s_items[0] < kRefineWaves * slots) {
                int64_t best_cost = s_cost[0];
                for (int i = 1; i < 9; ++i)
                    if (s_cost[i] * 100 < best_cost * 97) {
                        best = cand[i];
                        best_cost = s_cost[i];
                    }
            }
            s_chunk = best;
        }
        __syncthreads();
        chunk = s_chunk;
        __syncthreads();
    }

    // ---- phase 2: per-sequence counts and their exclusive scans (1024 sequences per round) ----
    if (tid < 4) s_carry[tid] = 0;
    __syncthreads();
    int max_key = 0;
    for (int base = 0; base < n && !bad; base += kPlanThreads) {
        const int r = base + tid;
        int n_row = 0, n_tile = 0, n_group = 0, n_part = 0;
        if (r < n) {
            const int q_r = p.cu_q_lens[r + 1] - p.cu_q_lens[r], L_r = p.kv_lens[r], c_r = L_r - q_r;
            if (q_r > 0) {
                if (to_tile(r, q_r, L_r)) {
                    n_tile = packing && s_pack[r] != 0 ? (s_pack[r] > 0 ? p.h_kv : 0)
                                                       : p.h_kv * ((q_r + p.tile_tokens - 1) / p.tile_tokens);
                } else {
                    for (int t0 = 0; t0 < q_r; t0 += tpi) {
                        const UnitSplit u = split_unit(p, q_r, c_r, L_r, t0, tpi, chunk);
                        n_row += u.emitted * p.h_kv;
                        if (u.emitted > 1) {
                            n_group += p.h_kv;
                            n_part += u.emitted * p.h_kv;
                        }
                        max_key = max(max_key, (min(u.part, u.visible_end) + kKvTile - 1) / kKvTile);
                    }
                }
            }
        }
        int total;
        const int c0 = s_carry[0], c1 = s_carry[1], c2 = s_carry[2], c3 = s_carry[3];
        const int e_row = block_exclusive_scan(n_row, s_warp, total);
        const int t_row = total;
        const int e_tile = block_exclusive_scan(n_tile, s_warp, total);
        const int t_tile = total;
        const int e_group = block_exclusive_scan(n_group, s_warp, total);
        const int t_group = total;
        const int e_part = block_exclusive_scan(n_part, s_warp, total);
        const int t_part = total;
        if (r < n) {
            if (r < kSmemSeqs) {
                s_off_tile[r] = c1 + e_tile;
                s_q_len[r] = p.cu_q_lens[r + 1] - p.cu_q_lens[r];
            }
            off_row[r] = c0 + e_row;
            off_tile[r] = c1 + e_tile;
            off_group[r] = c2 + e_group;
            off_part[r] = c3 + e_part;
        }
        __syncthreads();
        if (tid == 0) {
            s_carry[0] = c0 + t_row;
            s_carry[1] = c1 + t_tile;
            s_carry[2] = c2 + t_group;
            s_carry[3] = c3 + t_part;
        }
        __syncthreads();
    }
    const int total_rows = s_carry[0], total_tiles = s_carry[1], total_groups = s_carry[2], total_parts = s_carry[3];
    const bool over = total_rows > p.max_row_items || total_tiles > p.max_tile_items || total_groups > p.max_groups ||
                      total_parts > p.max_partials;
    // the longest row item, in KV tiles, over the whole CTA
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) max_key = max(max_key, __shfl_xor_sync(0xffffffffu, max_key, d));
    __syncthreads();
    if ((tid & 31) == 0) s_warp[tid >> 5] = max_key;
    __syncthreads();
    max_key = 0;
    for (int w = 0; w < kPlanThreads / 32; ++w) max_key = max(max_key, s_warp[w]);
    __syncthreads();

    if (bad || over || max_key >= p.hist_len) {
        if (tid == 0) {
            p.counts[0] = p.counts[1] = p.counts[2] = p.counts[3] = 0;
            p.counts[4] = bad ? 1 : 2;  // 1: invalid lengths, 2: capacity of the handle exceeded
            p.counts[5] = p.counts[kDevCountRowRows] = 0;
            atomicOr(p.status, kStatusBadInput | (bad ? 0x100000u : 0x200000u));
        }
        return;
    }

    // ---- phase 3: histogram of row item lengths; bucket b holds the items of max_key - b tiles ----
    // (in shared memory when it fits: the emit phase takes one atomic ticket per item, and a thread's
    // items come one after the other, so the ticket's latency is what the phase costs)
    __shared__ int s_hist[2 * kSmemBuckets];
    const bool small = max_key < kSmemBuckets;
    int* hist = small ? s_hist : p.hist;                               // counts, then starts
    int* fill = small ? s_hist + kSmemBuckets : p.hist + p.hist_len;   // items placed so far
    for (int k = tid; k <= max_key; k += kPlanThreads) hist[k] = fill[k] = 0;
    __syncthreads();
    for (int r = tid; r < n; r += kPlanThreads) {
        const int q_r = p.cu_q_lens[r + 1] - p.cu_q_lens[r], L_r = p.kv_lens[r], c_r = L_r - q_r;
        if (q_r == 0 || to_tile(r, q_r, L_r)) continue;
        for (int t0 = 0; t0 < q_r; t0 += tpi) {
            const UnitSplit u = split_unit(p, q_r, c_r, L_r, t0, tpi, chunk);
            for (int k = 0; k < u.emitted; ++k) {
                const int b = k * u.part, e = min(u.visible_end, b + u.part);
                atomicAdd(&hist[max_key - (e - b + kKvTile - 1) / kKvTile], p.h_kv);
            }
        }
    }
    __syncthreads();
    if (tid < 4) s_carry[tid] = 0;
    __syncthreads();
    for (int base = 0; base <= max_key; base += kPlanThreads) {
        const int k = base + tid;
        const int v = k <= max_key ? hist[k] : 0;
        int total;
        const int c0 = s_carry[0];
        const int ex = block_exclusive_scan(v, s_warp, total);
        if (k <= max_key) hist[k] = c0 + ex;
        __syncthreads();
        if (tid == 0) s_carry[0] = c0 + total;
        __syncthreads();
    }

    // ---- phase 4: emit ----
    // row items: one thread per (sequence, KV head)
    for (int e = tid; e < n * p.h_kv; e += kPlanThreads) {
        const int r = e / p.h_kv, h = e % p.h_kv;
        const int cu = p.cu_q_lens[r];
        const int q_r = p.cu_q_lens[r + 1] - cu, L_r = p.kv_lens[r], c_r = L_r - q_r;
        if (q_r == 0 || to_tile(r, q_r, L_r)) continue;
        int groups_before = 0, parts_before = 0;  // of this sequence's earlier units, per KV head
        for (int t0 = 0; t0 < q_r; t0 += tpi) {
            const UnitSplit u = split_unit(p, q_r, c_r, L_r, t0, tpi, chunk);
            const bool split = u.emitted > 1;
            const int group_at = off_group[r] + groups_before * p.h_kv + h;
            const int part_at = off_part[r] + parts_before * p.h_kv + h * u.emitted;
            for (int k = 0; k < u.emitted; ++k) {
                const int kv_begin = k * u.part, kv_end = min(u.visible_end, kv_begin + u.part);
                int flags = kv_end == u.visible_end ? kFlagWriteKv : 0;
                if (split) flags |= (group_at + 1) << kFlagGroupShift;
                const int bucket = max_key - (kv_end - kv_begin + kKvTile - 1) / kKvTile;
                uint4* dst = reinterpret_cast<uint4*>(p.rows + hist[bucket] + atomicAdd(&fill[bucket], 1));
                dst[0] = make_uint4((uint32_t)r, (uint32_t)h, (uint32_t)t0, (uint32_t)u.nt);
                dst[1] = make_uint4((uint32_t)kv_begin, (uint32_t)kv_end, (uint32_t)(split ? part_at + k : -1), (uint32_t)flags);
            }
            if (split) {
                uint4* dst = reinterpret_cast<uint4*>(p.groups + group_at);
                dst[0] = make_uint4((uint32_t)(cu + t0), (uint32_t)u.nt, (uint32_t)h, (uint32_t)part_at);
                dst[1] = make_uint4((uint32_t)u.emitted, 0u, 0u, 0u);
                ++groups_before;
                parts_before += u.emitted;
            }
        }
    }

    // tile items: item i belongs to the last sequence whose offset is <= i (sequences without tile
    // items share their successor's offset, hence "last"); inside a sequence one KV head after the
    // other, latest query tile first
    const int* tile_starts = n <= kSmemSeqs ? s_off_tile : off_tile;  // (filled in phase 2)
    for (int i = tid; i < total_tiles; i += kPlanThreads) {
        int lo = 0, hi = n - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (tile_starts[mid] <= i) lo = mid; else hi = mid - 1;
        }
        const int r = lo, q_r = n <= kSmemSeqs ? s_q_len[r] : p.cu_q_lens[r + 1] - p.cu_q_lens[r];
        if (packing && s_pack[r] > 0) {  // one item per KV head for the whole run
            const int m = s_pack[r];
            uint4* dst = reinterpret_cast<uint4*>(p.tiles + i);
            dst[0] = make_uint4((uint32_t)r, (uint32_t)(i - tile_starts[r]), 0u, (uint32_t)(p.cu_q_lens[r + m] - p.cu_q_lens[r]));
            dst[1] = make_uint4((uint32_t)(kFlagWriteKv | kFlagPacked), (uint32_t)m, 0u, 0u);
            continue;
        }
        const int tt = p.tile_tokens, per_head = (q_r + tt - 1) / tt, local = i - tile_starts[r];
        const int q_tok0 = (per_head - 1 - local % per_head) * tt;
        uint4* dst = reinterpret_cast<uint4*>(p.tiles + i);
        dst[0] = make_uint4((uint32_t)r, (uint32_t)(local / per_head), (uint32_t)q_tok0, (uint32_t)min(tt, q_r - q_tok0));
        dst[1] = make_uint4((uint32_t)kFlagWriteKv, 0u, 0u, 0u);
    }

    // ---- phase 5: counts and the SM split of a mixed batch (same estimate as the host planner) ----
    if (tid == 0) {
        int tile_ctas = p.num_sms;  // the tile kernel's persistent CTAs
        if (total_rows > 0 && total_tiles > 0) {
            const double t_tile = 4.0 * p.h_q * p.head_dim * (double)tile_pairs / (p.tile_tflops * 1e12);
            const double t_row = (double)row_bytes / (p.row_gbs * 1e9);
            const int want = (int)(p.num_sms * t_tile / fmax(t_row, 1e-9) + 0.5);
            tile_ctas = min(max(want, p.num_sms / 8), p.num_sms * 5 / 8);
        }
        p.counts[0] = total_rows;
        p.counts[1] = total_tiles;
        p.counts[2] = total_groups;
        p.counts[3] = min(tile_ctas, total_tiles);
        p.counts[4] = 0;
        p.counts[5] = total_parts;
        p.counts[6] = (int)min(chunk, (int64_t)INT_MAX);
        p.counts[kDevCountRowRows] = s_row_rows;
    }
}

cudaError_t launch_plan_kernel(const DevPlanArgs& p, cudaStream_t stream) {
    rpa_plan_kernel<<<1, kPlanThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace rpa
