/*
 * rpa.h -- C ABI of the B200 (sm_100a) ragged paged attention library.
 *
 * One call serves a mixed batch of requests with ragged query lengths (decode q_len = 1, chunked
 * prefill, full prefill) against a paged KV cache addressed through a per-request page table, and
 * writes the newly projected K/V of the batch into their cache pages from inside the attention
 * kernels (the paper's Section 3.4 "KV Cache Update Fusion" and Algorithm 1).
 *
 * Notation follows the paper's Table 2: n sequences, s tokens, h_q query heads, h_kv KV heads,
 * h_g = h_q / h_kv, d_k head dimension.  For sequence r: q_r = cu_q_lens[r+1] - cu_q_lens[r] new
 * tokens, L_r = kv_lens[r] keys in total (cached context plus the new tokens, Section 4.1.1), and
 * c_r = L_r - q_r cached keys.  New token i of sequence r sits at absolute position c_r + i.
 *
 * Tensor layouts (row-major, bf16 unless stated, device pointers aligned to 16 bytes):
 *   q, out          [max_num_tokens, h_q,  d_k]   rows [0, T) used, T = cu_q_lens[n]
 *   new_k, new_v    [max_num_tokens, h_kv, d_k]
 *   kv_cache        [num_pages, page_size, 2*h_kv, d_k]  merged, head-interleaved KV of Section
 *                   3.1.3: combined head 2h holds K of KV head h, 2h+1 holds V of KV head h, so a
 *                   single token slot carries K and V of every head
 *   page_table      int32 [n, max_pages_per_seq]; entry p of row r is the physical page of
 *                   positions [p*page_size, (p+1)*page_size); entries past ceil(L_r/page_size) are
 *                   never read
 *   cu_q_lens       int32 [n+1], cu_q_lens[0] = 0
 *   kv_lens         int32 [n]
 *
 * What a call computes (Algorithm 1's result): for every new token i of every sequence r and every
 * query head a, with KV head h = a / h_g (Section 3.1.2),
 *     out[cu_q_lens[r]+i][a] = sum_t softmax_t(sm_scale * <q, K_t>) * V_t,   t = 0 .. hi,
 * hi = c_r + i under the causal mask and L_r - 1 without it; and the K/V rows of every new token
 * are copied bit for bit into the cache slot of their position.  Scores, softmax state and the
 * output accumulator are fp32; probabilities are rounded to bf16 before the PV product; the output
 * is rounded to bf16 once.
 *
 * Quantised cache (the paper's per-tensor quantisation, Section 3.8).  With kv_dtype =
 * RPA_KV_FP8_E4M3 a cache element is one FP8 E4M3 byte that stands for byte_value * k_scale (K) or
 * byte_value * v_scale (V); kv_cache is then [num_pages, page_size, 2*h_kv, d_k] bytes.  q, new_k,
 * new_v and out stay bf16 at the boundary.  With q_scale > 0 the queries are taken in E4M3 precision
 * as well, each element as e4m3(float(q) * (1/q_scale)) * q_scale (the conversion K uses; a pass over
 * the call's T query rows that precedes the attention kernels).  The update stores e4m3(float(x) * (1/scale)) (fp32 multiply by the fp32
 * reciprocal, round to nearest even, saturating at +-448), and attention sees every key and value,
 * the batch's own new tokens included, in that quantised precision.  With head_dim 128 or 256
 * long queries run on the tensor-core tile kernels as with a bf16 cache (their new tokens are
 * quantised and stored by a pass of its own that precedes the tile kernel); head_dim 64 serves
 * every sequence on the row kernel.
 *
 * Ownership: the caller owns every tensor and the stream.  The handle owns the plan (device work
 * lists) and the split-KV workspace, both allocated in rpa_create from the capacities in
 * rpa_config_t; rpa_plan and rpa_forward allocate nothing.  Two optional paths allocate once more,
 * on their first use: rpa_forward_host_submit / rpa_forward_host (two sets of staging buffers for
 * the step's tensors) and rpa_plan_device (its own lists and scratch).  kv_cache is updated in place; out rows
 * >= T and every cache slot other than the T*h_kv updated ones are left bit-identical.
 *
 * Preconditions (undefined behaviour otherwise): page ids lie in [0, num_pages); pages holding
 * positions >= c_r of a sequence are not mapped by any other sequence of the same call (read-only
 * sharing of older pages is fine); the device copies of cu_q_lens / kv_lens given to rpa_forward
 * equal the host copies given to rpa_plan.
 *
 * Errors: every entry point returns a status code and throws nothing across the ABI.  Arguments are
 * validated on the host before anything is launched.  There is no CPU fallback: without a usable
 * CUDA device every call fails with RPA_ERR_CUDA.
 */
#ifndef RPA_H_
#define RPA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rpa_handle rpa_handle_t; /* opaque; owns plan and workspace */

typedef enum {
    RPA_OK = 0,
    RPA_ERR_INVALID_ARG = 1,   /* null/misaligned pointer, negative length, kv_len < q_len, ...      */
    RPA_ERR_UNSUPPORTED = 2,   /* (d_k, h_g, page_size) combination no kernel is built for           */
    RPA_ERR_CAPACITY = 3,      /* n, T or pages per sequence exceed what rpa_create was sized for    */
    RPA_ERR_PLAN_MISMATCH = 4, /* rpa_forward without a plan, or with another num_seqs               */
    RPA_ERR_CUDA = 5,          /* a CUDA runtime/driver call failed; see rpa_last_cuda_error          */
    RPA_ERR_TIMEOUT = 6        /* a bounded device-side wait gave up (reported by rpa_poll_status)   */
} rpa_status_t;

/* Storage type of the KV cache. */
enum { RPA_KV_BF16 = 0, RPA_KV_FP8_E4M3 = 1 };

/* Batch classes of the paper's distribution-aware dispatch (Section 3.5). */
enum { RPA_CASE_EMPTY = 0, RPA_CASE_DECODE = 1, RPA_CASE_PREFILL = 2, RPA_CASE_MIXED = 3 };

typedef struct {
    int32_t num_q_heads;       /* h_q                                                              */
    int32_t num_kv_heads;      /* h_kv; must divide h_q; h_g = h_q/h_kv in {1,2,4,8,16}             */
    int32_t head_dim;          /* d_k: 64, 128 or 256                                               */
    int32_t page_size;         /* tokens per page: a multiple of 16                                 */
    int32_t num_pages;         /* pages in the pool (first extent of kv_cache)                      */
    int32_t max_pages_per_seq; /* row stride of page_table                                          */
    int32_t max_num_seqs;      /* the paper's n: capacity in sequences                              */
    int32_t max_num_tokens;    /* the paper's s: capacity in new tokens per call                    */
    float sm_scale;            /* softmax scale; 0 selects 1/sqrt(d_k)                              */
    int32_t causal;            /* 1: new token i sees keys 0 .. c_r+i; 0: sees all L_r keys          */
    int32_t kv_dtype;          /* RPA_KV_BF16 (0) or RPA_KV_FP8_E4M3 (1)                            */
    float k_scale;             /* FP8 cache: per-tensor scales (Section 3.8); ignored for bf16      */
    float v_scale;
    float q_scale;             /* FP8 cache only: > 0 quantises Q to E4M3 with this per-tensor scale
                                  too (Section 3.8); 0 leaves Q in bf16                              */
} rpa_config_t;

typedef struct {
    int32_t batch_case;         /* RPA_CASE_*                                                        */
    int32_t num_seqs;
    int32_t num_tokens;         /* T                                                                 */
    int32_t num_decode_seqs;    /* q_r == 1                                                          */
    int32_t num_prefill_seqs;   /* q_r  > 1                                                          */
    int32_t num_row_items;      /* work items of the split-KV row kernel                             */
    int32_t num_tile_items;     /* work items of the tensor-core (tcgen05) tile kernel               */
    int32_t num_combine_groups; /* (q block, KV head) groups whose split partials are combined       */
    int32_t kv_chunk_tokens;    /* split-KV chunk length chosen for this batch                       */
    int32_t gpu_launches;       /* kernels one rpa_forward launches for this plan                    */
    int64_t algorithmic_bytes;  /* sum_r (L_r+q_r)*2*h_kv*d_k*B + q_r*2*h_q*d_k*2, B = bytes per cache
                                   element (Section 4.1.1)                                          */
    int64_t algorithmic_flops;  /* 4*h_q*d_k * visible (query,key) pairs            (Section 4.2.1)    */
    int64_t workspace_bytes;    /* split-KV partials this plan uses                                  */
    int64_t row_bytes;          /* algorithmic bytes of the sequences served by the row kernel       */
    int64_t tile_flops;         /* algorithmic FLOPs of the sequences served by the tile kernel      */
    int32_t tile_kernel;        /* which tensor-core kernel runs the tile items: 0 none, 1 two-tile,
                                   2 single-tile (d_k = 256), 3 CTA pair (see rpa_set_tile_pair)       */
    int32_t tile_short_items;   /* 1, 2: the two-tile kernel runs in its instantiation for short items (bf16
                                   cache, every sequence on the tile path has at most 256 key positions,
                                   so every tile item has one or two key blocks; 2: at most 64, so every
                                   item is one key block at most half full); 0 otherwise               */
} rpa_plan_info_t;

/*
 * Create a handle on CUDA device `device` (made current for the call).  Allocates the device work
 * lists, pinned staging for them and the split-KV workspace from the capacities in `cfg`.
 * device < 0 creates a planning-only handle that makes no CUDA call: rpa_plan, rpa_plan_info and
 * rpa_plan_dump work on the host, every call that needs the device fails with RPA_ERR_CUDA.
 * Returns RPA_ERR_UNSUPPORTED for shapes no kernel exists for, RPA_ERR_CUDA if the device or an
 * allocation is unavailable.  `*out` is null on failure.
 */
rpa_status_t rpa_create(const rpa_config_t* cfg, int device, rpa_handle_t** out);

/* Frees everything the handle owns.  Null is accepted.  The caller must have drained the streams. */
void rpa_destroy(rpa_handle_t* h);

/*
 * Host-side planner (the role of the paper's distribution indices and case enum, Section 3.5).
 * cu_q_lens_host [n+1] and kv_lens_host [n] are HOST pointers.  Classifies every sequence (decode
 * q_r == 1, prefill q_r > 1) and the batch, builds the work lists (split-KV chunks for the row
 * kernel, query tiles for the tile kernel, combine groups, one designated cache writer per new
 * token and KV head) and starts their copy to the device (one copy of one packed block: the lists,
 * then the lengths) on a stream the handle owns, into the next of a ring of four list buffers:
 * planning step i+1 never waits for the kernels of step i.  rpa_forward orders itself after the
 * copy.  `stream` is reserved (pass the stream the next rpa_forward will use, or null).  Does not
 * wait for the copy, and does not wait for the device at all unless the caller is four plans ahead
 * of it (the pinned mirror of the buffer it is about to fill then still feeds the copy of the plan
 * made four calls ago; a loop that enqueues steps without ever synchronising is throttled to that
 * depth).  A plan stays valid for any number of rpa_forward calls with the same lengths.
 */
rpa_status_t rpa_plan(rpa_handle_t* h, const int32_t* cu_q_lens_host, const int32_t* kv_lens_host,
                      int32_t num_seqs, void* stream);

/*
 * Attention plus fused cache update for the planned batch, enqueued on `stream` after the plan's
 * lists have reached the device.  All tensor arguments are DEVICE pointers in
 * the layouts above.  Returns after the launches; never synchronises.
 */
rpa_status_t rpa_forward(rpa_handle_t* h, const void* q, const void* new_k, const void* new_v, void* kv_cache,
                         const int32_t* page_table, const int32_t* cu_q_lens, const int32_t* kv_lens,
                         int32_t num_seqs, void* out, void* stream);

/*
 * End-to-end convenience for callers whose step inputs live in HOST memory (pinned memory makes
 * the copies asynchronous): q, new_k, new_v, page_table, cu_q_lens, kv_lens and out are HOST
 * pointers, kv_cache stays a DEVICE pointer (the cache is device-resident state).  Plans the
 * batch, copies the T used rows of the inputs to staging buffers the handle owns, runs
 * rpa_forward, copies the T output rows back and waits for them.  Equal to
 * rpa_forward_host_submit followed by rpa_forward_host_wait until nothing is outstanding.
 */
rpa_status_t rpa_forward_host(rpa_handle_t* h, const void* q_host, const void* new_k_host, const void* new_v_host,
                              void* kv_cache, const int32_t* page_table_host, const int32_t* cu_q_lens_host,
                              const int32_t* kv_lens_host, int32_t num_seqs, void* out_host, void* stream);

/*
 * The two halves of rpa_forward_host, for callers that keep more than one step in flight.
 * rpa_forward_host_submit takes the same arguments, plans on the calling thread, enqueues the
 * input copies (q, new_k, new_v and the page table; the lengths travel with the plan's lists) on a
 * copy stream of the handle, the kernels on `stream` and the output copy on a
 * second copy stream, and returns without waiting: the copies of a step run beside the kernels of
 * its neighbours (two sets of staging buffers; a third outstanding step waits, on the device, for
 * the first one's output copy).  Steps run in submission order on `stream`, so each sees the cache
 * as its predecessor left it.  The host arrays of a step (inputs and out_host) must stay untouched
 * until rpa_forward_host_wait has returned for it; the lengths are consumed before submit returns.
 * rpa_forward_host_wait blocks the calling thread until the oldest outstanding step has delivered
 * out_host (returns RPA_OK at once if none is outstanding).  A step that failed to submit is not
 * outstanding.  Device status (rpa_poll_status) is checked by the caller as after rpa_forward.
 */
rpa_status_t rpa_forward_host_submit(rpa_handle_t* h, const void* q_host, const void* new_k_host,
                                     const void* new_v_host, void* kv_cache, const int32_t* page_table_host,
                                     const int32_t* cu_q_lens_host, const int32_t* kv_lens_host, int32_t num_seqs,
                                     void* out_host, void* stream);
rpa_status_t rpa_forward_host_wait(rpa_handle_t* h);

/*
 * The same computation as rpa_plan + rpa_forward for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for deployment, not for the method.)
 *
 * Who needs it: a server that has given all free HBM to its own KV-cache pool, where any later
 * cudaMalloc fails or eats into that pool, and loops that cannot take the device-wide
 * synchronisation a cudaMalloc or cudaFree implies.  rpa_create allocates, so such callers cannot
 * hold a handle; this call takes none and makes no cudaMalloc, cudaFree or other device
 * allocation.  Its work lists and split-KV partials live in a fixed array inside the library image
 * (about 8.7 MB, held by every GPU that loads the library until the process exits).
 *
 * Arguments: `cfg` describes the shapes as for rpa_create (max_num_seqs and max_num_tokens bound
 * this call's num_seqs and token count); the tensor arguments are DEVICE pointers exactly as for
 * rpa_forward; cu_q_lens_host / kv_lens_host are HOST copies of the lengths, as for rpa_plan.  The
 * call runs on the CURRENT device, which must own the tensors, and is enqueued on `stream`.
 *
 * Limits: at most 4096 row-kernel work items, 512 split groups and 1024 split partials per call
 * (a decode batch of a few hundred requests; prefill-sized batches do not fit), head_dim <= 128.
 * A larger batch is rejected with RPA_ERR_CAPACITY and a message on stderr, before any launch.
 *
 * The first call on each device also resolves the array's device address and sets the kernel's
 * shared-memory attribute; make that first call before starting any stream capture.  All calls on
 * a device share the one array, which keeps the previous call's contents (nothing in it needs
 * clearing: a call reads only what it wrote itself).  Host-side, calls are serialised by a lock;
 * on the GPU, two calls that overlap in time (different streams) race on the array -- keep calls
 * on one device ordered on a single stream.  The work lists of a call are copied from ordinary host
 * memory, so the call returns only after earlier work on `stream` has finished (the kernels it
 * enqueues run asynchronously as usual); a stream that is being captured is refused with
 * RPA_ERR_UNSUPPORTED, as are head_dim 256 and an FP8 cache.
 */
rpa_status_t rpa_forward_static(const rpa_config_t* cfg, const void* q, const void* new_k, const void* new_v,
                                void* kv_cache, const int32_t* page_table, const int32_t* cu_q_lens,
                                const int32_t* kv_lens, const int32_t* cu_q_lens_host, const int32_t* kv_lens_host,
                                int32_t num_seqs, void* out, void* stream);

/* Describes the current plan (work counts follow Sections 4.1.1 and 4.2.1). */
rpa_status_t rpa_plan_info(const rpa_handle_t* h, rpa_plan_info_t* info);

/*
 * Copies the current plan's work lists to host arrays for inspection: row items (8 int32 each:
 * seq, kv_head, q_tok0, n_tok, kv_begin, kv_end, partial, flags), tile items (8 int32 each: seq,
 * kv_head, q_tok0, n_tok, flags, n_seqs of a packed item, reserved...) and combine groups (8 int32 each: out_tok0, n_tok, kv_head,
 * first_partial, n_partials, reserved...).  Each pointer may be null; capacities are in items.
 * Pure host work.
 */
rpa_status_t rpa_plan_dump(const rpa_handle_t* h, int32_t* row_items, int32_t row_capacity, int32_t* tile_items,
                           int32_t tile_capacity, int32_t* combine_groups, int32_t group_capacity);

/*
 * Device-side planner: the same plan as rpa_plan, built by a kernel on `stream` from the DEVICE
 * copies of the lengths (cu_q_lens [n+1], kv_lens [n], the pointers rpa_forward gets), with no host
 * round trip: the remedy for the metadata work the paper leaves on the critical path (Section 5,
 * Discussion and Future Directions).  The following rpa_forward with the same num_seqs launches fixed grids that read
 * their item counts from device memory, so the pair may be captured in a CUDA graph and replayed
 * after the caller has changed the lengths, page table and inputs in place.  Differences from
 * rpa_plan: runs of short sequences are packed into shared tile items only in batches of up to 1024
 * sequences; row items of equal length come in no particular order; q, new_k, new_v and out must hold max_num_tokens rows (the
 * tensor maps cover that extent).  Invalid
 * lengths or a batch beyond the handle's capacities are found on the device: the step's kernels
 * then do nothing and rpa_poll_status reports RPA_ERR_INVALID_ARG (bit 29 of the word; bit 20:
 * bad lengths, bit 21: capacity).  That word is STICKY: until rpa_poll_status has reported and cleared
 * it, every later device-planned step (and every later validated host-planned step) also returns at
 * once without writing `out` or the cache - a loop that replays a graph and polls only now and then
 * drops steps in the meantime.  The first call allocates the device lists and scratch - make it
 * before capturing.  rpa_plan_info and rpa_plan_dump do not describe a device-made plan, and
 * rpa_set_validation has no effect on a device-planned step.
 * Streams: the handle keeps two sets of device lists.  Outside a capture, each rpa_plan_device
 * writes the set the previous plan did not use, after the last rpa_forward that read that set (an
 * event the handle records), and the next rpa_forward waits for the plan's kernel whatever stream
 * it ran on.  So the plan of step i+1 may be enqueued on a second stream as soon as step i's
 * rpa_forward has been, and runs beside step i's kernels.  At most one plan may be ahead of the
 * forwards: issue calls in the order plan, forward, plan, forward, ... from one host thread.
 * Inside a stream capture the set does not change and no events are used: capture plan and forward on
 * one stream (or order them yourself).  The counts word 7 is the largest number of query rows of
 * any row item.
 */
rpa_status_t rpa_plan_device(rpa_handle_t* h, const int32_t* cu_q_lens, const int32_t* kv_lens, int32_t num_seqs,
                             void* stream);

/*
 * Inspection of a device-made plan: waits for the device, then copies the planner's counts
 * (8 int32: row items, tile items, combine groups, CTAs given to the tile kernel, error code,
 * split partials, split-KV chunk, most query rows of a row item) and, where the pointers are not null, the lists in the
 * layout of rpa_plan_dump.  Host pointers; capacities in items.
 */
rpa_status_t rpa_plan_device_dump(rpa_handle_t* h, int32_t* counts, int32_t* row_items, int32_t row_capacity,
                                  int32_t* tile_items, int32_t tile_capacity, int32_t* combine_groups,
                                  int32_t group_capacity);

/*
 * Reads the device status word the kernels write instead of trapping (a bounded wait that gave
 * up).  Synchronises `stream`.  Returns RPA_OK, RPA_ERR_TIMEOUT or RPA_ERR_INVALID_ARG; `*detail`,
 * if not null, receives the raw word (bit 28 set: a wait expired; low byte: which one).  A nonzero
 * word is cleared by the call that reports it.
 */
rpa_status_t rpa_poll_status(rpa_handle_t* h, void* stream, uint32_t* detail);

/*
 * Input validation on the device (off by default).  While enabled, rpa_forward first launches a small
 * kernel that checks, for every sequence, that the device copy of kv_lens equals the planned one and
 * that every page id the sequence maps lies in [0, num_pages).  On a violation bit 29 of the status
 * word is set (low 20 bits: a sequence at fault), the attention kernels of that call return at once
 * without touching kv_cache or out, and rpa_poll_status reports RPA_ERR_INVALID_ARG.  The word stays
 * set until it is polled, and while it is set every later validated call returns at once in the same
 * way.  Costs one extra launch per call.
 *
 * Bounds-checked build: `librpa_b200_debug.so` (python -m paper_2604_15464_b200.build --debug) is the
 * same library compiled with -DRPA_DEBUG.  Its kernels check every page id, token row and ring stage
 * before the access; the first violation of a call sets bit 27 of the status word (bits 24..26: 1 page
 * id, 2 token row, 3 stage index; low 24 bits: the offending value) and the access is skipped.
 */
rpa_status_t rpa_set_validation(rpa_handle_t* h, int32_t enable);

/*
 * Every device-side wait of the library is bounded: when it expires the kernel records a code in
 * the status word and returns normally (it never traps or spins forever).  This call launches one
 * warp whose wait cannot succeed (about a millisecond), so that a caller can check the whole
 * reporting path on demand: afterwards rpa_poll_status returns RPA_ERR_TIMEOUT once (detail
 * 0x1000007F) and the handle stays usable.
 */
rpa_status_t rpa_selftest_bounded_wait(rpa_handle_t* h, void* stream);

/* Bench-only switches mirroring the paper's ablation study (Section 4, "Ablation Study Setting"):
 * bit 0 skips the fused cache update ("w/o KV update"); bit 1 runs the two kernels of a mixed batch
 * one after the other instead of side by side; bit 2 skips the attention arithmetic and keeps the
 * K/V movement ("w/o FA"); bit 3 skips the K/V (and Q tile) loads and keeps the arithmetic, on
 * whatever shared memory holds ("w/o DMA").  With bit 2 or 3 set `out` is undefined (bit 2: not
 * written by the tile kernel); the row kernel and the two-tile kernel honour them, the head_dim 256
 * tile kernel only bits 0 and 1.  0 restores the full path. */
rpa_status_t rpa_set_ablation(rpa_handle_t* h, uint32_t mask);

/*
 * Per-kernel timing for benchmarks.  While enabled, rpa_forward records a CUDA event pair on the
 * launch stream around each of its kernels (at most 8192 launches per kernel are kept; enabling
 * again clears them).  rpa_get_kernel_timing waits for the recorded events and returns, for kernel
 * kinds 0 = row kernel, 1 = tile kernel, 2 = combine kernel, the summed device time in
 * milliseconds and the number of launches; both arrays have 3 entries.
 */
rpa_status_t rpa_set_kernel_timing(rpa_handle_t* h, int32_t enable);
rpa_status_t rpa_get_kernel_timing(rpa_handle_t* h, float* total_ms, int32_t* launches);

/* Overrides the planner's split-KV chunk length (tokens, rounded up to a multiple of 16); 0 restores
 * the automatic choice.  Invalidates the current plan.  Meant for tests and tuning. */
rpa_status_t rpa_set_kv_chunk(rpa_handle_t* h, int32_t tokens);

/* Sequences with at least this many new tokens go to the tensor-core tile kernel, shorter ones to
 * the row kernel, and nothing else decides: an explicit threshold switches off the packing of short
 * sequences and the extra rule for small queries on long contexts.  0 restores the default rules
 * (tile kernel from more than two row items' worth of query rows, q*h_g > 32; from more than one
 * with at least 1024 keys on pages of 32 slots or more; runs of short sequences without context
 * packed into shared tile items); a value above max_num_tokens keeps everything on the row kernel.
 * Invalidates the current plan.  Meant for tests and tuning. */
rpa_status_t rpa_set_tile_min_q(rpa_handle_t* h, int32_t tokens);

/* Which tensor-core kernel runs the tile items of host-made plans.  The CTA-pair kernel runs
 * Algorithm 1's products for four query tiles at a time on two neighbouring SMs that share every key
 * block (each stages half of it), with items of twice the tokens that follow one another without a
 * pause; it pays off where items are full.  mode 2 (the default): the pair kernel for pure long-prefill
 * batches (every sequence goes to the tile path and brings at least two full pair items of new
 * tokens, and there are at least two pair items per SM), the two-tile kernel otherwise (mixed batches, small-q steps over long contexts, short
 * prompts).  mode 1: the pair kernel for every host-made plan with tile items (RPA_ERR_UNSUPPORTED
 * unless the cache is bf16 and d_k = 128).  mode 0: the two-tile kernel only.  Plans made on the device
 * and plans of handles without a device keep the two-tile kernel's items.  Invalidates the current
 * plan.  Results are the same function of the inputs either way (same tolerance against the
 * definition, cache bytes identical). */
rpa_status_t rpa_set_tile_pair(rpa_handle_t* h, int32_t mode);

const char* rpa_status_string(rpa_status_t s);

/* Text of the last CUDA error seen by this handle ("" if none). */
const char* rpa_last_cuda_error(const rpa_handle_t* h);

#ifdef __cplusplus
}
#endif
#endif /* RPA_H_ */
