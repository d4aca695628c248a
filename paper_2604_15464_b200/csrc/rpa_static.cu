// rpa_forward_static: the split-KV row path for callers that cannot allocate device memory.
//
// Some callers may not call cudaMalloc at all: an inference server that has already handed every
// free byte of HBM to its own KV-cache pool, so that a later cudaMalloc fails or fragments that
// pool; or a latency-critical loop that cannot afford the device-wide synchronisation a
// cudaMalloc/cudaFree implies.  rpa_create allocates (work lists, split-KV workspace), so those
// callers cannot use a handle.  This entry point needs no handle and allocates nothing on the
// device: its work lists and its split-KV partials live in one file-scope __device__ array of fixed
// size that is part of the library image.
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>

#include <mutex>

#include "../../include/rpa.h"
#include "rpa_kernels.h"
#include "rpa_planner.h"

using namespace rpa;

namespace {

// Capacity of the built-in scratch.  Every GPU that loads the library holds these bytes until the
// process exits, so the limits are modest: enough for a decode batch of a few hundred requests.
constexpr int kStaticMaxRowItems = 4096;
constexpr int kStaticMaxGroups = 512;
constexpr int kStaticMaxPartials = 1024;
constexpr int kStaticMaxHeadDim = 128;

constexpr size_t kOffRows = 0;
constexpr size_t kOffGroups = kOffRows + (size_t)kStaticMaxRowItems * sizeof(RowItem);
constexpr size_t kOffPartialO = kOffGroups + (size_t)kStaticMaxGroups * sizeof(CombineGroup);
constexpr size_t kOffPartialMl = kOffPartialO + (size_t)kStaticMaxPartials * kRowTileRows * kStaticMaxHeadDim * sizeof(float);
constexpr size_t kScratchBytes = kOffPartialMl + (size_t)kStaticMaxPartials * kRowTileRows * 2 * sizeof(float);
static_assert(kOffGroups % 256 == 0 && kOffPartialO % 256 == 0 && kOffPartialMl % 256 == 0, "sections stay aligned");

// The scratch itself (about 8.7 MB).  In host code this name is only a handle for the runtime's
// symbol calls, not a device address: a kernel must be given the pointer cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;                         // serialises host-side planning and set-up
unsigned char* g_scratch_ptr[kMaxDevices];  // device address of the scratch, per device ordinal
int g_num_sms[kMaxDevices];
Plan g_plan;                                // host-side plan storage, reused by every call

// Once per device, with that device current: resolve the scratch's device address and opt the row
// kernel in to its shared memory.  No allocation.
cudaError_t setup_device(int dev, int head_dim, int group) {
    if (!g_scratch_ptr[dev]) {
        unsigned char* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        e = cudaDeviceGetAttribute(&g_num_sms[dev], cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = p;
    }
    return row_kernel_prepare(head_dim, group);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" rpa_status_t rpa_forward_static(const rpa_config_t* cfg, const void* q, const void* new_k, const void* new_v,
                                           void* kv_cache, const int32_t* page_table, const int32_t* cu_q_lens,
                                           const int32_t* kv_lens, const int32_t* cu_q_lens_host,
                                           const int32_t* kv_lens_host, int32_t num_seqs, void* out, void* stream) {
    if (!cfg || !cu_q_lens_host || !kv_lens_host) return RPA_ERR_INVALID_ARG;
    if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads) return RPA_ERR_INVALID_ARG;
    if (cfg->page_size <= 0 || cfg->max_pages_per_seq <= 0 || !(cfg->sm_scale >= 0.f)) return RPA_ERR_INVALID_ARG;
    const int group = cfg->num_q_heads / cfg->num_kv_heads;
    if (!row_kernel_supported(cfg->head_dim, group) || cfg->page_size % kKvTile || cfg->head_dim > kStaticMaxHeadDim ||
        cfg->kv_dtype != RPA_KV_BF16)
        return RPA_ERR_UNSUPPORTED;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The work lists travel from ordinary (pageable) host memory.  On a stream that executes, the
    // runtime has read the bytes by the time the copy call returns, so g_plan may be reused at once;
    // the price is that the call waits for earlier work on `stream`.  A stream that is being captured
    // would instead record g_plan's address in the graph and read it at every replay, long after the
    // plan has changed: such a stream is refused.
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &capture) != cudaSuccess) return RPA_ERR_CUDA;
    if (capture != cudaStreamCaptureStatusNone) return RPA_ERR_UNSUPPORTED;

    std::lock_guard<std::mutex> lock(g_mutex);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RPA_ERR_CUDA;
    e = setup_device(dev, cfg->head_dim, group);
    if (e != cudaSuccess) {
        fprintf(stderr, "rpa_forward_static: device set-up failed: %s\n", cudaGetErrorString(e));
        return RPA_ERR_CUDA;
    }

    rpa_config_t c = *cfg;
    if (c.sm_scale == 0.f) c.sm_scale = 1.f / sqrtf((float)c.head_dim);
    PlanPolicy policy;
    policy.num_slots = g_num_sms[dev] * row_kernel_ctas_per_sm(c.head_dim, group);
    policy.max_row_items = kStaticMaxRowItems;
    policy.max_groups = kStaticMaxGroups;
    policy.max_partials = kStaticMaxPartials;
    rpa_status_t st = build_plan(c, policy, cu_q_lens_host, kv_lens_host, num_seqs, g_plan);
    if (st == RPA_ERR_CAPACITY)
        fprintf(stderr,
                "rpa_forward_static: batch exceeds the built-in scratch (at most %d work items, %d split groups, "
                "%d split partials, max_num_seqs/max_num_tokens/max_pages_per_seq of the config)\n",
                kStaticMaxRowItems, kStaticMaxGroups, kStaticMaxPartials);
    if (st != RPA_OK) return st;
    if (g_plan.info.num_tokens == 0) return RPA_OK;
    if (!q || !new_k || !new_v || !kv_cache || !page_table || !cu_q_lens || !kv_lens || !out) return RPA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(new_k) || !aligned16(new_v) || !aligned16(kv_cache) || !aligned16(out))
        return RPA_ERR_INVALID_ARG;

    unsigned char* scratch = g_scratch_ptr[dev];
    e = cudaMemcpyAsync(scratch + kOffRows, g_plan.rows.data(), g_plan.rows.size() * sizeof(RowItem),
                        cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess && !g_plan.groups.empty())
        e = cudaMemcpyAsync(scratch + kOffGroups, g_plan.groups.data(), g_plan.groups.size() * sizeof(CombineGroup),
                            cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return RPA_ERR_CUDA;

    KernelArgs a{};
    a.q = static_cast<const uint16_t*>(q);
    a.new_k = static_cast<const uint16_t*>(new_k);
    a.new_v = static_cast<const uint16_t*>(new_v);
    a.kv_cache = static_cast<uint16_t*>(kv_cache);
    a.page_table = page_table;
    a.cu_q_lens = cu_q_lens;
    a.kv_lens = kv_lens;
    a.out = static_cast<uint16_t*>(out);
    a.row_items = reinterpret_cast<const RowItem*>(scratch + kOffRows);
    a.groups = reinterpret_cast<const CombineGroup*>(scratch + kOffGroups);
    // Nothing here has to start at zero: every partial row a call combines was written earlier in
    // that same call, so the previous call's leftovers are never read.
    a.partial_o = reinterpret_cast<float*>(scratch + kOffPartialO);
    a.partial_ml = reinterpret_cast<float*>(scratch + kOffPartialMl);
    a.num_row_items = (int32_t)g_plan.rows.size();
    a.num_groups = (int32_t)g_plan.groups.size();
    a.h_q = c.num_q_heads;
    a.h_kv = c.num_kv_heads;
    a.head_dim = c.head_dim;
    a.page_size = c.page_size;
    a.max_pages_per_seq = c.max_pages_per_seq;
    a.num_pages = c.num_pages;
    a.causal = c.causal ? 1 : 0;
    a.scale_log2 = c.sm_scale * 1.4426950408889634f;
    a.out_scale = 1.f;
    a.token_cap = c.max_num_tokens;
    e = launch_row_kernel(a, s);
    if (e == cudaSuccess) e = launch_combine_kernel(a, s);
    return e == cudaSuccess ? RPA_OK : RPA_ERR_CUDA;
}
