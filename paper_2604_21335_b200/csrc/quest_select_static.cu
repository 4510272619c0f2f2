// stc_quest_select_static: page selection for callers that cannot hand the
// library a workspace.
//
// Some hosts of this library have no way to obtain device memory at the moment
// they need a selection: code running inside a region where the allocator must
// not be touched (a latency-critical serving loop whose memory pool is frozen,
// a plugin that is only given its input and output buffers by the framework
// that owns the device, a process whose device memory is fully pre-assigned).
// For them the scratch space of the selection (per-problem arrival counters
// and the fp32 page scores) lives in an array that is part of the library
// image itself: it exists on every GPU that loads the library, from load until
// the process exits, and costs kStaticScratchBytes of device memory there.
//
// The array's name is only meaningful to device code.  On the host it is a
// stand-in object, not a device address, so the host asks the runtime for the
// real address (once per device, while that device is current) and passes that
// to the ordinary selection launch.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)STC_STATIC_SCRATCH_BYTES;

static __device__ __align__(256) unsigned char g_select_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the current device; looked up on the first call
// made while that device is current and remembered afterwards.
int32_t scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return STC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p) return STC_ERR_CUDA;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return STC_OK;
}

}  // namespace

extern "C" int32_t stc_quest_select_static(const stc_shape* shape, const stc_cache* cache, const void* q,
                                           int32_t token_budget, int32_t max_pages, int32_t* page_ids,
                                           int32_t* n_pages, float* scores_opt, void* stream) {
    size_t need = 0;
    int32_t rc = stc_workspace_bytes(shape, STC_OP_QUEST_SELECT, 0, &need);
    if (rc != STC_OK) return rc;
    if (need > kStaticScratchBytes) return STC_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    if (need > 0) {
        rc = scratch_for_current_device(&scratch);
        if (rc != STC_OK) return rc;
    }
    // The selection launch clears the arrival counters it uses at the start of
    // every call, so whatever the previous call left in the array is harmless.
    return stc_quest_select(shape, cache, q, token_budget, max_pages, page_ids, n_pages, scores_opt,
                            scratch, need, stream);
}
