// polyspec_verify_level_static: polyspec_verify_level for callers that have no way to hand the
// library a workspace because they cannot allocate device memory themselves -- code that runs
// inside someone else's memory plan (a serving engine that has already carved up the whole
// device, a plugin called from a framework's execution callback, a process that must stay
// within a fixed memory budget after start-up).  The row-statistics partials, which the regular
// call keeps in the caller's workspace, live here in a fixed array inside the library image.
#include <mutex>

#include "polyspec_kernels.cuh"

namespace {

// The scratch itself.  Every GPU that loads the library carries these bytes until the process
// exits, which is why the limit is modest.
static __device__ __align__(256) unsigned char g_static_scratch[POLYSPEC_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// In host code `g_static_scratch` is only a handle for the runtime, not a device address, so the
// address each device gave the array is looked up once per device (with that device current)
// and cached.
polyspec_status scratch_on_current_device(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return POLYSPEC_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return POLYSPEC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || p == nullptr) return POLYSPEC_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return POLYSPEC_OK;
}

}  // namespace

extern "C" {

size_t polyspec_static_scratch_bytes(void) { return POLYSPEC_STATIC_SCRATCH_BYTES; }

polyspec_status polyspec_verify_level_static(
    const void* logits_p, const void* logits_q, const int32_t* draft_tokens, const float* uniforms,
    const int32_t* block_len, int B, int k, int V, polyspec_dtype dt, float temperature,
    int32_t* accepted_len, int32_t* next_token, float* p_at_draft, float* q_at_draft,
    int32_t* device_status, void* cuda_stream)
{
    size_t need = 0;
    const polyspec_status st = polyspec::verify_level_two_launch_workspace(B, k, V, dt, &need);
    if (st != POLYSPEC_OK) return st;
    if (need > POLYSPEC_STATIC_SCRATCH_BYTES) return POLYSPEC_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    const polyspec_status ss = scratch_on_current_device(&scratch);
    if (ss != POLYSPEC_OK) return ss;
    // Every partial the second kernel reads is written by the first kernel of the same call, so
    // nothing in the array has to start at zero and the previous call's contents are harmless.
    return polyspec::verify_level_two_launch(logits_p, logits_q, draft_tokens, uniforms, block_len, B, k, V, dt, temperature,
                                             accepted_len, next_token, p_at_draft, q_at_draft, device_status,
                                             scratch, POLYSPEC_STATIC_SCRATCH_BYTES, cuda_stream);
}

}  // extern "C"
