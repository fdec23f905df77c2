// gdn_prefill_static: chunked prefill for callers that cannot allocate device memory.
//
// Some callers of this library run where cudaMalloc is off limits: inside a
// serving loop whose memory is fully carved up by a pool allocator, inside a
// plugin that is handed tensors but no allocator, or in a process that must not
// disturb another framework's caching allocator.  gdn_prefill needs a scratch
// workspace; this variant brings its own, a fixed array that lives in the
// library's device image.  Every GPU that loads the library carries the array
// (kStaticWorkspaceBytes) until the process exits, which is why it is kept modest.
//
// The array is shared by all calls on a device and keeps whatever the last call
// left in it.  Nothing in it has to start at zero: each call's prep kernel
// rewrites the chunk table it reads, and every record is written by the
// intra-chunk kernel before the state-pass kernel reads it.  Two calls that
// overlap on the GPU (different streams, or different host threads) would write
// the same scratch and race; callers must serialise them.
#include "gdn_prefill_chunk.cuh"
#include "../../include/gdn.h"
#include <mutex>

namespace {

constexpr size_t kStaticWorkspaceBytes = GDN_STATIC_WORKSPACE_BYTES;

// File-scope device array.  In host code this NAME is only a handle for the runtime, not a
// device address: it must go through cudaGetSymbolAddress before a kernel can use it.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_workspace_ptr[kMaxDevices] = {};

// Device address of the array on the current device; resolved once per device.
int static_workspace(unsigned char** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return GDN_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_workspace_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return GDN_ERR_CUDA;
        }
        g_workspace_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_workspace_ptr[dev];
    return GDN_OK;
}

}  // namespace

extern "C" {

size_t gdn_prefill_static_workspace_bytes(void) { return kStaticWorkspaceBytes; }

int gdn_prefill_static(const void* q, const void* k, const void* v, const float* g,
                       const float* beta, const int32_t* cu_seqlens, const float* init_state,
                       float* final_state, const int32_t* slot_idx, void* o,
                       int32_t T, int32_t N, int32_t max_seqlen_hint,
                       int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                       int32_t num_slots, float scale, int32_t* dev_status, void* stream) {
    // Sizes first: a batch whose scratch does not fit the fixed array is refused outright.
    const size_t need = gdn_prefill_workspace_bytes(T, N, Hqk, Hv, dk, dv, chunk);
    if (need > kStaticWorkspaceBytes) return GDN_ERR_LIMIT;
    if (T <= 0 || N <= 0 || need == 0)      // empty batch or a shape gdn_prefill rejects: let it answer
        return gdn_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, T, N,
                           max_seqlen_hint, Hqk, Hv, dk, dv, chunk, num_slots, scale, nullptr, 0,
                           dev_status, stream);
    unsigned char* ws = nullptr;
    const int rc = static_workspace(&ws);
    if (rc != GDN_OK) return rc;
    return gdn_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, T, N,
                       max_seqlen_hint, Hqk, Hv, dk, dv, chunk, num_slots, scale, ws,
                       kStaticWorkspaceBytes, dev_status, stream);
}

}  // extern "C"
