// Measurement aids: how long the HOST spends inside one gdn_decode / gdn_prefill call (argument
// checks, tensor-map encoding, launches), measured by a plain C++ loop so that no interpreter is
// on the clock.  See include/gdn.h.
#include "../../include/gdn.h"
#include <chrono>
#include <cuda_runtime.h>

extern "C" {

double gdn_host_us_per_decode_call(const void* q, const void* k, const void* v, const float* g,
                                   const float* beta, float* state_pool, const int32_t* slot_idx,
                                   void* o, int32_t B, int32_t Hqk, int32_t Hv, int32_t dk,
                                   int32_t dv, int32_t num_slots, float scale, void* stream,
                                   int32_t reps) {
    if (reps <= 0) return static_cast<double>(GDN_ERR_SIZE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = gdn_decode(q, k, v, g, beta, state_pool, slot_idx, o, B, Hqk, Hv, dk, dv, num_slots,
                        scale, nullptr, stream);       // first call: lazy set-up is not on the clock
    if (rc != GDN_OK) return static_cast<double>(rc);
    if (cudaStreamSynchronize(st) != cudaSuccess) return static_cast<double>(GDN_ERR_CUDA);
    const auto t0 = std::chrono::steady_clock::now();
    for (int i = 0; i < reps && rc == GDN_OK; ++i)
        rc = gdn_decode(q, k, v, g, beta, state_pool, slot_idx, o, B, Hqk, Hv, dk, dv, num_slots,
                        scale, nullptr, stream);
    const auto t1 = std::chrono::steady_clock::now();
    if (cudaStreamSynchronize(st) != cudaSuccess) return static_cast<double>(GDN_ERR_CUDA);
    if (rc != GDN_OK) return static_cast<double>(rc);
    return std::chrono::duration<double, std::micro>(t1 - t0).count() / reps;
}

double gdn_host_us_per_prefill_call(const void* q, const void* k, const void* v, const float* g,
                                    const float* beta, const int32_t* cu_seqlens,
                                    const float* init_state, float* final_state,
                                    const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                                    int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk,
                                    int32_t dv, int32_t chunk, int32_t num_slots, float scale,
                                    void* workspace, size_t workspace_bytes, void* stream,
                                    int32_t reps) {
    if (reps <= 0) return static_cast<double>(GDN_ERR_SIZE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int rc = gdn_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, T, N,
                         max_seqlen_hint, Hqk, Hv, dk, dv, chunk, num_slots, scale, workspace,
                         workspace_bytes, nullptr, stream);
    if (rc != GDN_OK) return static_cast<double>(rc);
    if (cudaStreamSynchronize(st) != cudaSuccess) return static_cast<double>(GDN_ERR_CUDA);
    const auto t0 = std::chrono::steady_clock::now();
    for (int i = 0; i < reps && rc == GDN_OK; ++i)
        rc = gdn_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, slot_idx, o, T, N,
                         max_seqlen_hint, Hqk, Hv, dk, dv, chunk, num_slots, scale, workspace,
                         workspace_bytes, nullptr, stream);
    const auto t1 = std::chrono::steady_clock::now();
    if (cudaStreamSynchronize(st) != cudaSuccess) return static_cast<double>(GDN_ERR_CUDA);
    if (rc != GDN_OK) return static_cast<double>(rc);
    return std::chrono::duration<double, std::micro>(t1 - t0).count() / reps;
}

}  // extern "C"
