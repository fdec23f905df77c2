// The persistent state pass as a kernel of its own (after the intra-chunk kernel); the role itself
// is in gdn_prefill_stream.cuh.
#include "gdn_prefill_stream.cuh"

namespace gdn {

__global__ void __launch_bounds__(kStreamThreads, 1)
prefill_state_stream_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p,
                            uint8_t* ws, const WorkspaceLayout lay) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ uint32_t tmem_base_s;
    const int warp = threadIdx.x >> 5;
    if (warp == kSIssueWarp) {
        tmem_alloc(&tmem_base_s, kStateTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    state_stream_role<0>(maps, p, ws, lay, smem, tmem, blockIdx.x, gridDim.x);
    __syncwarp();
    if (warp == kSIssueWarp) tmem_dealloc(tmem, kStateTmemCols);
}

// Prep (chunk table + sequences ranked by chunk count) is the fused path's; then the intra-chunk
// kernel over all items; then this kernel on min(units, SMs) CTAs.
cudaError_t launch_prefill_stream(const ChunkedParams& cp, cudaStream_t stream) {
    const PrefillParams& p = cp.p;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    const int sms = di.sms;
    e = ensure_dynamic_smem(prefill_state_stream_kernel, kStreamSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_prefill_tensor_maps(&maps, p)) return cudaErrorInvalidValue;
    const bool inline_tables = prefill_tables_inline(cp);
    if (!inline_tables) {
        e = launch_prefill_ranked_prep(cp, stream, 0);
        if (e != cudaSuccess) return e;
    }
    if (cp.lay.max_chunks > 0) {
        e = launch_prefill_intra(maps, cp, stream, inline_tables);
        if (e != cudaSuccess) return e;
    }
    const long long units = static_cast<long long>(p.N) * p.Hv;
    const int grid = static_cast<int>(units < sms ? units : sms);
    return launch_dependent(prefill_state_stream_kernel, dim3(grid), dim3(kStreamThreads), kStreamSmem,
                            stream, maps, p, cp.ws, cp.lay);
}

}  // namespace gdn
