// Chunked prefill with the record production in two parts around the persistent state pass.
//
// With few (sequence, v-head) units of unequal length the state pass is a handful of long serial
// chains: most SMs hold a short chain that ends early, or none, while the intra-chunk kernel
// before it needs the whole machine.  Here the intra-chunk work is cut in two along the order in
// which the chains consume the records (by position inside the sequence first): the first part
// runs alone, then the state pass starts, one CTA per unit, and the second part runs beside it on
// the SMs that have no live chain, each record published through a flag (release) that the state
// pass's loading warp waits for (acquire, bounded).
//
// Five launches in one stream, the first four each a programmatic dependent of the one before:
//   prep          chunk table, ranking, processing order, cleared flags and done table, the cut
//   first part    waits for prep; items [0, cut) of the order, 4 CTAs per SM
//   state pass    waits for the first part, THEN lets its dependent start, so the second part's
//                 CTAs are scheduled only once every state-pass CTA is resident: they can never
//                 take the SMs the chains need, and every chain that waits for a record is
//                 resident while the producers still have SMs of their own (the launcher keeps
//                 units <= SMs - kOverlapSpareSms, so every CTA has one unit)
//   second part   does not wait for the state pass (it only feeds it); items [cut, total), pulled
//                 from a queue by seven CTAs per unit (at most four per SM).  Its CTA 0 waits
//                 for the state pass at its very end, so that the completion of this launch
//                 implies the state pass's.
//   rest          an ordinary launch.  CUDA lets a programmatic dependent start early, it does not
//                 promise to; if the second part did not run beside the state pass, the state
//                 pass's waits for records ran out (soon, and without an error: a unit's final
//                 state is written only after its last record has been loaded, so an unfinished
//                 unit has left its initial state alone), it marked the units it finished, and
//                 this launch runs the persistent pass over the others now that every record
//                 exists.  Normally every CTA finds its unit done and returns at once.
#include "gdn_prefill_stream.cuh"
#include <cstdlib>

namespace gdn {

constexpr int kOverlapSpareSms = 8;

// First part: one CTA per item [0, cut) of the processing order (surplus CTAs exit).
__global__ void __launch_bounds__(kIntraThreads, 4)
prefill_intra_first_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p,
                           uint8_t* ws, const WorkspaceLayout lay) {
    pdl_launch_dependents();
    pdl_wait();                     // the tables are the prep kernel's
    const int32_t* hdr = reinterpret_cast<const int32_t*>(ws);
    const int item = blockIdx.x;
    if (item >= hdr[kHdrSplit]) return;
    const int k = item / p.Hv;
    const int hv = item - k * p.Hv;
    const int c = reinterpret_cast<const int32_t*>(ws + lay.order)[k];
    const ChunkInfo ci = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks)[c];
    uint8_t* rec = ws + lay.records + (static_cast<size_t>(c) * p.Hv + hv) * kRecBytes;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ IntraStatics st;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kIntraTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    intra_item(maps, p, rec, ci, hv / (p.Hv / p.Hqk), hv, smem, st, tmem, tid, [] { __syncthreads(); });
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
}

// Second part: resident CTAs pull the items [cut, total) from a queue, in the order the chains
// consume them, and publish each record through its flag.  No wait for the state pass (this kernel
// feeds it): every state-pass CTA has passed its own wait for the first part, hence for prep,
// before this kernel's CTAs are scheduled.
__global__ void __launch_bounds__(kIntraThreads, 4)
prefill_intra_second_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p,
                            uint8_t* ws, const WorkspaceLayout lay) {
    int32_t* hdr = reinterpret_cast<int32_t*>(ws);
    const int32_t cut = hdr[kHdrSplit], total = hdr[kHdrTotalItems];
    const int32_t* order = reinterpret_cast<const int32_t*>(ws + lay.order);
    const ChunkInfo* chunks = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks);
    uint32_t* flags = reinterpret_cast<uint32_t*>(ws + lay.flags);
    const int G = p.Hv / p.Hqk;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ IntraStatics st;
    __shared__ uint32_t tmem_base_s;
    const int tid = threadIdx.x, warp = tid >> 5;
    if (cut < total) {
        if (warp == 0) {
            tmem_alloc(&tmem_base_s, kIntraTmemCols);
            tmem_relinquish();
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        const uint32_t tmem = tmem_base_s;
        uint32_t n_done = 0;
        for (;;) {
            if (tid == 0) st.item = cut + atomicAdd(&hdr[kHdrItemHead], 1);
            __syncthreads();
            const int item = st.item;
            if (item >= total) break;
            const int k = item / p.Hv;
            const int hv = item - k * p.Hv;
            const int c = order[k];
            const ChunkInfo ci = chunks[c];
            const size_t slot = static_cast<size_t>(c) * p.Hv + hv;
            uint8_t* rec = ws + lay.records + slot * kRecBytes;
            const bool ok = intra_item(maps, p, rec, ci, hv / G, hv, smem, st, tmem, tid,
                                       [] { __syncthreads(); }, n_done);
            ++n_done;
            // publish: every thread's own stores first, then the bulk stores, then the flag
            __threadfence();
            tc_fence_before_sync();
            __syncthreads();
            if (tid == 0) {
                bulk_wait_all();
                fence_proxy_async_all();
                __threadfence();
                st_release_u32(&flags[slot], ok ? 1u : 2u);      // 2 = produced after a timeout
            }
            if (!ok) break;
        }
        tc_fence_before_sync();
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
    }
    if (blockIdx.x == 0) pdl_wait();        // the call is complete when this launch is
}

__global__ void __launch_bounds__(kStreamThreads, 1)
prefill_state_stream_gated_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p,
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
    pdl_wait();                     // tables, cleared flags and the first part's records
    pdl_launch_dependents();        // now the second part may take the SMs that are left
    state_stream_role<2>(maps, p, ws, lay, smem, tmem, blockIdx.x, gridDim.x);
    __syncwarp();
    if (warp == kSIssueWarp) tmem_dealloc(tmem, kStateTmemCols);
}

// Last launch: the plain persistent pass over the units the gated pass did not finish (none, when
// the producers ran beside it as intended: then every CTA finds its units done and returns).
__global__ void __launch_bounds__(kStreamThreads, 1)
prefill_state_stream_rest_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p,
                                 uint8_t* ws, const WorkspaceLayout lay) {
    // nothing left for this CTA: leave before any set-up
    {
        const int32_t* done = reinterpret_cast<const int32_t*>(ws + lay.done);
        const int total_units = p.N * p.Hv;
        bool any = false;
        for (int unit = blockIdx.x; unit < total_units; unit += gridDim.x) any = any || done[unit] == 0;
        if (!any) return;
    }
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
    state_stream_role<3>(maps, p, ws, lay, smem, tmem, blockIdx.x, gridDim.x);
    __syncwarp();
    if (warp == kSIssueWarp) tmem_dealloc(tmem, kStateTmemCols);
}

cudaError_t launch_prefill_overlap(const ChunkedParams& cp, cudaStream_t stream, int split_permille) {
    const PrefillParams& p = cp.p;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    const int sms = di.sms;
    e = ensure_dynamic_smem(prefill_state_stream_gated_kernel, kStreamSmem);
    if (e != cudaSuccess) return e;
    e = ensure_dynamic_smem(prefill_state_stream_rest_kernel, kStreamSmem);
    if (e != cudaSuccess) return e;
    e = ensure_dynamic_smem(prefill_intra_first_kernel, kIntraSmem);
    if (e != cudaSuccess) return e;
    e = ensure_dynamic_smem(prefill_intra_second_kernel, kIntraSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_prefill_tensor_maps(&maps, p)) return cudaErrorInvalidValue;

    // The second part needs SMs of its own for as long as a chain may wait for it: with (nearly)
    // as many units as SMs everything is produced before the state pass starts.
    // split_permille == -2 (for tests): the second part is launched as an ordinary successor of
    // the state pass, i.e. the launches are serialised on purpose
    const bool serialised = split_permille == -2;
    const long long units = static_cast<long long>(p.N) * p.Hv;
    if (units > sms - kOverlapSpareSms) split_permille = 1000;
    // The state pass waits for a launch that comes after it in the stream: the two must be able to
    // run at the same time.  Where launches are known to be serialised, produce everything first
    // (then no record is waited for).  A profiler that replays kernels one at a time cannot be
    // seen from here: under it the waits run out (GDN_DEV_TIMEOUT, no hang); profile
    // gdn_prefill_stream instead, which runs the same kernels' arithmetic.
    const char* blocking = std::getenv("CUDA_LAUNCH_BLOCKING");
    if (blocking && blocking[0] != '\0' && blocking[0] != '0') split_permille = 1000;
    if (split_permille > 1000) split_permille = 1000;

    e = launch_prefill_ranked_prep(cp, stream, 2, split_permille, sms);
    if (e != cudaSuccess) return e;
    const dim3 items(static_cast<unsigned>(cp.lay.max_chunks) * static_cast<unsigned>(p.Hv));
    e = launch_dependent(prefill_intra_first_kernel, items, dim3(kIntraThreads), kIntraSmem,
                         stream, maps, p, cp.ws, cp.lay);
    if (e != cudaSuccess) return e;
    const int grid = static_cast<int>(units < sms ? units : sms);
    e = launch_dependent(prefill_state_stream_gated_kernel, dim3(grid), dim3(kStreamThreads),
                         kStreamSmem, stream, maps, p, cp.ws, cp.lay);
    if (e != cudaSuccess) return e;
    // Producers beyond what the chains consume only add memory traffic beside them (one sequence
    // of 32768 tokens at 32 heads: 1024 us with 592 producer CTAs, 986 us with 222, 1203 us with
    // 148): a unit takes a record per chunk step and a producer CTA needs about seven chunk steps
    // per item, so seven CTAs per unit keep up.
    unsigned resident = 7u * static_cast<unsigned>(units);
    if (resident < static_cast<unsigned>(sms)) resident = static_cast<unsigned>(sms);
    if (resident > 4u * static_cast<unsigned>(sms)) resident = 4u * static_cast<unsigned>(sms);
    const dim3 producers(items.x < resident ? items.x : resident);
    if (serialised) {
        prefill_intra_second_kernel<<<producers, kIntraThreads, kIntraSmem, stream>>>(maps, p, cp.ws, cp.lay);
        e = cudaGetLastError();
    } else {
        e = launch_dependent(prefill_intra_second_kernel, producers, dim3(kIntraThreads), kIntraSmem,
                             stream, maps, p, cp.ws, cp.lay);
    }
    if (e != cudaSuccess) return e;
    // an ordinary launch: it starts when the second part has ended, and the second part's first
    // CTA ends only after the state pass
    prefill_state_stream_rest_kernel<<<grid, kStreamThreads, kStreamSmem, stream>>>(maps, p, cp.ws, cp.lay);
    return cudaGetLastError();
}

}  // namespace gdn
