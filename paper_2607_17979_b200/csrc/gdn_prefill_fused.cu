// Chunked prefill in ONE cooperative launch: the record producers and the state pass overlap.
//
// The grid has one CTA of 512 threads per SM.  The first `n_state` CTAs run the serial state pass
// (the role of the persistent state pass, gdn_prefill_stream.cuh: 8 chain warps, 4 output warps, an
// issuing warp and a loading warp), CTA b over the units b, b + n_state, ... of the list that has
// the longest sequences first.  The other CTAs run two independent groups of 256 threads that pull
// (chunk, v-head) items from a queue and write their records (the intra-chunk routine of
// gdn_prefill_device.cuh), in the order the state pass consumes them: by position inside the
// sequence first, by sequence rank second.  A record is published through a flag in global
// memory (release) and the state pass waits for the flag (acquire, bounded) before it copies the
// record in.  Producers never wait for consumers, every CTA is resident (cooperative launch with
// grid <= SM count), so the consumers' waits always end.
#include "gdn_prefill_stream.cuh"

namespace gdn {

// =============================================================================================
// Prep: chunk table, processing order, cleared queues and flags.  One CTA.
// =============================================================================================
constexpr int kFPrepThreads = 256;
// model of the two-part production (see the kernel): items per SM and chunk step, start-up lag of
// the second part in chunk steps, and a safety margin in items
constexpr int kSplitProdPermille = 600;
constexpr int kSplitLeadSteps = 6;
constexpr int kSplitMarginItems = 128;

__global__ void __launch_bounds__(kFPrepThreads)
prefill_fused_prep_kernel(const int32_t* __restrict__ cu, int32_t T, int32_t N, int32_t Hv,
                          uint8_t* ws, WorkspaceLayout lay, int32_t* dev_status,
                          const int for_fused,     // 0: only the chunk table and the ranking;
                                                   // 1: + processing order, cleared queues and flags;
                                                   // 2: + where the two-part production is cut
                          const int split_permille, const int sms) {
    int32_t* hdr = reinterpret_cast<int32_t*>(ws);
    int32_t* seq_first = reinterpret_cast<int32_t*>(ws + lay.seq_first);
    int32_t* seq_bad = reinterpret_cast<int32_t*>(ws + lay.seq_bad);
    ChunkInfo* chunks = reinterpret_cast<ChunkInfo*>(ws + lay.chunks);
    int32_t* seq_by_rank = reinterpret_cast<int32_t*>(ws + lay.seq_by_rank);
    int32_t* order = reinterpret_cast<int32_t*>(ws + lay.order);
    int32_t* hist = reinterpret_cast<int32_t*>(ws + lay.hist);
    int32_t* fill = reinterpret_cast<int32_t*>(ws + lay.fill);
    int32_t* cnt = reinterpret_cast<int32_t*>(ws + lay.cnt);     // #sequences with more than v chunks
    int32_t* pos = reinterpret_cast<int32_t*>(ws + lay.pos);     // #chunks at positions < j
    uint32_t* flags = reinterpret_cast<uint32_t*>(ws + lay.flags);
    __shared__ int32_t warp_sums[kFPrepThreads / 32];
    __shared__ int32_t running;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();        // the next kernel's CTAs may become resident (they wait for us)

    for (int i = tid; i < lay.max_nc + 2; i += kFPrepThreads) { hist[i] = 0; fill[i] = 0; }
    if (for_fused)
        for (size_t i = tid; i < static_cast<size_t>(lay.max_chunks) * Hv; i += kFPrepThreads)
            flags[i] = 0u;
    if (for_fused == 2) {
        int32_t* done = reinterpret_cast<int32_t*>(ws + lay.done);
        for (int i = tid; i < N * Hv; i += kFPrepThreads) done[i] = 0;
    }
    if (tid == 0) {
        running = 0;
        hdr[kHdrItemHead] = 0;
        hdr[kHdrUnitHead] = 0;
        if (cu[0] != 0 || cu[N] != T) report(dev_status, kDevBadCuSeqlens);
    }
    __syncthreads();
    // chunk counts, prefix sums, chunk table (as in the three-launch path) + histogram of counts
    for (int base = 0; base < N; base += kFPrepThreads) {
        const int n = base + tid;
        int32_t nc = 0;
        if (n < N) {
            const int32_t t0 = cu[n], t1 = cu[n + 1];
            const bool ok = t0 >= 0 && t1 >= t0 && t1 <= T;
            if (!ok) report(dev_status, kDevBadCuSeqlens);
            seq_bad[n] = ok ? 0 : 1;
            nc = ok ? (t1 - t0 + kChunk - 1) / kChunk : 0;
            atomicAdd(&hist[nc], 1);
        }
        int32_t incl = nc;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        int32_t warp_off = 0;
        for (int w = 0; w < warp; ++w) warp_off += warp_sums[w];
        const int32_t first = running + warp_off + incl - nc;
        if (n < N) {
            seq_first[n] = first;
            const int32_t t0 = cu[n];
            const int32_t len = cu[n + 1] - t0;
            for (int j = 0; j < nc; ++j) {
                ChunkInfo ci;
                ci.seq = n;
                ci.t0 = t0 + j * kChunk;
                ci.len = min(kChunk, len - j * kChunk);
                ci.pad = 0;
                chunks[first + j] = ci;
            }
        }
        __syncthreads();
        if (tid == kFPrepThreads - 1) running = first + nc;
        __syncthreads();
    }
    if (tid == 0) {
        seq_first[N] = running;
        hdr[kHdrTotalChunks] = running;
        hdr[kHdrTotalItems] = running * Hv;
        running = 0;
    }
    __syncthreads();
    // cnt[v] = number of sequences with more than v chunks: exclusive suffix sum of the histogram,
    // as a block scan over tiles of the reversed index u = max_nc - v
    for (int base = 0; base <= lay.max_nc; base += kFPrepThreads) {
        const int u = base + tid;
        const int32_t x = u <= lay.max_nc ? hist[lay.max_nc - u] : 0;
        int32_t incl = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        int32_t warp_off = 0;
        for (int w = 0; w < warp; ++w) warp_off += warp_sums[w];
        const int32_t excl = running + warp_off + incl - x;
        if (u <= lay.max_nc) cnt[lay.max_nc - u] = excl;
        __syncthreads();
        if (tid == kFPrepThreads - 1) running = excl + x;
        __syncthreads();
    }
    if (tid == 0) running = 0;
    __syncthreads();
    // pos[j] = number of chunks at positions < j: exclusive prefix sum of cnt (fused launch only)
    for (int base = 0; for_fused != 0 && base <= lay.max_nc; base += kFPrepThreads) {
        const int j = base + tid;
        const int32_t x = j <= lay.max_nc ? cnt[j] : 0;
        int32_t incl = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int32_t y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        if (lane == 31) warp_sums[warp] = incl;
        __syncthreads();
        int32_t warp_off = 0;
        for (int w = 0; w < warp; ++w) warp_off += warp_sums[w];
        const int32_t excl = running + warp_off + incl - x;
        if (j <= lay.max_nc) pos[j] = excl;
        __syncthreads();
        if (tid == kFPrepThreads - 1) running = excl + x;
        __syncthreads();
    }
    // Two-part production (mode 2).  The items of the processing order before the cut are
    // produced before the state pass starts, the others beside it, on the SMs it leaves free.
    // The cut is the smallest head start with which the chains never catch up with the
    // producers, by a simple model: every live (sequence, v-head) unit consumes one item per
    // chunk step, the SMs without a live unit produce kProdPermille / 1000 items per chunk step
    // each, and an item started when the state pass starts is ready kLeadSteps chunk steps
    // later.  In step j the chains need the Hv * pos[j + 1] first items of the order; by then the
    // second part has produced r * sum_{i < j - lead} (sms - Hv * cnt[i]), and that sum is
    // m * sms - Hv * pos[m] with m = j - lead.
    if (for_fused == 2) {
        __shared__ int32_t need_max;
        if (tid == 0) need_max = 0;
        __syncthreads();
        const long long total_items = hdr[kHdrTotalItems];
        long long local = 0;
        const int lead = kSplitLeadSteps, prod = kSplitProdPermille;
        for (int j = tid; j < lay.max_nc; j += kFPrepThreads) {
            const int m = j > lead ? j - lead : 0;
            long long produced =
                (static_cast<long long>(m) * sms - static_cast<long long>(Hv) * pos[m]) * prod / 1000;
            if (produced < 0) produced = 0;
            const long long need = static_cast<long long>(Hv) * pos[j + 1] - produced;
            local = need > local ? need : local;
        }
        if (local > total_items) local = total_items;
        atomicMax(&need_max, static_cast<int32_t>(local));
        __syncthreads();
        if (tid == 0) {
            long long cut = split_permille >= 0 ? total_items * split_permille / 1000
                                                : static_cast<long long>(need_max) + kSplitMarginItems;
            if (cut > total_items) cut = total_items;
            hdr[kHdrSplit] = static_cast<int32_t>(cut);
        }
    }
    // rank of a sequence = its place in the order "more chunks first"; chunk j of the sequence of
    // rank r is processed at place pos[j] + r (the sequences that have a chunk j are ranks < cnt[j])
    int32_t* rank_of = reinterpret_cast<int32_t*>(ws + lay.rank_of);
    for (int n = tid; n < N; n += kFPrepThreads) {
        const int32_t nc = seq_first[n + 1] - seq_first[n];
        const int32_t rank = cnt[nc] + atomicAdd(&fill[nc], 1);
        seq_by_rank[rank] = n;
        rank_of[n] = rank;
    }
    if (for_fused) {
        // one thread per chunk (a loop per sequence would be a chain of dependent loads as long
        // as the longest sequence)
        __syncthreads();
        const int32_t total_chunks = hdr[kHdrTotalChunks];
        for (int c = tid; c < total_chunks; c += kFPrepThreads) {
            const int32_t n = chunks[c].seq;
            order[pos[c - seq_first[n]] + rank_of[n]] = c;
        }
    }
}

// The same tables for a batch of at most kFPrepThreads sequences when only the chunk table and the
// ranking are wanted (mode 0): one thread per sequence, one block scan, the ranking by counting in
// shared memory; no histogram, no cleared arrays.  About half the time of the general kernel, which
// every three-launch call of such a batch waits for.
__global__ void __launch_bounds__(kFPrepThreads)
prefill_small_prep_kernel(const int32_t* __restrict__ cu, int32_t T, int32_t N, uint8_t* ws,
                          WorkspaceLayout lay, int32_t* dev_status) {
    int32_t* hdr = reinterpret_cast<int32_t*>(ws);
    int32_t* seq_first = reinterpret_cast<int32_t*>(ws + lay.seq_first);
    int32_t* seq_bad = reinterpret_cast<int32_t*>(ws + lay.seq_bad);
    ChunkInfo* chunks = reinterpret_cast<ChunkInfo*>(ws + lay.chunks);
    int32_t* seq_by_rank = reinterpret_cast<int32_t*>(ws + lay.seq_by_rank);
    int32_t* rank_of = reinterpret_cast<int32_t*>(ws + lay.rank_of);
    __shared__ int32_t warp_sums[kFPrepThreads / 32];
    __shared__ int32_t s_nc[kFPrepThreads];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();        // the next kernel's CTAs may become resident (they wait for us)
    const int n = tid;
    int32_t nc = 0, t0 = 0, len = 0;
    if (n < N) {
        t0 = cu[n];
        const int32_t t1 = cu[n + 1];
        const bool ok = t0 >= 0 && t1 >= t0 && t1 <= T;
        if (!ok) report(dev_status, kDevBadCuSeqlens);
        seq_bad[n] = ok ? 0 : 1;
        len = t1 - t0;
        nc = ok ? (len + kChunk - 1) / kChunk : 0;
    }
    if (tid == 0 && (cu[0] != 0 || cu[N] != T)) report(dev_status, kDevBadCuSeqlens);
    s_nc[tid] = n < N ? nc : -1;
    int32_t incl = nc;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int32_t y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    int32_t warp_off = 0, total = 0;
    for (int w = 0; w < kFPrepThreads / 32; ++w) {
        if (w < warp) warp_off += warp_sums[w];
        total += warp_sums[w];
    }
    const int32_t first = warp_off + incl - nc;
    if (n < N) {
        seq_first[n] = first;
        for (int j = 0; j < nc; ++j) {
            ChunkInfo ci;
            ci.seq = n;
            ci.t0 = t0 + j * kChunk;
            ci.len = min(kChunk, len - j * kChunk);
            ci.pad = 0;
            chunks[first + j] = ci;
        }
        // rank = place in the order "more chunks first" (ties by index)
        int32_t rank = 0;
        for (int m = 0; m < N; ++m) {
            const int32_t nm = s_nc[m];
            rank += (nm > nc || (nm == nc && m < n)) ? 1 : 0;
        }
        seq_by_rank[rank] = n;
        rank_of[n] = rank;
    }
    if (tid == 0) {
        seq_first[N] = total;
        hdr[kHdrTotalChunks] = total;
        hdr[kHdrTotalItems] = 0;       // (the queues of the other modes are not used)
        hdr[kHdrItemHead] = 0;
        hdr[kHdrUnitHead] = 0;
    }
}

// =============================================================================================
// The fused kernel
// =============================================================================================
constexpr int kFusedThreads = 512;
constexpr int kFGroups = 2;                          // intra role: two groups of 256 threads
constexpr uint32_t kFGroupSmem = (kI_End + 1023u) & ~1023u;
constexpr uint32_t kFusedSmem =
    (kFGroups * kFGroupSmem > kStreamSmem - 1024 ? kFGroups * kFGroupSmem : kStreamSmem - 1024) + 1024;

template <int kId, int kCount> __device__ __forceinline__ void named_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(kId), "n"(kCount) : "memory");
}

// ------------------------------------------------------------------ intra role
__device__ __forceinline__ void fused_intra_role(const TensorMaps& maps, const PrefillParams& p,
                                                 uint8_t* ws, const WorkspaceLayout& lay,
                                                 uint8_t* smem, IntraStatics* statics,
                                                 const uint32_t tmem_base) {
    const int group = threadIdx.x >> 8;
    const int gtid = threadIdx.x & 255;
    IntraStatics& st = statics[group];
    uint8_t* gsmem = smem + group * kFGroupSmem;
    const uint32_t tmem = tmem_base + group * kIntraTmemCols;
    int32_t* hdr = reinterpret_cast<int32_t*>(ws);
    const int32_t total_items = hdr[kHdrTotalItems];
    const int32_t* order = reinterpret_cast<const int32_t*>(ws + lay.order);
    const ChunkInfo* chunks = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks);
    uint32_t* flags = reinterpret_cast<uint32_t*>(ws + lay.flags);
    const int G = p.Hv / p.Hqk;

    auto gsync = [group] {
        if (group == 0) named_sync<1, 256>();
        else if (group == 1) named_sync<2, 256>();
        else named_sync<3, 256>();
    };
    uint32_t n_done = 0;
    for (;;) {
        if (gtid == 0) st.item = atomicAdd(&hdr[kHdrItemHead], 1);
        gsync();
        const int item = st.item;
        if (item >= total_items) break;
        const int k = item / p.Hv;
        const int hv = item - k * p.Hv;
        const int c = order[k];
        const ChunkInfo ci = chunks[c];
        const size_t slot = static_cast<size_t>(c) * p.Hv + hv;
        uint8_t* rec = ws + lay.records + slot * kRecBytes;
        const bool ok = intra_item(maps, p, rec, ci, hv / G, hv, gsmem, st, tmem, gtid, gsync, n_done);
        ++n_done;
        // publish: every thread's own stores first, then the bulk stores, then the flag
        __threadfence();
        tc_fence_before_sync();
        gsync();
        if (gtid == 0) {
            bulk_wait_all();
            fence_proxy_async_all();
            __threadfence();
            st_release_u32(&flags[slot], ok ? 1u : 2u);      // 2 = produced after a timeout
        }
        if (!ok) break;
    }
}

// ---------------------------------------------------------------------------------------------
// The kernel: 512 threads per CTA (128 registers).  State CTA b runs the persistent state pass's
// role over the units b, b + n_state, ... of the rank-sorted list, its loading warp waiting for
// each record's flag; the other CTAs run two producer groups.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kFusedThreads, 1)
prefill_fused_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay, const int n_state) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ IntraStatics intra_statics[kFGroups];
    __shared__ uint32_t tmem_base_s;
    const int warp = threadIdx.x >> 5;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    if (static_cast<int>(blockIdx.x) < n_state) {
        state_stream_role<1>(maps, p, ws, lay, smem, tmem, blockIdx.x, n_state);
    } else {
        fused_intra_role(maps, p, ws, lay, smem, intra_statics, tmem);
        tc_fence_before_sync();
        __syncthreads();
    }
    if (warp == 0) tmem_dealloc(tmem, 512);
}

// =============================================================================================
// host side
// =============================================================================================
cudaError_t launch_prefill_ranked_prep(const ChunkedParams& cp, cudaStream_t stream, int mode,
                                       int split_permille, int sms) {
    if (mode == 0 && cp.p.N <= kFPrepThreads) {
        prefill_small_prep_kernel<<<1, kFPrepThreads, 0, stream>>>(cp.p.cu_seqlens, cp.p.T, cp.p.N, cp.ws,
                                                                   cp.lay, cp.p.dev_status);
        return cudaGetLastError();
    }
    prefill_fused_prep_kernel<<<1, kFPrepThreads, 0, stream>>>(cp.p.cu_seqlens, cp.p.T, cp.p.N,
                                                               cp.p.Hv, cp.ws, cp.lay,
                                                               cp.p.dev_status, mode, split_permille, sms);
    return cudaGetLastError();
}

cudaError_t launch_prefill_fused(const ChunkedParams& cp, cudaStream_t stream) {
    const PrefillParams& p = cp.p;
    DeviceInfo di;
    cudaError_t e = device_info(&di);
    if (e != cudaSuccess) return e;
    const int sms = di.sms, coop = di.cooperative;
    if (!coop || sms < 2) return cudaErrorNotSupported;
    e = ensure_dynamic_smem(prefill_fused_kernel, kFusedSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_prefill_tensor_maps(&maps, p)) return cudaErrorInvalidValue;

    e = launch_prefill_ranked_prep(cp, stream, 1);
    if (e != cudaSuccess) return e;

    // How many CTAs run the state pass: one per unit when the units are few (the shapes routed
    // here), else about 0.43 of the SMs; always at least one producer CTA.
    const long long units = static_cast<long long>(p.N) * p.Hv;
    int n_state = (sms * 7) / 16;
    if (n_state > units) n_state = static_cast<int>(units);
    if (n_state < 1) n_state = 1;
    if (n_state > sms - 1) n_state = sms - 1;
    int grid = sms;
    uint8_t* ws = cp.ws;
    WorkspaceLayout lay = cp.lay;
    PrefillParams pp = p;
    void* args[] = {&maps, &pp, &ws, &lay, &n_state};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(prefill_fused_kernel), dim3(grid),
                                       dim3(kFusedThreads), args, kFusedSmem, stream);
}

}  // namespace gdn
