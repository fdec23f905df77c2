// Chunked prefill in ONE cooperative launch: the record producers and the state pass overlap.
//
// The grid has one CTA of 768 threads per SM.  The first `n_state` CTAs run the serial state pass
// (8 chain warps + an issuing warp + a loading warp), each pulling (sequence, v-head) units from
// a queue, longest sequence first.  The other CTAs run three independent groups of 256 threads that pull
// (chunk, v-head) items from a second queue and write their records (the intra-chunk routine of
// gdn_prefill_device.cuh), in the order the state pass consumes them: by position inside the
// sequence first, by sequence rank second.  A record is published through a flag in global
// memory (release) and the state pass waits for the flag (acquire, bounded) before it copies the
// record in.  Producers never wait for consumers, every CTA is resident (cooperative launch with
// grid <= SM count), so the consumers' waits always end.
#include "gdn_prefill_device.cuh"

namespace gdn {

// =============================================================================================
// Prep: chunk table, processing order, cleared queues and flags.  One CTA.
// =============================================================================================
constexpr int kFPrepThreads = 256;

__global__ void __launch_bounds__(kFPrepThreads)
prefill_fused_prep_kernel(const int32_t* __restrict__ cu, int32_t T, int32_t N, int32_t Hv,
                          uint8_t* ws, WorkspaceLayout lay, int32_t* dev_status,
                          const int for_fused) {   // 0: only the chunk table and the ranking
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
    for (int base = 0; for_fused && base <= lay.max_nc; base += kFPrepThreads) {
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
    // rank of a sequence = its place in the order "more chunks first"; chunk j of the sequence of
    // rank r is processed at place pos[j] + r (the sequences that have a chunk j are ranks < cnt[j])
    for (int n = tid; n < N; n += kFPrepThreads) {
        const int32_t nc = seq_first[n + 1] - seq_first[n];
        const int32_t rank = cnt[nc] + atomicAdd(&fill[nc], 1);
        seq_by_rank[rank] = n;
        const int32_t first = seq_first[n];
        if (for_fused)
            for (int j = 0; j < nc; ++j) order[pos[j] + rank] = first + j;
    }
}

// =============================================================================================
// The fused kernel
// =============================================================================================
constexpr int kFusedThreads = 768;
constexpr int kFGroups = 3;                          // intra role: three groups of 256 threads
constexpr uint32_t kFGroupSmem = (kI_End + 1023u) & ~1023u;
constexpr int kFEpiWarps = 8;                        // state role: warps 0-7 chain
constexpr int kFEpiThreads = kFEpiWarps * 32;
constexpr int kFIssueWarp = kFEpiWarps;              //   warp 8: tcgen05.mma issue
constexpr int kFLoadWarp = kFEpiWarps + 1;           //   warp 9: record flags and TMA copies
constexpr int kFOutWarp0 = 12;                       //   warps 12-15: output rows
constexpr int kFOutThreads = 128;
constexpr int kFRoleThreads = kFEpiThreads + 64 + kFOutThreads;   // threads that take part in the state role
constexpr uint32_t kFStateSmem = 2 * kStageBytes + 16384;
constexpr uint32_t kFusedSmem =
    (kFGroups * kFGroupSmem > kFStateSmem ? kFGroups * kFGroupSmem : kFStateSmem) + 1024;
constexpr uint32_t kSpinFlagLimit = 1u << 22;

struct StateStatics {
    uint64_t bar_full[2], bar_free[2], bar_y[2], bar_yfree[2], bar_d1, bar_d4, bar_s, bar_u;
    int unit;
    int abort_flag;
};

template <int kId, int kCount> __device__ __forceinline__ void named_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(kId), "n"(kCount) : "memory");
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() {
    asm volatile("fence.proxy.async;" ::: "memory");
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

// ------------------------------------------------------------------ state role
// kRole 1: the copy the eight chain warps run; 0: the issuing and loading warps' copy; 2: the four
// output warps' copy.  One copy per register budget, so that each is wholly dominated by its own
// register re-allocation (the compiler budgets registers per setmaxnreg region).
template <int kRole>
__device__ __forceinline__ void fused_state_role_impl(const TensorMaps& maps, const PrefillParams& p,
                                                      uint8_t* ws, const WorkspaceLayout& lay,
                                                      uint8_t* smem, StateStatics& ss,
                                                      const uint32_t tmem) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr bool kEpi = kRole == 1, kOut = kRole == 2, kIssueLoad = kRole == 0;
    constexpr bool is_epi = kEpi;
    const int half = (warp >> 2) & 1;                 // which half of the columns this thread owns
    const int dv = (warp & 3) * 32 + lane;            // TMEM lane = state row
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    int32_t* hdr = reinterpret_cast<int32_t*>(ws);
    const int32_t* seq_first = reinterpret_cast<const int32_t*>(ws + lay.seq_first);
    const int32_t* seq_bad = reinterpret_cast<const int32_t*>(ws + lay.seq_bad);
    const int32_t* seq_by_rank = reinterpret_cast<const int32_t*>(ws + lay.seq_by_rank);
    const uint32_t* flags = reinterpret_cast<const uint32_t*>(ws + lay.flags);
    const int total_units = p.N * p.Hv;
    const int G = p.Hv / p.Hqk;
    volatile int* abortp = &ss.abort_flag;
    auto role_sync = [] { named_sync<4, kFRoleThreads>(); };
    auto out_sync = [] { named_sync<5, kFOutThreads>(); };

    // The mbarriers are initialised once and keep flipping phase from unit to unit (an mbarrier
    // must not be re-initialised while it is a valid object).  Every role thread keeps the same
    // running counts of completed phases: per unit of nc chunks, bar_full[0] completes
    // and bar_free[0] ceil(nc/2) times, bar_full[1] and bar_free[1] floor(nc/2) times, bar_d1 /
    // bar_d4 / bar_y / bar_u nc times and bar_s nc + 1 times.  Each waiter is arranged so that
    // the barrier it waits on cannot run two phases ahead of it (a parity wait cannot tell).
    if (tid == 0) {
        mbar_init(&ss.bar_full[0], 1);
        mbar_init(&ss.bar_full[1], 1);
        mbar_init(&ss.bar_free[0], kFEpiWarps + 1);     // the chain warps + the last product
        mbar_init(&ss.bar_free[1], kFEpiWarps + 1);
        mbar_init(&ss.bar_d1, 1);
        mbar_init(&ss.bar_d4, 1);
        mbar_init(&ss.bar_y[0], 1);                    // one per Y tile, see the persistent pass
        mbar_init(&ss.bar_y[1], 1);
        mbar_init(&ss.bar_yfree[0], kFOutThreads / 32);
        mbar_init(&ss.bar_yfree[1], kFOutThreads / 32);
        mbar_init(&ss.bar_s, kFEpiWarps);
        mbar_init(&ss.bar_u, kFEpiWarps);
        fence_barrier_init();
    }
    uint32_t ph_full0 = 0, ph_full1 = 0, ph_chunk = 0, ph_s = 0;

    for (;;) {
        // one lane decides for the whole role, so that every warp leaves the loop together
        if (warp == kFIssueWarp && lane == 0)
            ss.unit = *abortp ? total_units : atomicAdd(&hdr[kHdrUnitHead], 1);
        role_sync();
        const int unit = ss.unit;
        if (unit >= total_units) break;
        const int rank = unit / p.Hv;
        const int hv = unit - rank * p.Hv;
        const int n = seq_by_rank[rank];
        const int hqk = hv / G;
        const int c_first = seq_first[n];
        const int nc = seq_first[n + 1] - c_first;
        const int seq_t0 = p.cu_seqlens[n];
        const int seq_len = p.cu_seqlens[n + 1] - seq_t0;
        const int slot = p.slot_idx ? p.slot_idx[n] : n;
        const bool bad_slot = slot < 0 || slot >= p.num_slots;
        if (seq_bad[n] || bad_slot) {
            if (!seq_bad[n]) {
                if (slot >= p.num_slots && tid == 0) report(p.dev_status, kDevBadSlot);
                const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                for (int idx = tid; is_epi && idx < seq_len * 16; idx += kFEpiThreads)
                    *reinterpret_cast<uint4*>(p.o + (static_cast<size_t>(seq_t0 + (idx >> 4)) * p.Hv + hv) * kD +
                                              (idx & 15) * 8) = zero;
            }
            role_sync();
            continue;
        }
        const size_t tile_off = (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD) +
                                static_cast<size_t>(dv) * kD + half * 64;
        if (nc == 0) {          // empty sequence: the state passes through untouched
            if (is_epi) {
#pragma unroll 4
                for (int j = 0; j < 64; j += 4) {
                    const float4 x = p.init_state
                                         ? *reinterpret_cast<const float4*>(p.init_state + tile_off + j)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                    *reinterpret_cast<float4*>(p.final_state + tile_off + j) = x;
                }
            }
            role_sync();
            continue;
        }
        // parities of this unit's phases: chunk j uses (base + j), its stage (base + j / 2)
        const uint32_t b_full0 = ph_full0, b_full1 = ph_full1, b_chunk = ph_chunk, b_s = ph_s;
        ph_full0 += (nc + 1) >> 1;
        ph_full1 += nc >> 1;
        ph_chunk += nc;
        ph_s += nc + 1;
        auto par_full = [&](int j) { return (((j & 1) ? b_full1 : b_full0) + (j >> 1)) & 1u; };
        auto par_chunk = [&](int j) { return (b_chunk + j) & 1u; };
        auto par_s = [&](int j) { return (b_s + j) & 1u; };

        if (kIssueLoad && warp == kFLoadWarp) {
            // ===================== loading warp: wait for each record's flag, then copy it in
            if (lane == 0) {
                const uint8_t* records =
                    ws + lay.records + (static_cast<size_t>(c_first) * p.Hv + hv) * kRecBytes;
                const size_t rec_stride = static_cast<size_t>(p.Hv) * kRecBytes;
                const uint32_t* uflags = flags + static_cast<size_t>(c_first) * p.Hv + hv;
                for (int j = 0; j < nc; ++j) {
                    const int st = j & 1;
                    // the record must have been published by its producer (polled first: this
                    // wait overlaps the one for the stage below)
                    const uint32_t* f = uflags + static_cast<size_t>(j) * p.Hv;
                    uint32_t v = 0;
                    for (uint32_t i = 0; i < kSpinFlagLimit; ++i) {
                        v = ld_acquire_u32(f);
                        if (v != 0 || *abortp) break;
                        __nanosleep(64);
                    }
                    if (v != 1) { *abortp = 1; break; }
                    if (j >= 2) {
                        // stage st held chunk j-2: free once that chunk's last product has
                        // retired and every epilogue warp is done with its record
                        if (!wait_or_abort(&ss.bar_free[st], par_full(j - 2), abortp)) break;
                    }
                    fence_proxy_async_all();
                    uint8_t* base = smem + st * kStageBytes;
                    mbar_expect_tx(&ss.bar_full[st], kRecBytes + 16384);
                    bulk_load(base + kS_Rec, records + j * rec_stride, kRecBytes, &ss.bar_full[st]);
                    tma_load_2d(base + kS_K, &maps.k, hqk * kD, seq_t0 + j * kChunk, &ss.bar_full[st]);
                    tma_load_2d(base + kS_K + 8192, &maps.k, hqk * kD + 64, seq_t0 + j * kChunk,
                                &ss.bar_full[st]);
                }
            }
            __syncwarp();
        } else if constexpr (kIssueLoad) {
            // ===================== issuing warp: tensor-core instructions
            // (warp-uniform code run by the whole warp; one elected lane executes each instruction)
            {
                const uint32_t id64 = make_idesc_bf16(128, 64, false, false);
                const uint32_t id128mn = make_idesc_bf16(128, 128, false, true);
                const uint32_t id64mn = make_idesc_bf16(128, 64, false, true);
                const uint32_t sRec0 = smem_u32(smem + kS_Rec), sRec1 = sRec0 + kStageBytes;
                const uint64_t dW0 = make_sdesc_sw128(sRec0 + kRecW, 8192, 1024);
                const uint64_t dQ0 = make_sdesc_sw128(sRec0 + kRecQg, 16, 1024);
                const uint64_t dP0 = make_sdesc_sw128(sRec0 + kRecP, 16, 1024);
                const uint64_t dK0 = make_sdesc_sw128(sRec0 + kS_K, 8192, 1024);
                const uint64_t dW1 = make_sdesc_sw128(sRec1 + kRecW, 8192, 1024);
                const uint64_t dQ1 = make_sdesc_sw128(sRec1 + kRecQg, 16, 1024);
                const uint64_t dP1 = make_sdesc_sw128(sRec1 + kRecP, 16, 1024);
                const uint64_t dK1 = make_sdesc_sw128(sRec1 + kS_K, 8192, 1024);
                const uint32_t tS = tmem + kT_S, tD1 = tmem + kT_D1, tD4 = tmem + kT_D4;
                for (int j = 0; j < nc; ++j) {
                    const int st = j & 1;
                    const uint64_t w = st ? dW1 : dW0, qg = st ? dQ1 : dQ0, pp = st ? dP1 : dP0,
                                   kk = st ? dK1 : dK0;
                    const uint32_t tY = tmem + kT_Y + st * 64;
                    if (!wait_or_abort(&ss.bar_full[st], par_full(j), abortp)) break;
                    if (!wait_or_abort(&ss.bar_s, par_s(j), abortp)) break;    // bf16 S of chunk j in TMEM
                    tc_fence_after_sync();
                    // D1 = S W^T  (on the chain); W is MN-major: k-step ks reads 16 dk rows = 2048 bytes
                    if (elect_one()) mma_ts_c<false>(tD1, tS, w, id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 8, sdesc_advance(w, 2048), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 16, sdesc_advance(w, 4096), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 24, sdesc_advance(w, 6144), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 32, sdesc_advance(w, 8192), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 40, sdesc_advance(w, 10240), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 48, sdesc_advance(w, 12288), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 56, sdesc_advance(w, 14336), id64mn);
                    if (elect_one()) mma_commit(&ss.bar_d1);
                    // Y = S Qg^T  (off the chain) overwrites the tile the output warps read two chunks ago
                    if (j >= 2 && !wait_or_abort(&ss.bar_yfree[st], par_full(j - 2), abortp)) break;
                    if (elect_one()) mma_ts_c<false>(tY, tS, qg, id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 8, sdesc_advance(qg, 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 16, sdesc_advance(qg, 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 24, sdesc_advance(qg, 96), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 32, sdesc_advance(qg, 8192), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 40, sdesc_advance(qg, 8192 + 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 48, sdesc_advance(qg, 8192 + 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 56, sdesc_advance(qg, 8192 + 96), id64);
                    if (!wait_or_abort(&ss.bar_u, par_chunk(j), abortp)) break;    // U operands in TMEM
                    tc_fence_after_sync();
                    // D4 = (U decayed, hi + lo) K   (K tile MN-major: 16 tokens = 2048 bytes)
                    if (elect_one()) mma_ts_c<false>(tD4, tmem + kT_Us, kk, id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 8, sdesc_advance(kk, 2048), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 16, sdesc_advance(kk, 4096), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 24, sdesc_advance(kk, 6144), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo, kk, id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 8, sdesc_advance(kk, 2048), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 16, sdesc_advance(kk, 4096), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 24, sdesc_advance(kk, 6144), id128mn);
                    if (elect_one()) mma_commit(&ss.bar_d4);
                    // Y += U P^T
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U, pp, id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 8, sdesc_advance(pp, 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 16, sdesc_advance(pp, 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 24, sdesc_advance(pp, 96), id64);
                    if (elect_one()) mma_commit(&ss.bar_y[st]);
                    if (elect_one()) mma_commit(&ss.bar_free[st]);
                }
            }
            __syncwarp();
        } else if constexpr (kOut) {
            // ===================== output warps: Y = S Qg^T + U P^T (fp32, TMEM) -> o rows, one warp
            // per TMEM lane quadrant; transposed through shared memory, written as whole rows
            const int q4 = warp & 3;
            const uint32_t olane = static_cast<uint32_t>(q4 * 32) << 16;
            const int ot = tid - kFOutWarp0 * 32;
            const size_t tok_stride = static_cast<size_t>(p.Hv) * kD;
            __nv_bfloat16* sO = reinterpret_cast<__nv_bfloat16*>(smem + kS_Out);
            bool ok = true;
            for (int j = 0; j < nc; ++j) {
                const int buf = j & 1;
                // every warp runs both group barriers of every chunk, also after a failed wait
                if (ok && !warp_wait_or_abort(&ss.bar_y[buf], par_full(j), abortp)) ok = false;
                tc_fence_after_sync();
                // The Y tile (lanes = dv, columns = tokens) is read as accumulator fragments, 16 lanes
                // at a time, rounded in pairs and stored transposed, 8 dv of one token per 16 bytes,
                // into a [token][dv] tile of two 128B-swizzled halves of 64 dv: far fewer
                // instructions than scalar conversions and two-byte stores, and what these warps
                // issue comes out of the chain warps' issue slots.
                if (ok) {
                    const uint32_t tY = tmem + kT_Y + buf * 64;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t y[32];
                        tmem_ld_16x256b_x8(tY + olane + (static_cast<uint32_t>(16 * h) << 16), y);
                        tmem_wait_ld();
                        const int dv0 = q4 * 32 + 16 * h + 8 * ((lane >> 3) & 1);    // 8 dv behind this lane's address
                        const uint32_t dst = smem_u32(sO) + (dv0 >> 6) * 8192;
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            stmatrix_x2_trans(dst + sw128_offset(8 * i + (lane & 7), (dv0 & 63) >> 3),
                                              pack_bf16(__uint_as_float(y[4 * i]), __uint_as_float(y[4 * i + 1])),
                                              pack_bf16(__uint_as_float(y[4 * i + 2]), __uint_as_float(y[4 * i + 3])));
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&ss.bar_yfree[buf]);     // the tile may be overwritten
                out_sync();
                if (ok) {
                    const int len = min(kChunk, seq_len - j * kChunk);
                    __nv_bfloat16* og = p.o + (static_cast<size_t>(seq_t0 + j * kChunk) * p.Hv + hv) * kD;
                    const uint8_t* src = reinterpret_cast<const uint8_t*>(sO) + ((ot & 15) >> 3) * 8192;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int row = it * 8 + (ot >> 4), piece = ot & 15;
                        if (row < len)
                            *reinterpret_cast<uint4*>(og + row * tok_stride + piece * 8) =
                                *reinterpret_cast<const uint4*>(src + sw128_offset(row, piece & 7));
                    }
                }
                out_sync();
            }
        } else {
            // ===================== chain warps: U and the state refresh (the dependent chain)
            // The fp32 master state lives in registers (64 per thread: row dv, columns
            // [64*half, 64*half + 64)); its bf16 copy in TMEM is the A operand of S W^T and S Qg^T.
            auto hand_over = [&](uint64_t* bar) {     // after tcgen05.st: publish to the issuing lane
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar);
            };
            float S[64];
            auto store_state_bf16 = [&]() {           // S (fp32 regs) -> bf16 A operand in TMEM
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(S[c0 + 2 * j], S[c0 + 2 * j + 1]);
                    tmem_st16(tmem + kT_S + lane_base + half * 32 + (c0 >> 1), pk);
                }
            };
            bool ok = true;
            auto await = [&](uint64_t* bar, uint32_t parity) {   // bounded wait + tcgen05 fence
                if (ok && !warp_wait_or_abort(bar, parity, abortp)) ok = false;
                tc_fence_after_sync();
            };
            // Every warp runs every group barrier and hand-over below, also after a wait has
            // failed (ok == false: later waits and all work are skipped), so that no warp is ever
            // left alone at a barrier.
            if (p.init_state) {
#pragma unroll
                for (int j = 0; j < 64; j += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(p.init_state + tile_off + j);
                    S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 64; ++j) S[j] = 0.f;
            }
            store_state_bf16();
            hand_over(&ss.bar_s);
            for (int j = 0; j < nc; ++j) {
                const int st = j & 1;
                const uint8_t* base = smem + st * kStageBytes;
                await(&ss.bar_full[st], par_full(j));
                await(&ss.bar_d1, par_chunk(j));
                if (ok) {   // U^T[dv][c] = U~^T - D1 for the thread's 32 tokens [32*half, 32*half+32)
                    const float4* sU = reinterpret_cast<const float4*>(base + kS_Rec + kRecU);
                    const float* sdec = reinterpret_cast<const float*>(base + kS_Rec + kRecDecay);
#pragma unroll
                    for (int c0 = 0; c0 < 32; c0 += 16) {
                        const int cb = half * 32 + c0;
                        uint32_t x[16];
                        tmem_ld16(tmem + kT_D1 + lane_base + cb, x);
                        tmem_wait_ld();
                        uint32_t pu[8], ph[8], pl[8];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float4 ut = sU[((cb >> 2) + q4) * kD + dv];
                            const float4 dd = *reinterpret_cast<const float4*>(sdec + cb + 4 * q4);
                            const float u0 = ut.x - __uint_as_float(x[4 * q4 + 0]);
                            const float u1 = ut.y - __uint_as_float(x[4 * q4 + 1]);
                            const float u2 = ut.z - __uint_as_float(x[4 * q4 + 2]);
                            const float u3 = ut.w - __uint_as_float(x[4 * q4 + 3]);
                            const float s0 = u0 * dd.x, s1 = u1 * dd.y, s2 = u2 * dd.z, s3 = u3 * dd.w;
                            pu[2 * q4] = pack_bf16(u0, u1);
                            pu[2 * q4 + 1] = pack_bf16(u2, u3);
                            ph[2 * q4] = pack_bf16(s0, s1);
                            ph[2 * q4 + 1] = pack_bf16(s2, s3);
                            pl[2 * q4] = pack_bf16(s0 - __uint_as_float(ph[2 * q4] << 16),
                                                   s1 - __uint_as_float(ph[2 * q4] & 0xffff0000u));
                            pl[2 * q4 + 1] = pack_bf16(s2 - __uint_as_float(ph[2 * q4 + 1] << 16),
                                                       s3 - __uint_as_float(ph[2 * q4 + 1] & 0xffff0000u));
                        }
                        tmem_st8(tmem + kT_Us + lane_base + (cb >> 1), ph);
                        tmem_st8(tmem + kT_UsLo + lane_base + (cb >> 1), pl);
                        tmem_st8(tmem + kT_U + lane_base + (cb >> 1), pu);
                    }
                }
                hand_over(&ss.bar_u);
                const bool last = j + 1 == nc;
                await(&ss.bar_d4, par_chunk(j));
                if (ok) {   // S <- e^{b_C} S + D4 on the thread's 64 dk columns
                    const float gC = reinterpret_cast<const float*>(base + kS_Rec + kRecGammaC)[0];
#pragma unroll
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t xa[16], xb[16];
                        tmem_ld16(tmem + kT_D4 + lane_base + half * 64 + c0, xa);
                        tmem_ld16(tmem + kT_D4 + lane_base + half * 64 + c0 + 16, xb);
                        tmem_wait_ld();
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            S[c0 + jj] = fmaf(gC, S[c0 + jj], __uint_as_float(xa[jj]));
                            S[c0 + 16 + jj] = fmaf(gC, S[c0 + 16 + jj], __uint_as_float(xb[jj]));
                        }
                    }
                    if (!last) {
                        store_state_bf16();
                    } else {
#pragma unroll
                        for (int j4 = 0; j4 < 64; j4 += 4)
                            *reinterpret_cast<float4*>(p.final_state + tile_off + j4) =
                                make_float4(S[j4], S[j4 + 1], S[j4 + 2], S[j4 + 3]);
                    }
                }
                if (lane == 0) mbar_arrive(&ss.bar_free[st]);     // this warp is done with the stage
                hand_over(&ss.bar_s);
            }
        }
        tc_fence_before_sync();
        role_sync();                                   // end of the unit: barriers are re-armed next
        if (warp == kFIssueWarp && lane == 0 && *abortp) {
            report(p.dev_status, kDevTimeout);
            // let copies already in flight land before the shared memory is reused or freed
            mbar_wait(&ss.bar_full[0], 0, 1u << 12);
            mbar_wait(&ss.bar_full[1], 0, 1u << 12);
        }
    }
}

__device__ __forceinline__ void fused_state_role(const TensorMaps& maps, const PrefillParams& p,
                                                 uint8_t* ws, const WorkspaceLayout& lay,
                                                 uint8_t* smem, StateStatics& ss,
                                                 const uint32_t tmem) {
    // The kernel is compiled for 768 threads (80 registers each) because of the producer CTAs.
    // In a state-pass CTA the spare warps and the issuing / loading group hand registers back and
    // the eight chain warps take 128 each, enough to keep the fp32 master state in registers.
    // setmaxnreg works on groups of four warps and WAITS, unbounded, until the registers it asks
    // for have been given back by other warps of the SAME CTA (registers the SM never gave this CTA
    // do not count: asking for more than was handed back hangs the CTA).  All counts are multiples
    // of 16 (the allocation unit may be that coarse).  Given back: 256 x 48 (spare warps) +
    // 128 x 16 (issuing / loading) = 14336, the output warps keep their 80 (the call only tells
    // the compiler their budget); taken by the chain warps: 256 x 48 = 12288.
    const int warp = threadIdx.x >> 5;
    if (warp >= 16) {
        reg_dealloc<32>();                            // spare warps of the CTA
    } else if (warp >= kFOutWarp0) {
        reg_dealloc<80>();
        fused_state_role_impl<2>(maps, p, ws, lay, smem, ss, tmem);
    } else if (warp >= 8) {
        reg_dealloc<64>();
        if (warp <= kFLoadWarp) fused_state_role_impl<0>(maps, p, ws, lay, smem, ss, tmem);
    } else {
        reg_alloc<128>();
        fused_state_role_impl<1>(maps, p, ws, lay, smem, ss, tmem);
    }
}

__global__ void __launch_bounds__(kFusedThreads, 1)
prefill_fused_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay, const int n_state) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ IntraStatics intra_statics[kFGroups];
    __shared__ StateStatics state_statics;
    __shared__ uint32_t tmem_base_s;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) state_statics.abort_flag = 0;
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    if (static_cast<int>(blockIdx.x) < n_state)
        fused_state_role(maps, p, ws, lay, smem, state_statics, tmem);
    else
        fused_intra_role(maps, p, ws, lay, smem, intra_statics, tmem);
    tc_fence_before_sync();
    __syncthreads();

    if (warp == 0) tmem_dealloc(tmem, 512);
}

// =============================================================================================
// host side
// =============================================================================================
cudaError_t launch_prefill_ranked_prep(const ChunkedParams& cp, cudaStream_t stream, bool for_fused) {
    prefill_fused_prep_kernel<<<1, kFPrepThreads, 0, stream>>>(cp.p.cu_seqlens, cp.p.T, cp.p.N,
                                                               cp.p.Hv, cp.ws, cp.lay,
                                                               cp.p.dev_status, for_fused ? 1 : 0);
    return cudaGetLastError();
}

cudaError_t launch_prefill_fused(const ChunkedParams& cp, cudaStream_t stream) {
    const PrefillParams& p = cp.p;
    int dev = 0, sms = 0, coop = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (!coop || sms < 2) return cudaErrorNotSupported;
    e = cudaFuncSetAttribute(prefill_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kFusedSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_prefill_tensor_maps(&maps, p)) return cudaErrorInvalidValue;

    e = launch_prefill_ranked_prep(cp, stream, true);
    if (e != cudaSuccess) return e;

    // How many CTAs run the state pass: measured best near 0.43 of the SMs when there are more
    // units than that (one chunk step of the chain holds an SM ~2.8 us, an item holds a third of
    // an SM ~15 us); never more than there are units, and always at least one producer CTA.
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
