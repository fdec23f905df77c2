// Chunked prefill on the sm_100a tensor cores (tcgen05 + TMEM, operands staged by TMA).
// The algebra and the record layout are described in gdn_prefill_chunk.cuh.
#include "gdn_prefill_device.cuh"

namespace gdn {

// =============================================================================================
// K0: chunk table from cu_seqlens (device side, no host sync).  One CTA.
// =============================================================================================
constexpr int kPrepThreads = 256;

__global__ void __launch_bounds__(kPrepThreads)
prefill_prep_kernel(const int32_t* __restrict__ cu, int32_t T, int32_t N, uint8_t* ws,
                    WorkspaceLayout lay, int32_t* dev_status) {
    int32_t* total_chunks = reinterpret_cast<int32_t*>(ws);
    int32_t* seq_first = reinterpret_cast<int32_t*>(ws + lay.seq_first);
    int32_t* seq_bad = reinterpret_cast<int32_t*>(ws + lay.seq_bad);
    ChunkInfo* chunks = reinterpret_cast<ChunkInfo*>(ws + lay.chunks);
    __shared__ int32_t warp_sums[kPrepThreads / 32];
    __shared__ int32_t running;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();        // the next kernel's CTAs may become resident (they wait for us)
    if (tid == 0) {
        running = 0;
        if (cu[0] != 0 || cu[N] != T) report(dev_status, kDevBadCuSeqlens);
    }
    __syncthreads();
    for (int base = 0; base < N; base += kPrepThreads) {
        const int n = base + tid;
        int32_t nc = 0;
        if (n < N) {
            const int32_t t0 = cu[n], t1 = cu[n + 1];
            const bool ok = t0 >= 0 && t1 >= t0 && t1 <= T;
            if (!ok) report(dev_status, kDevBadCuSeqlens);
            seq_bad[n] = ok ? 0 : 1;
            nc = ok ? (t1 - t0 + kChunk - 1) / kChunk : 0;
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
        if (tid == kPrepThreads - 1) running = first + nc;
        __syncthreads();
    }
    if (tid == 0) {
        seq_first[N] = running;
        *total_chunks = running;
    }
}

// =============================================================================================
// K1: intra-chunk quantities, one CTA (256 threads) per (chunk, v-head); see intra_item().
// =============================================================================================
// kInlineTable: a batch of at most kInlineTableSeqs sequences needs no table-building launch in
// front: every CTA finds its own chunk by walking cu_seqlens, and CTA (0, 0) writes the two small
// per-sequence tables the state pass reads after this kernel (2.5 us less on a 100-token prompt).
template <bool kInlineTable>
__global__ void __launch_bounds__(kIntraThreads, 4)
prefill_intra_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay) {
    const int c = blockIdx.x;
    const int hv = blockIdx.y;
    pdl_launch_dependents();
    pdl_wait();                     // the chunk table is the previous kernel's
    ChunkInfo ci;
    if constexpr (kInlineTable) {
        // same rules as the table-building kernel: a sequence whose bounds are out of order or
        // out of range has no chunks and is flagged
        const bool writer = blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0;
        int32_t* seq_first = reinterpret_cast<int32_t*>(ws + lay.seq_first);
        int32_t* seq_bad = reinterpret_cast<int32_t*>(ws + lay.seq_bad);
        // one round trip for all bounds (a loop of dependent global loads would cost one each)
        __shared__ int32_t s_cu[kInlineTableSeqs + 1];
        if (static_cast<int>(threadIdx.x) <= p.N) s_cu[threadIdx.x] = p.cu_seqlens[threadIdx.x];
        __syncthreads();
        if (writer && (s_cu[0] != 0 || s_cu[p.N] != p.T)) report(p.dev_status, kDevBadCuSeqlens);
        int first = 0;
        ci.seq = -1;
        for (int n = 0; n < p.N; ++n) {
            const int32_t t0 = s_cu[n], t1 = s_cu[n + 1];
            const bool ok = t0 >= 0 && t1 >= t0 && t1 <= p.T;
            const int nc = ok ? (t1 - t0 + kChunk - 1) / kChunk : 0;
            if (writer) {
                if (!ok) report(p.dev_status, kDevBadCuSeqlens);
                seq_bad[n] = ok ? 0 : 1;
                seq_first[n] = first;
            }
            if (c >= first && c < first + nc) {
                ci.seq = n;
                ci.t0 = t0 + (c - first) * kChunk;
                ci.len = min(kChunk, t1 - ci.t0);
                ci.pad = 0;
            }
            first += nc;
        }
        if (writer) {
            seq_first[p.N] = first;
            *reinterpret_cast<int32_t*>(ws) = first;
            // sequences by chunk count, more chunks first (the persistent state pass walks them in
            // this order); with so few sequences, by counting
            int32_t* seq_by_rank = reinterpret_cast<int32_t*>(ws + lay.seq_by_rank);
            for (int n = 0; n < p.N; ++n) {
                const int nc_n = seq_first[n + 1] - seq_first[n];
                int rank = 0;
                for (int m = 0; m < p.N; ++m) {
                    const int nc_m = seq_first[m + 1] - seq_first[m];
                    rank += (nc_m > nc_n || (nc_m == nc_n && m < n)) ? 1 : 0;
                }
                seq_by_rank[rank] = n;
            }
        }
        if (ci.seq < 0) return;
    } else {
        const int32_t total = *reinterpret_cast<const int32_t*>(ws);
        if (c >= total) return;
        ci = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks)[c];
    }
    const int hqk = hv / (p.Hv / p.Hqk);
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
    intra_item(maps, p, rec, ci, hqk, hv, smem, st, tmem, tid, [] { __syncthreads(); });
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
}

// =============================================================================================
// K2: inter-chunk state pass, one CTA per (sequence, v-head): 8 epilogue warps + 1 issuing warp.
//
// Per chunk the dependent chain is  D1 = S W^T  ->  U = U~ - D1  ->  D4 = (U decayed) K  ->
// S = e^{b_C} S + D4.  The output product  Y = S Qg^T + U P^T  is accumulated in a second,
// double-buffered TMEM tile and is turned into o rows one chunk later, while the next chunk's
// D1 is in flight.  One lane of warp 8 issues every TMA copy and every tcgen05.mma; the
// epilogue warps hand it the bf16 state ("s") and the U operands ("u") through mbarriers, so
// nobody but the issuing lane ever waits for the tensor pipe to accept instructions.
// =============================================================================================
__global__ void __launch_bounds__(kStateThreads, 1)
prefill_state_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay) {
    const int n = blockIdx.x / p.Hv;
    const int hv = blockIdx.x - n * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_epi = warp < kStateEpiWarps;
    const int half = (warp >> 2) & 1;                 // which half of the columns this thread owns
    const int dv = (warp & 3) * 32 + lane;            // TMEM lane = state row
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;

    const int32_t* seq_first = reinterpret_cast<const int32_t*>(ws + lay.seq_first);
    const int32_t* seq_bad = reinterpret_cast<const int32_t*>(ws + lay.seq_bad);
    pdl_wait();                     // tables and records are the previous kernels'
    if (seq_bad[n]) return;
    const int c_first = seq_first[n];
    const int nc = seq_first[n + 1] - c_first;
    const int seq_t0 = p.cu_seqlens[n];
    const int seq_len = p.cu_seqlens[n + 1] - seq_t0;

    const int slot = p.slot_idx ? p.slot_idx[n] : n;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && tid == 0) report(p.dev_status, kDevBadSlot);
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        for (int idx = tid; idx < seq_len * 16; idx += kStateThreads)
            *reinterpret_cast<uint4*>(p.o + (static_cast<size_t>(seq_t0 + (idx >> 4)) * p.Hv + hv) * kD +
                                      (idx & 15) * 8) = zero;
        return;
    }

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ uint64_t bar_full[2], bar_d1, bar_d4, bar_y, bar_s, bar_u;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    // the thread's 64 state columns [64*half, 64*half+64) of row dv, fp32 master copy
    float S[64];
    const size_t tile_off = (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD) +
                            static_cast<size_t>(dv) * kD + half * 64;
    if (is_epi && p.init_state) {
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
            const float4 x = *reinterpret_cast<const float4*>(p.init_state + tile_off + j);
            S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < 64; ++j) S[j] = 0.f;
    }

    if (nc > 0) {
        if (tid == 0) {
            mbar_init(&bar_full[0], 1);
            mbar_init(&bar_full[1], 1);
            mbar_init(&bar_d1, 1);
            mbar_init(&bar_d4, 1);
            mbar_init(&bar_y, 1);
            mbar_init(&bar_s, kStateEpiWarps);
            mbar_init(&bar_u, kStateEpiWarps);
            abort_flag = 0;
            fence_barrier_init();
        }
        if (warp == kStateEpiWarps) {
            tmem_alloc(&tmem_base_s, kStateTmemCols);
            tmem_relinquish();
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        const uint32_t tmem = tmem_base_s;
        volatile int* abortp = &abort_flag;

        if (!is_epi) {
            // ===================== issuing warp: TMA copies and tensor-core instructions
            if (lane == 0) {
                const uint8_t* records =
                    ws + lay.records + (static_cast<size_t>(c_first) * p.Hv + hv) * kRecBytes;
                const size_t rec_stride = static_cast<size_t>(p.Hv) * kRecBytes;
                auto issue_loads = [&](int j) {
                    const int st = j & 1;
                    uint8_t* base = smem + st * kStageBytes;
                    mbar_expect_tx(&bar_full[st], kRecBytes + 16384);
                    bulk_load(base + kS_Rec, records + j * rec_stride, kRecBytes, &bar_full[st]);
                    tma_load_2d(base + kS_K, &maps.k, hqk * kD, seq_t0 + j * kChunk, &bar_full[st]);
                    tma_load_2d(base + kS_K + 8192, &maps.k, hqk * kD + 64, seq_t0 + j * kChunk,
                                &bar_full[st]);
                };
                const uint32_t id64 = make_idesc_bf16(128, 64, false, false);
                const uint32_t id128mn = make_idesc_bf16(128, 128, false, true);
                const uint32_t id64mn = make_idesc_bf16(128, 64, false, true);
                // base descriptors of both stages, built once; the loop only adds offsets
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
                issue_loads(0);
                if (nc > 1) issue_loads(1);
                for (int j = 0; j < nc; ++j) {
                    const int st = j & 1;
                    const uint64_t w = st ? dW1 : dW0, qg = st ? dQ1 : dQ0, pp = st ? dP1 : dP0,
                                   kk = st ? dK1 : dK0;
                    const uint32_t tY = tmem + kT_Y + st * 64;
                    if (!wait_or_abort(&bar_full[st], (j >> 1) & 1, abortp)) break;
                    if (!wait_or_abort(&bar_s, j & 1, abortp)) break;       // bf16 S of chunk j in TMEM
                    tc_fence_after_sync();
                    // D1 = S W^T  (on the chain); W is MN-major: k-step ks reads 16 dk rows = 2048 bytes
                    mma_ts_c<false>(tD1, tS, w, id64mn);
                    mma_ts_c<true>(tD1, tS + 8, sdesc_advance(w, 2048), id64mn);
                    mma_ts_c<true>(tD1, tS + 16, sdesc_advance(w, 4096), id64mn);
                    mma_ts_c<true>(tD1, tS + 24, sdesc_advance(w, 6144), id64mn);
                    mma_ts_c<true>(tD1, tS + 32, sdesc_advance(w, 8192), id64mn);
                    mma_ts_c<true>(tD1, tS + 40, sdesc_advance(w, 10240), id64mn);
                    mma_ts_c<true>(tD1, tS + 48, sdesc_advance(w, 12288), id64mn);
                    mma_ts_c<true>(tD1, tS + 56, sdesc_advance(w, 14336), id64mn);
                    mma_commit(&bar_d1);
                    if (j > 0 && j + 1 < nc) {
                        // the other stage is free once chunk j-1's last product has retired (the
                        // epilogue warps left it before they handed over this chunk's S)
                        if (!wait_or_abort(&bar_y, (j - 1) & 1, abortp)) break;
                        issue_loads(j + 1);
                    }
                    // Y = S Qg^T  (off the chain)
                    mma_ts_c<false>(tY, tS, qg, id64);
                    mma_ts_c<true>(tY, tS + 8, sdesc_advance(qg, 32), id64);
                    mma_ts_c<true>(tY, tS + 16, sdesc_advance(qg, 64), id64);
                    mma_ts_c<true>(tY, tS + 24, sdesc_advance(qg, 96), id64);
                    mma_ts_c<true>(tY, tS + 32, sdesc_advance(qg, 8192), id64);
                    mma_ts_c<true>(tY, tS + 40, sdesc_advance(qg, 8192 + 32), id64);
                    mma_ts_c<true>(tY, tS + 48, sdesc_advance(qg, 8192 + 64), id64);
                    mma_ts_c<true>(tY, tS + 56, sdesc_advance(qg, 8192 + 96), id64);
                    if (!wait_or_abort(&bar_u, j & 1, abortp)) break;       // U operands in TMEM
                    tc_fence_after_sync();
                    // D4 = (U decayed, hi + lo) K   (K tile MN-major: 16 tokens = 2048 bytes)
                    mma_ts_c<false>(tD4, tmem + kT_Us, kk, id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_Us + 8, sdesc_advance(kk, 2048), id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_Us + 16, sdesc_advance(kk, 4096), id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_Us + 24, sdesc_advance(kk, 6144), id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_UsLo, kk, id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_UsLo + 8, sdesc_advance(kk, 2048), id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_UsLo + 16, sdesc_advance(kk, 4096), id128mn);
                    mma_ts_c<true>(tD4, tmem + kT_UsLo + 24, sdesc_advance(kk, 6144), id128mn);
                    mma_commit(&bar_d4);
                    // Y += U P^T
                    mma_ts_c<true>(tY, tmem + kT_U, pp, id64);
                    mma_ts_c<true>(tY, tmem + kT_U + 8, sdesc_advance(pp, 32), id64);
                    mma_ts_c<true>(tY, tmem + kT_U + 16, sdesc_advance(pp, 64), id64);
                    mma_ts_c<true>(tY, tmem + kT_U + 24, sdesc_advance(pp, 96), id64);
                    mma_commit(&bar_y);
                }
            }
            __syncwarp();
        } else {
            // ===================== epilogue warps: the fp32 state, U, and the output rows
            auto hand_over = [&](uint64_t* bar) {     // after tcgen05.st: publish to the issuing lane
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar);
            };
            auto store_state_bf16 = [&]() {           // S (fp32 regs) -> bf16 A operand in TMEM
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 32) {
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(S[c0 + 2 * j], S[c0 + 2 * j + 1]);
                    tmem_st16(tmem + kT_S + lane_base + half * 32 + (c0 >> 1), pk);
                }
            };
            // o rows of chunk j from Y[j & 1], in two parts that fit the two waits of the chain:
            // (A) scale, round to bf16, transpose into shared memory; (B) write whole rows in
            // 16-byte pieces.  A group barrier precedes each part (all of B(j-1) before A(j),
            // all of A(j) before B(j)).
            auto outputs_stage = [&](int j) {
                const uint32_t tY = tmem + kT_Y + (j & 1) * 64;
                __nv_bfloat16* sO = reinterpret_cast<__nv_bfloat16*>(smem + kS_Out);
                uint32_t x[16], y[16];
                tmem_ld16(tY + lane_base + half * 32, x);
                tmem_ld16(tY + lane_base + half * 32 + 16, y);
                tmem_wait_ld();
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    sO[(half * 32 + jj) * kD + dv] = __float2bfloat16(__uint_as_float(x[jj]));
                    sO[(half * 32 + 16 + jj) * kD + dv] = __float2bfloat16(__uint_as_float(y[jj]));
                }
            };
            auto outputs_flush = [&](int j) {
                const __nv_bfloat16* sO = reinterpret_cast<const __nv_bfloat16*>(smem + kS_Out);
                const int len = min(kChunk, seq_len - j * kChunk);
                __nv_bfloat16* og = p.o + (static_cast<size_t>(seq_t0 + j * kChunk) * p.Hv + hv) * kD;
                const size_t tok_stride = static_cast<size_t>(p.Hv) * kD;
#pragma unroll
                for (int it = 0; it < 4; ++it) {
                    const int row = it * 16 + (tid >> 4), piece = tid & 15;
                    if (row < len)
                        *reinterpret_cast<uint4*>(og + row * tok_stride + piece * 8) =
                            *reinterpret_cast<const uint4*>(sO + row * kD + piece * 8);
                }
            };

            store_state_bf16();
            hand_over(&bar_s);
            bool ok = true;
            auto await = [&](uint64_t* bar, uint32_t parity) {   // bounded wait + tcgen05 fence
                if (ok && !warp_wait_or_abort(bar, parity, abortp)) ok = false;
                tc_fence_after_sync();
            };
            for (int j = 0; j < nc; ++j) {
                const int st = j & 1;
                const uint8_t* base = smem + st * kStageBytes;
                // Every warp runs every group barrier and hand-over of every iteration, also after a
                // wait has failed (ok == false: later waits and all work are skipped), so that no
                // warp is ever left alone at a barrier.
                if (j > 0) {     // part A of the previous chunk's outputs, while D1 is in flight
                    await(&bar_y, (j - 1) & 1);
                    epi_group_sync();
                    if (ok) outputs_stage(j - 1);
                }
                await(&bar_full[st], (j >> 1) & 1);
                await(&bar_d1, j & 1);

                const float* sdec = reinterpret_cast<const float*>(base + kS_Rec + kRecDecay);
                if (ok) {   // U^T[dv][c] = U~^T - D1 for the thread's 32 tokens [32*half, 32*half+32)
                    const float4* sU = reinterpret_cast<const float4*>(base + kS_Rec + kRecU);
                    uint32_t xa[16], xb[16];
                    tmem_ld16(tmem + kT_D1 + lane_base + half * 32, xa);
                    tmem_ld16(tmem + kT_D1 + lane_base + half * 32 + 16, xb);
                    tmem_wait_ld();
                    auto u_block = [&](const uint32_t (&x)[16], const int cb) {
                        float u[16];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float4 ut = sU[((cb >> 2) + q4) * kD + dv];
                            u[4 * q4 + 0] = ut.x - __uint_as_float(x[4 * q4 + 0]);
                            u[4 * q4 + 1] = ut.y - __uint_as_float(x[4 * q4 + 1]);
                            u[4 * q4 + 2] = ut.z - __uint_as_float(x[4 * q4 + 2]);
                            u[4 * q4 + 3] = ut.w - __uint_as_float(x[4 * q4 + 3]);
                        }
                        // U for the output product; the decayed U for the state update is kept
                        // as hi + lo bf16 pairs so that its rounding does not limit the state
                        uint32_t pu[8], ph[8], pl[8];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float4 dd = *reinterpret_cast<const float4*>(sdec + cb + 4 * q4);
                            const float s0 = u[4 * q4 + 0] * dd.x, s1 = u[4 * q4 + 1] * dd.y;
                            const float s2 = u[4 * q4 + 2] * dd.z, s3 = u[4 * q4 + 3] * dd.w;
                            pu[2 * q4] = pack_bf16(u[4 * q4 + 0], u[4 * q4 + 1]);
                            pu[2 * q4 + 1] = pack_bf16(u[4 * q4 + 2], u[4 * q4 + 3]);
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
                    };
                    u_block(xa, half * 32);
                    u_block(xb, half * 32 + 16);
                }
                hand_over(&bar_u);
                if (j > 0) {     // part B, while this chunk's state product is in flight
                    epi_group_sync();
                    if (ok) outputs_flush(j - 1);
                }

                await(&bar_d4, j & 1);
                if (ok) {   // S <- e^{b_C} S + D4 on the thread's 64 dk columns; refresh the bf16 copy
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
                    store_state_bf16();
                }
                hand_over(&bar_s);
            }
            await(&bar_y, (nc - 1) & 1);
            epi_group_sync();
            if (ok) outputs_stage(nc - 1);
            epi_group_sync();
            if (ok) outputs_flush(nc - 1);
        }
        tc_fence_before_sync();
        __syncthreads();
        const bool failed = abort_flag != 0;
        if (failed && warp == kStateEpiWarps && lane == 0) {
            report(p.dev_status, kDevTimeout);
            // let copies already in flight land before the CTA's shared memory goes away
            mbar_wait(&bar_full[0], 0, 1u << 12);
            mbar_wait(&bar_full[1], 0, 1u << 12);
        }
        __syncwarp();
        if (warp == kStateEpiWarps) tmem_dealloc(tmem, kStateTmemCols);
        if (failed) return;
    }

    if (is_epi) {
#pragma unroll
        for (int j = 0; j < 64; j += 4)
            *reinterpret_cast<float4*>(p.final_state + tile_off + j) =
                make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
    }
}

// =============================================================================================
// host side
// =============================================================================================
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) !=
                cudaSuccess || q != cudaDriverEntryPointSuccess)
            return nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// [rows][cols] bf16 row-major tensor, boxes of 64 rows x 64 columns (128 bytes), 128B swizzle,
// out-of-range rows read as zero.
bool make_token_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols) {
    EncodeTiledFn enc = encode_fn();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
    const cuuint32_t box[2] = {64, 64};
    const cuuint32_t elem[2] = {1, 1};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
               elem, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool make_prefill_tensor_maps(TensorMaps* maps, const PrefillParams& p) {
    return make_token_map(&maps->q, p.q, p.T, static_cast<int64_t>(p.Hqk) * kD) &&
           make_token_map(&maps->k, p.k, p.T, static_cast<int64_t>(p.Hqk) * kD) &&
           make_token_map(&maps->v, p.v, p.T, static_cast<int64_t>(p.Hv) * kD);
}

bool prefill_tables_inline(const ChunkedParams& cp) {
    // Worth it for small batches only: the walk costs every CTA a barrier and a few hundred cycles,
    // which over many waves of CTAs adds up to more than the launch it saves (config 3: +2 us).
    return cp.p.N <= kInlineTableSeqs && cp.lay.max_chunks > 0 &&
           static_cast<long long>(cp.lay.max_chunks) * cp.p.Hv <= kInlineTableItems;
}

cudaError_t launch_prefill_intra(const TensorMaps& maps, const ChunkedParams& cp, cudaStream_t stream,
                                 bool inline_tables) {
    auto kernel = inline_tables ? prefill_intra_kernel<true> : prefill_intra_kernel<false>;
    cudaError_t e = ensure_dynamic_smem(kernel, kIntraSmem);
    if (e != cudaSuccess) return e;
    dim3 grid(cp.lay.max_chunks, cp.p.Hv);
    return launch_dependent(kernel, grid, dim3(kIntraThreads), kIntraSmem, stream, maps, cp.p, cp.ws,
                            cp.lay);
}

cudaError_t launch_prefill_chunked(const ChunkedParams& cp, cudaStream_t stream) {
    const PrefillParams& p = cp.p;
    cudaError_t e = ensure_dynamic_smem(prefill_state_kernel, kStateSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_prefill_tensor_maps(&maps, p)) return cudaErrorInvalidValue;

    if (prefill_tables_inline(cp)) {
        // few sequences: no table-building launch, the intra-chunk kernel walks cu_seqlens itself
        e = launch_prefill_intra(maps, cp, stream, true);
        if (e != cudaSuccess) return e;
    } else {
        prefill_prep_kernel<<<1, kPrepThreads, 0, stream>>>(p.cu_seqlens, p.T, p.N, cp.ws, cp.lay,
                                                            p.dev_status);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        if (cp.lay.max_chunks > 0) {
            e = launch_prefill_intra(maps, cp, stream, false);
            if (e != cudaSuccess) return e;
        }
    }
    return launch_dependent(prefill_state_kernel, dim3(p.N * p.Hv), dim3(kStateThreads), kStateSmem,
                            stream, maps, p, cp.ws, cp.lay);
}

}  // namespace gdn
