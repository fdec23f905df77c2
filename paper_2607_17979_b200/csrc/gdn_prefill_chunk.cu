// Chunked prefill on the sm_100a tensor cores (tcgen05 + TMEM, operands staged by TMA).
// The algebra and the record layout are described in gdn_prefill_chunk.cuh.
#include "gdn_prefill_chunk.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

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
// K1: intra-chunk quantities, one CTA (128 threads) per (chunk, v-head).
// =============================================================================================
constexpr int kIntraThreads = 128;
constexpr uint32_t kIntraTmemCols = 256;
// shared memory map (bytes from a 1024-aligned base)
constexpr uint32_t kI_QK = 0;          // 2 halves x [128 rows x 128 B]: rows 0-63 Q, 64-127 K
constexpr uint32_t kI_V = 32768;       // 2 halves x [64 x 128 B]
constexpr uint32_t kI_Tw = 49152;      // [64 r x 64 i] bf16, K-major SW128
constexpr uint32_t kI_Tu = 57344;      // T_u rounded to bf16 ...
constexpr uint32_t kI_TuLo = 65536;    // ... and the bf16 remainder (T_u = hi + lo to ~2^-17)
constexpr uint32_t kI_P = 73728;       // P image staging
constexpr uint32_t kI_AT = 81920;      // A transposed, fp32 [64 i][64 r]
constexpr uint32_t kI_End = 81920 + 16384;
constexpr uint32_t kIntraSmem = kI_End + 1024;   // + alignment slack

struct TensorMaps {
    CUtensorMap q, k, v;
};

__global__ void __launch_bounds__(kIntraThreads)
prefill_intra_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay) {
    const int c = blockIdx.x;
    const int hv = blockIdx.y;
    const int32_t total = *reinterpret_cast<const int32_t*>(ws);
    if (c >= total) return;
    const ChunkInfo ci = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks)[c];
    const int hqk = hv / (p.Hv / p.Hqk);
    uint8_t* rec = ws + lay.records + (static_cast<size_t>(c) * p.Hv + hv) * kRecBytes;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ uint64_t bar_tma, bar_mma;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ float s_g[kChunk], s_b[kChunk], s_beta[kChunk];

    const int tid = threadIdx.x, warp = tid >> 5;
    if (tid == 0) {
        mbar_init(&bar_tma, 1);
        mbar_init(&bar_mma, 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 0) {
        tmem_alloc(&tmem_base_s, kIntraTmemCols);
        tmem_relinquish();
    }
    if (tid < kChunk) {
        const bool valid = tid < ci.len;
        const size_t th = static_cast<size_t>(ci.t0 + (valid ? tid : 0)) * p.Hv + hv;
        s_g[tid] = valid ? p.g[th] : 0.f;
        s_beta[tid] = valid ? p.beta[th] : 0.f;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;

    if (tid == 0) {
        mbar_expect_tx(&bar_tma, 32768 + 16384);
        tma_load_2d(smem + kI_QK, &maps.q, hqk * kD, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 8192, &maps.k, hqk * kD, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 16384, &maps.q, hqk * kD + 64, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 24576, &maps.k, hqk * kD + 64, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_V, &maps.v, hv * kD, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_V + 8192, &maps.v, hv * kD + 64, ci.t0, &bar_tma);
    }
    if (tid < kChunk) {            // inclusive prefix sum of the log gates, in token order
        float acc = 0.f;
        for (int i = 0; i <= tid; ++i) acc += s_g[i];
        s_b[tid] = acc;
    }
    if (!mbar_wait(&bar_tma, 0)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) {
        if (tid == 0) report(p.dev_status, kDevTimeout);
        if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
        return;
    }
    tc_fence_after_sync();

    const uint32_t tG = tmem, tW = tmem + 64, tU = tmem + 128;
    const uint32_t sQK = smem_u32(smem + kI_QK);
    if (tid == 0) {
        // [Q;K] (128 x 128, K-major) times K^T: lanes 0-63 = q.k, lanes 64-127 = k.k
        const uint32_t idesc = make_idesc_bf16(128, 64, false, false);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint32_t off = (ks >> 2) * 16384 + (ks & 3) * 32;
            mma_ss(tG, make_sdesc_sw128(sQK + off, 16, 1024),
                   make_sdesc_sw128(sQK + 8192 + off, 16, 1024), idesc, ks > 0);
        }
        mma_commit(&bar_mma);
    }
    if (!mbar_wait(&bar_mma, 0)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) {
        if (tid == 0) report(p.dev_status, kDevTimeout);
        if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
        return;
    }
    tc_fence_after_sync();

    const uint32_t lane_base = static_cast<uint32_t>(warp * 32) << 16;
    float* sAT = reinterpret_cast<float*>(smem + kI_AT);
    {
        const int r = tid & 63;
        const float br = s_b[r];
        const float beta_r = s_beta[r];
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {
            uint32_t x[16];
            tmem_ld16(tG + lane_base + c0, x);
            tmem_wait_ld();
            if (tid < 64) {        // P row r -> bf16 image
                float pv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int i = c0 + j;
                    pv[j] = (i <= r) ? __expf(br - s_b[i]) * __uint_as_float(x[j]) : 0.f;
                }
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint4 w;
                    w.x = pack_bf16(pv[8 * h + 0], pv[8 * h + 1]);
                    w.y = pack_bf16(pv[8 * h + 2], pv[8 * h + 3]);
                    w.z = pack_bf16(pv[8 * h + 4], pv[8 * h + 5]);
                    w.w = pack_bf16(pv[8 * h + 6], pv[8 * h + 7]);
                    *reinterpret_cast<uint4*>(smem + kI_P + sw128_offset(r, (c0 >> 3) + h)) = w;
                }
            } else {               // A row r, stored transposed for the solve
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int i = c0 + j;
                    sAT[i * 64 + r] =
                        (i < r) ? beta_r * __expf(br - s_b[i]) * __uint_as_float(x[j]) : 0.f;
                }
            }
        }
    }
    __syncthreads();

    // T = (I + A)^{-1} by forward substitution; thread j owns column j of T.
    if (tid < 64) {
        const int j = tid;
        float t[64];
#pragma unroll
        for (int r = 0; r < 64; ++r) t[r] = (r == j) ? 1.f : 0.f;
#pragma unroll
        for (int i = 0; i < 63; ++i) {
            const float ti = t[i];
#pragma unroll
            for (int r4 = (i + 1) & ~3; r4 < 64; r4 += 4) {
                const float4 a = *reinterpret_cast<const float4*>(sAT + i * 64 + r4);
                if (r4 + 0 > i) t[r4 + 0] = fmaf(-a.x, ti, t[r4 + 0]);
                if (r4 + 1 > i) t[r4 + 1] = fmaf(-a.y, ti, t[r4 + 1]);
                if (r4 + 2 > i) t[r4 + 2] = fmaf(-a.z, ti, t[r4 + 2]);
                if (r4 + 3 > i) t[r4 + 3] = fmaf(-a.w, ti, t[r4 + 3]);
            }
        }
        const float bj = s_beta[j];
        const float bgj = bj * __expf(s_b[j]);
        const uint32_t col_off = ((j & 7) << 1);
#pragma unroll
        for (int r = 0; r < 64; ++r) {
            const uint32_t off = sw128_offset(r, j >> 3) + col_off;
            *reinterpret_cast<__nv_bfloat16*>(smem + kI_Tw + off) = __float2bfloat16(t[r] * bgj);
            const float tu = t[r] * bj;
            const __nv_bfloat16 tu_hi = __float2bfloat16(tu);
            *reinterpret_cast<__nv_bfloat16*>(smem + kI_Tu + off) = tu_hi;
            *reinterpret_cast<__nv_bfloat16*>(smem + kI_TuLo + off) =
                __float2bfloat16(tu - __bfloat162float(tu_hi));
        }
    }
    fence_proxy_async_smem();
    __syncthreads();

    if (tid == 0) {
        // W^T (dk x r) = K^T (MN-major A from the K tile) times T_w^T ; U~^T (dv x r) likewise from V
        const uint32_t idesc = make_idesc_bf16(128, 64, true, false);
        const uint32_t sTw = smem_u32(smem + kI_Tw), sTu = smem_u32(smem + kI_Tu);
        const uint32_t sTuLo = smem_u32(smem + kI_TuLo);
        const uint32_t sV = smem_u32(smem + kI_V);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            mma_ss(tW, make_sdesc_sw128(sQK + 8192 + ks * 2048, 16384, 1024),
                   make_sdesc_sw128(sTw + ks * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            mma_ss(tU, make_sdesc_sw128(sV + ks * 2048, 8192, 1024),
                   make_sdesc_sw128(sTu + ks * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            mma_ss(tU, make_sdesc_sw128(sV + ks * 2048, 8192, 1024),
                   make_sdesc_sw128(sTuLo + ks * 32, 16, 1024), idesc, true);
        mma_commit(&bar_mma);
    }
    if (!mbar_wait(&bar_mma, 1)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) {
        if (tid == 0) report(p.dev_status, kDevTimeout);
        if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
        return;
    }
    tc_fence_after_sync();

    {   // thread d (TMEM lane) holds W^T[d][0..63] and U~^T[d][0..63]
        const int d = tid;
        uint8_t* sW = smem + kI_QK;     // the Q/K tiles are dead now: stage the W image there
        const uint32_t wbase = (d >> 6) * 8192 + ((d & 7) << 1);
        const uint32_t wchunk = (d & 63) >> 3;
        float4* urec = reinterpret_cast<float4*>(rec + kRecU);
#pragma unroll
        for (int c0 = 0; c0 < 64; c0 += 16) {
            uint32_t x[16], y[16];
            tmem_ld16(tW + lane_base + c0, x);
            tmem_ld16(tU + lane_base + c0, y);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j)
                *reinterpret_cast<__nv_bfloat16*>(sW + wbase + sw128_offset(c0 + j, wchunk)) =
                    __float2bfloat16(__uint_as_float(x[j]));
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                urec[((c0 >> 2) + q4) * kD + d] =
                    make_float4(__uint_as_float(y[4 * q4]), __uint_as_float(y[4 * q4 + 1]),
                                __uint_as_float(y[4 * q4 + 2]), __uint_as_float(y[4 * q4 + 3]));
        }
        if (tid < kChunk) reinterpret_cast<float*>(rec + kRecB)[tid] = s_b[tid];
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        bulk_store(rec + kRecW, smem + kI_QK, 16384);
        bulk_store(rec + kRecP, smem + kI_P, 8192);
        bulk_commit();
        bulk_wait_read_all();
    }
    if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
}

// =============================================================================================
// K2: inter-chunk state pass, one CTA (256 threads) per (sequence, v-head).
// =============================================================================================
constexpr int kStateThreads = 256;
constexpr uint32_t kStateTmemCols = 512;
constexpr uint32_t kS_Rec = 0;                 // record image (57600 B, padded to 58368)
constexpr uint32_t kS_K = 58368;               // K tile, 2 halves [64 x 128 B]
constexpr uint32_t kS_Q = 58368 + 16384;       // Q tile
constexpr uint32_t kStageBytes = 58368 + 32768;                 // 91136
constexpr uint32_t kStateSmem = 2 * kStageBytes + 1024;
// TMEM columns
constexpr uint32_t kT_D1 = 0, kT_D2 = 64, kT_D3 = 128, kT_D4 = 192, kT_S = 320, kT_U = 384,
                   kT_Us = 416, kT_UsLo = 448;

__global__ void __launch_bounds__(kStateThreads, 1)
prefill_state_kernel(const __grid_constant__ TensorMaps maps, const PrefillParams p, uint8_t* ws,
                     const WorkspaceLayout lay) {
    const int n = blockIdx.x / p.Hv;
    const int hv = blockIdx.x - n * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int tid = threadIdx.x, warp = tid >> 5;
    const int half = warp >> 2;                       // which half of the columns this thread owns
    const int dv = (warp & 3) * 32 + (tid & 31);      // TMEM lane = state row
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;

    const int32_t* seq_first = reinterpret_cast<const int32_t*>(ws + lay.seq_first);
    const int32_t* seq_bad = reinterpret_cast<const int32_t*>(ws + lay.seq_bad);
    if (seq_bad[n]) return;
    const int c_first = seq_first[n];
    const int nc = seq_first[n + 1] - c_first;
    const ChunkInfo* chunks = reinterpret_cast<const ChunkInfo*>(ws + lay.chunks);

    const int slot = p.slot_idx ? p.slot_idx[n] : n;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && tid == 0) report(p.dev_status, kDevBadSlot);
        for (int j = 0; j < nc; ++j) {
            const ChunkInfo ci = chunks[c_first + j];
            for (int idx = tid; idx < ci.len * kD; idx += kStateThreads)
                p.o[(static_cast<size_t>(ci.t0 + idx / kD) * p.Hv + hv) * kD + (idx % kD)] =
                    __float2bfloat16(0.f);
        }
        return;
    }

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                               ~static_cast<uintptr_t>(1023));
    __shared__ uint64_t bar_full[2], bar_mma1, bar_mma2;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;

    // the thread's 64 state columns [64*half, 64*half+64) of row dv, fp32 master copy
    float S[64];
    const size_t tile_off = (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD) +
                            static_cast<size_t>(dv) * kD + half * 64;
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

    if (nc > 0) {
        if (tid == 0) {
            mbar_init(&bar_full[0], 1);
            mbar_init(&bar_full[1], 1);
            mbar_init(&bar_mma1, 1);
            mbar_init(&bar_mma2, 1);
            abort_flag = 0;
            fence_barrier_init();
        }
        if (warp == 0) {
            tmem_alloc(&tmem_base_s, kStateTmemCols);
            tmem_relinquish();
        }
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
        const uint32_t tmem = tmem_base_s;
        const uint8_t* records = ws + lay.records;

        auto issue_loads = [&](int j) {       // thread 0 only
            const int st = j & 1;
            const ChunkInfo ci = chunks[c_first + j];
            uint8_t* base = smem + st * kStageBytes;
            mbar_expect_tx(&bar_full[st], kRecBytes + 32768);
            bulk_load(base + kS_Rec,
                      records + (static_cast<size_t>(c_first + j) * p.Hv + hv) * kRecBytes, kRecBytes,
                      &bar_full[st]);
            tma_load_2d(base + kS_K, &maps.k, hqk * kD, ci.t0, &bar_full[st]);
            tma_load_2d(base + kS_K + 8192, &maps.k, hqk * kD + 64, ci.t0, &bar_full[st]);
            tma_load_2d(base + kS_Q, &maps.q, hqk * kD, ci.t0, &bar_full[st]);
            tma_load_2d(base + kS_Q + 8192, &maps.q, hqk * kD + 64, ci.t0, &bar_full[st]);
        };
        auto store_state_bf16 = [&]() {       // S (fp32 regs) -> bf16 A operand in TMEM
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(S[c0 + 2 * j], S[c0 + 2 * j + 1]);
                tmem_st16(tmem + kT_S + lane_base + half * 32 + (c0 >> 1), pk);
            }
        };

        if (tid == 0) issue_loads(0);
        store_state_bf16();
        tmem_wait_st();
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();

        bool ok = true;
        for (int j = 0; j < nc && ok; ++j) {
            const int st = j & 1;
            uint8_t* base = smem + st * kStageBytes;
            const ChunkInfo ci = chunks[c_first + j];
            if (tid == 0 && j + 1 < nc) issue_loads(j + 1);
            if (!mbar_wait(&bar_full[st], (j >> 1) & 1)) abort_flag = 1;
            __syncthreads();
            if (abort_flag) { ok = false; break; }
            tc_fence_after_sync();

            const uint32_t sRec = smem_u32(base + kS_Rec);
            const uint32_t sK = smem_u32(base + kS_K), sQ = smem_u32(base + kS_Q);
            if (tid == 0) {
                const uint32_t idesc = make_idesc_bf16(128, 64, false, false);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {       // D1 = S W^T
                    const uint32_t off = (ks >> 2) * 8192 + (ks & 3) * 32;
                    mma_ts(tmem + kT_D1, tmem + kT_S + ks * 8,
                           make_sdesc_sw128(sRec + kRecW + off, 16, 1024), idesc, ks > 0);
                }
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {       // D2 = S Q^T
                    const uint32_t off = (ks >> 2) * 8192 + (ks & 3) * 32;
                    mma_ts(tmem + kT_D2, tmem + kT_S + ks * 8, make_sdesc_sw128(sQ + off, 16, 1024),
                           idesc, ks > 0);
                }
                mma_commit(&bar_mma1);
            }
            if (!mbar_wait(&bar_mma1, j & 1)) abort_flag = 1;
            __syncthreads();
            if (abort_flag) { ok = false; break; }
            tc_fence_after_sync();

            const float* sb = reinterpret_cast<const float*>(base + kS_Rec + kRecB);
            const float bC = sb[kChunk - 1];
            {   // U^T[dv][c] = U~^T - D1 for the thread's 32 tokens [32*half, 32*half+32)
                const float4* sU = reinterpret_cast<const float4*>(base + kS_Rec + kRecU);
#pragma unroll
                for (int c0 = 0; c0 < 32; c0 += 16) {
                    const int cb = half * 32 + c0;
                    uint32_t x[16];
                    tmem_ld16(tmem + kT_D1 + lane_base + cb, x);
                    tmem_wait_ld();
                    float u[16];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const float4 ut = sU[((cb >> 2) + q4) * kD + dv];
                        u[4 * q4 + 0] = ut.x - __uint_as_float(x[4 * q4 + 0]);
                        u[4 * q4 + 1] = ut.y - __uint_as_float(x[4 * q4 + 1]);
                        u[4 * q4 + 2] = ut.z - __uint_as_float(x[4 * q4 + 2]);
                        u[4 * q4 + 3] = ut.w - __uint_as_float(x[4 * q4 + 3]);
                    }
                    // U for the output product; the decayed U for the state update is kept as
                    // hi + lo bf16 pairs so that its rounding does not limit the state's accuracy
                    uint32_t pu[8], ph[8], pl[8];
#pragma unroll
                    for (int jj = 0; jj < 8; ++jj) {
                        const float s0 = u[2 * jj] * __expf(bC - sb[cb + 2 * jj]);
                        const float s1 = u[2 * jj + 1] * __expf(bC - sb[cb + 2 * jj + 1]);
                        pu[jj] = pack_bf16(u[2 * jj], u[2 * jj + 1]);
                        ph[jj] = pack_bf16(s0, s1);
                        pl[jj] = pack_bf16(s0 - __uint_as_float(ph[jj] << 16),
                                           s1 - __uint_as_float(ph[jj] & 0xffff0000u));
                    }
                    tmem_st8(tmem + kT_U + lane_base + (cb >> 1), pu);
                    tmem_st8(tmem + kT_Us + lane_base + (cb >> 1), ph);
                    tmem_st8(tmem + kT_UsLo + lane_base + (cb >> 1), pl);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();

            if (tid == 0) {
                const uint32_t id3 = make_idesc_bf16(128, 64, false, false);
                const uint32_t id4 = make_idesc_bf16(128, 128, false, true);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)          // D3 = U P^T
                    mma_ts(tmem + kT_D3, tmem + kT_U + ks * 8,
                           make_sdesc_sw128(sRec + kRecP + ks * 32, 16, 1024), id3, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)          // D4 = (U decayed) K   (K tile MN-major)
                    mma_ts(tmem + kT_D4, tmem + kT_Us + ks * 8,
                           make_sdesc_sw128(sK + ks * 2048, 8192, 1024), id4, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    mma_ts(tmem + kT_D4, tmem + kT_UsLo + ks * 8,
                           make_sdesc_sw128(sK + ks * 2048, 8192, 1024), id4, true);
                mma_commit(&bar_mma2);
            }
            if (!mbar_wait(&bar_mma2, j & 1)) abort_flag = 1;
            __syncthreads();
            if (abort_flag) { ok = false; break; }
            tc_fence_after_sync();

            {   // S <- e^{b_C} S + D4 on the thread's 64 dk columns; refresh the bf16 copy
                const float gC = __expf(bC);
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 16) {
                    uint32_t x[16];
                    tmem_ld16(tmem + kT_D4 + lane_base + half * 64 + c0, x);
                    tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj)
                        S[c0 + jj] = fmaf(gC, S[c0 + jj], __uint_as_float(x[jj]));
                }
                store_state_bf16();
            }
            {   // o[t0+c][hv][dv] = scale (e^{b_c} D2 + D3) for the thread's 32 tokens
                __nv_bfloat16* op = p.o + (static_cast<size_t>(ci.t0) * p.Hv + hv) * kD + dv;
                const size_t tok_stride = static_cast<size_t>(p.Hv) * kD;
#pragma unroll
                for (int c0 = 0; c0 < 32; c0 += 16) {
                    const int cb = half * 32 + c0;
                    uint32_t x[16], y[16];
                    tmem_ld16(tmem + kT_D2 + lane_base + cb, x);
                    tmem_ld16(tmem + kT_D3 + lane_base + cb, y);
                    tmem_wait_ld();
#pragma unroll
                    for (int jj = 0; jj < 16; ++jj) {
                        const int cc = cb + jj;
                        if (cc < ci.len)
                            op[cc * tok_stride] = __float2bfloat16(
                                p.scale * fmaf(__expf(sb[cc]), __uint_as_float(x[jj]),
                                               __uint_as_float(y[jj])));
                    }
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncthreads();
            tc_fence_after_sync();
        }
        if (!ok) {
            if (tid == 0) report(p.dev_status, kDevTimeout);
            // let copies already in flight land before the CTA's shared memory goes away
            mbar_wait(&bar_full[0], 0, 1u << 12);
            mbar_wait(&bar_full[1], 0, 1u << 12);
        }
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, kStateTmemCols);
        if (!ok) return;
    }

#pragma unroll
    for (int j = 0; j < 64; j += 4)
        *reinterpret_cast<float4*>(p.final_state + tile_off + j) =
            make_float4(S[j], S[j + 1], S[j + 2], S[j + 3]);
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

cudaError_t launch_prefill_chunked(const ChunkedParams& cp, cudaStream_t stream) {
    const PrefillParams& p = cp.p;
    cudaError_t e = cudaFuncSetAttribute(prefill_intra_kernel,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, kIntraSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(prefill_state_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kStateSmem);
    if (e != cudaSuccess) return e;
    TensorMaps maps;
    if (!make_token_map(&maps.q, p.q, p.T, static_cast<int64_t>(p.Hqk) * kD) ||
        !make_token_map(&maps.k, p.k, p.T, static_cast<int64_t>(p.Hqk) * kD) ||
        !make_token_map(&maps.v, p.v, p.T, static_cast<int64_t>(p.Hv) * kD))
        return cudaErrorInvalidValue;

    prefill_prep_kernel<<<1, kPrepThreads, 0, stream>>>(p.cu_seqlens, p.T, p.N, cp.ws, cp.lay,
                                                        p.dev_status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (cp.lay.max_chunks > 0) {
        dim3 grid(cp.lay.max_chunks, p.Hv);
        prefill_intra_kernel<<<grid, kIntraThreads, kIntraSmem, stream>>>(maps, p, cp.ws, cp.lay);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    prefill_state_kernel<<<p.N * p.Hv, kStateThreads, kStateSmem, stream>>>(maps, p, cp.ws, cp.lay);
    return cudaGetLastError();
}

}  // namespace gdn
