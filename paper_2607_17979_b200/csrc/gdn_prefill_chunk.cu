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
// K1: intra-chunk quantities, one CTA (256 threads) per (chunk, v-head).
// =============================================================================================
constexpr int kIntraThreads = 256;
constexpr uint32_t kIntraTmemCols = 128;
constexpr int kLdA = 68;               // row stride (floats) of the fp32 A / T matrix
// Shared memory map (bytes from a 1024-aligned base).  Regions are reused as their contents die
// so that three CTAs fit on an SM:
//   R1  Q/K tiles.  Q halves -> Qg image (stored early) -> T_w and T_u(hi);  K halves -> W image.
//   R2  A, then T, in fp32 plus the solve scratch -> V tile (loaded after the solve).
//   R3  P image (stored early) -> T_u(lo).
constexpr uint32_t kI_QK = 0;          // 2 halves x [128 rows x 128 B]: rows 0-63 Q, 64-127 K
constexpr uint32_t kI_Tw = 0;          // over Q half 0: T diag(beta e^b) [64 r x 64 i] bf16, K-major
constexpr uint32_t kI_Tu = 16384;      // over Q half 1: T diag(beta) rounded to bf16 ...
constexpr uint32_t kI_A = 32768;       // A, then T in place: fp32 [64][kLdA]
constexpr uint32_t kI_Scr = kI_A + 64 * kLdA * 4;      // solve scratch, fp32 [32][40]
constexpr uint32_t kI_V = 32768;       // over A: 2 halves x [64 x 128 B]
constexpr uint32_t kI_P = 32768 + 22528;               // P image staging
constexpr uint32_t kI_TuLo = kI_P;     // ... and the bf16 remainder of T diag(beta)
constexpr uint32_t kI_End = kI_P + 8192;
constexpr uint32_t kIntraSmem = kI_End + 1024;         // + alignment slack
static_assert(kI_Scr + 32 * 40 * 4 <= kI_P, "solve scratch overlaps the P image");

struct TensorMaps {
    CUtensorMap q, k, v;
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One 16x8 output tile  C += A[16 x 8*ksteps] * B[8*ksteps x 8]  on mma.sync m16n8k8 with both
// operands split into tf32 hi + lo parts (three products; the lo*lo term is dropped), which keeps
// fp32-level accuracy.  A, B: fp32 row-major in shared memory; g = lane / 4, t = lane % 4.
__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
    const float rem = x - __uint_as_float(hi);
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(rem));
}
__device__ __forceinline__ void mma_m16n8k8_tf32(float (&c)[4], const uint32_t (&a)[4],
                                                 const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ void mma_tile_tf32x3(const float* A, int lda, const float* B, int ldb,
                                                int ksteps, float (&c)[4], int g, int t) {
    float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};   // separate dependency chains
#pragma unroll 4
    for (int ks = 0; ks < ksteps; ++ks) {
        const float* a_ = A + 8 * ks;
        const float* b_ = B + (8 * ks) * ldb;
        const float af[4] = {a_[g * lda + t], a_[(g + 8) * lda + t], a_[g * lda + t + 4],
                             a_[(g + 8) * lda + t + 4]};
        const float bf[2] = {b_[t * ldb + g], b_[(t + 4) * ldb + g]};
        uint32_t ah[4], al[4], bh[2], bl[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) split_tf32(af[i], ah[i], al[i]);
#pragma unroll
        for (int i = 0; i < 2; ++i) split_tf32(bf[i], bh[i], bl[i]);
        mma_m16n8k8_tf32(c1, al, bh);
        mma_m16n8k8_tf32(c2, ah, bl);
        mma_m16n8k8_tf32(c, ah, bh);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] += c1[i] + c2[i];
}

// T = (I + A)^{-1} for the strictly lower-triangular 64x64 A in sA (row-major, stride kLdA),
// in place, by 256 threads: four 16x16 diagonal blocks by forward substitution in fp32, then the
// off-diagonal blocks by block elimination at block sizes 16 and 32
//     [[Ta, 0], [X, Tb]],  X = -Tb (A_ba Ta),
// whose small products run on the legacy mma.sync path with split-tf32 operands (fp32-level
// accuracy; tcgen05 needs M >= 64).  Ends with a __syncthreads().
__device__ __forceinline__ void solve_unit_lower_64(float* sA, float* scr, int tid) {
    // ---- diagonal blocks: thread (I, j) computes column j of (I + A_II)^{-1}, right-looking
    if (tid < 64) {
        const int I = tid >> 4, j = tid & 15;
        float* blk = sA + (16 * I) * kLdA + 16 * I;
        float t[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) t[r] = (r == j) ? 1.f : 0.f;
#pragma unroll
        for (int i = 0; i < 15; ++i) {
            const float ti = t[i];
#pragma unroll
            for (int r = i + 1; r < 16; ++r) t[r] = fmaf(-blk[r * kLdA + i], ti, t[r]);
        }
        __syncwarp();                      // every column of the block has read A_II
#pragma unroll
        for (int r = 0; r < 16; ++r) blk[r * kLdA + j] = t[r];
    }
    __syncthreads();
    // ---- off-diagonal blocks on the tensor cores (mma.sync m16n8k8, 3xTF32: fp32-level accuracy)
    const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    // 16-blocks (1,0) and (3,2): X = A_IJ T_JJ, then T_IJ = -T_II X.  Four 16x8 tiles, warps 0-3.
    {
        const int pr = warp >> 1, nb = warp & 1;            // pair, 8-column block
        const int I = 2 * pr + 1, J = 2 * pr;
        float* X = scr + pr * (16 * 24);
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        if (warp < 4) {
            mma_tile_tf32x3(sA + (16 * I) * kLdA + 16 * J, kLdA, sA + (16 * J) * kLdA + 16 * J + 8 * nb,
                            kLdA, 2, c, g, t);
            *reinterpret_cast<float2*>(X + g * 24 + 8 * nb + 2 * t) = make_float2(c[0], c[1]);
            *reinterpret_cast<float2*>(X + (g + 8) * 24 + 8 * nb + 2 * t) = make_float2(c[2], c[3]);
        }
        __syncthreads();
        if (warp < 4) {
            c[0] = c[1] = c[2] = c[3] = 0.f;
            mma_tile_tf32x3(sA + (16 * I) * kLdA + 16 * I, kLdA, X + 8 * nb, 24, 2, c, g, t);
            float* dst = sA + (16 * I) * kLdA + 16 * J + 8 * nb;
            *reinterpret_cast<float2*>(dst + g * kLdA + 2 * t) = make_float2(-c[0], -c[1]);
            *reinterpret_cast<float2*>(dst + (g + 8) * kLdA + 2 * t) = make_float2(-c[2], -c[3]);
        }
    }
    __syncthreads();
    // 32-block (1,0): Y = A_ba Ta, then X = -Tb Y.  Eight 16x8 tiles, one per warp.
    {
        const int mr = warp >> 2, nb = warp & 3;
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        mma_tile_tf32x3(sA + (32 + 16 * mr) * kLdA, kLdA, sA + 8 * nb, kLdA, 4, c, g, t);
        *reinterpret_cast<float2*>(scr + (16 * mr + g) * 40 + 8 * nb + 2 * t) = make_float2(c[0], c[1]);
        *reinterpret_cast<float2*>(scr + (16 * mr + g + 8) * 40 + 8 * nb + 2 * t) = make_float2(c[2], c[3]);
        __syncthreads();
        c[0] = c[1] = c[2] = c[3] = 0.f;
        mma_tile_tf32x3(sA + (32 + 16 * mr) * kLdA + 32, kLdA, scr + 8 * nb, 40, 4, c, g, t);
        float* dst = sA + (32 + 16 * mr) * kLdA + 8 * nb;
        *reinterpret_cast<float2*>(dst + g * kLdA + 2 * t) = make_float2(-c[0], -c[1]);
        *reinterpret_cast<float2*>(dst + (g + 8) * kLdA + 2 * t) = make_float2(-c[2], -c[3]);
    }
    __syncthreads();
}

// Lane 0 polls the mbarrier (bounded), the other lanes block at the warp barrier instead of
// competing for issue slots; returns the same verdict on every lane.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t packed, float f) {
    return pack_bf16(__uint_as_float(packed << 16) * f, __uint_as_float(packed & 0xffff0000u) * f);
}

__global__ void __launch_bounds__(kIntraThreads, 3)
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
    __shared__ uint64_t bar_tma, bar_v, bar_mma;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_flag;
    __shared__ __align__(16) float s_b2[kChunk];     // b_r log2(e): inclusive log-decay prefix
    __shared__ __align__(16) float s_beta[kChunk];   // beta_r (0 past the chunk's length)
    __shared__ __align__(16) float s_bg[kChunk];     // beta_r e^{b_r}
    __shared__ __align__(16) float s_eb[kChunk];     // e^{b_r}

    const int tid = threadIdx.x, warp = tid >> 5;
    const int colhalf = warp >> 2;                   // which 32 of the 64 accumulator columns
    if (tid == 0) {
        mbar_init(&bar_tma, 1);
        mbar_init(&bar_v, 1);
        mbar_init(&bar_mma, 1);
        abort_flag = 0;
        fence_barrier_init();
        // Q and K first: everything below overlaps their flight (V comes later, over dead data)
        mbar_expect_tx(&bar_tma, 32768);
        tma_load_2d(smem + kI_QK, &maps.q, hqk * kD, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 8192, &maps.k, hqk * kD, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 16384, &maps.q, hqk * kD + 64, ci.t0, &bar_tma);
        tma_load_2d(smem + kI_QK + 24576, &maps.k, hqk * kD + 64, ci.t0, &bar_tma);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(&tmem_base_s, kIntraTmemCols);
        tmem_relinquish();
    }
    if (warp == 1) {
        // inclusive prefix sum of the log gates over the chunk (two tokens per lane); rows past
        // the chunk's length get g = 0, beta = 0 and so change nothing downstream
        const int lane = tid & 31;
        float g0 = 0.f, g1 = 0.f, be0 = 0.f, be1 = 0.f;
        if (2 * lane < ci.len) {
            const size_t th = static_cast<size_t>(ci.t0 + 2 * lane) * p.Hv + hv;
            g0 = p.g[th]; be0 = p.beta[th];
        }
        if (2 * lane + 1 < ci.len) {
            const size_t th = static_cast<size_t>(ci.t0 + 2 * lane + 1) * p.Hv + hv;
            g1 = p.g[th]; be1 = p.beta[th];
        }
        float incl = g0 + g1;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const float y = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += y;
        }
        const float kLog2e = 1.4426950408889634f;
        const float b1 = incl, b0 = incl - g1;
        const float bC = __shfl_sync(0xffffffffu, incl, 31);
        s_b2[2 * lane] = b0 * kLog2e; s_b2[2 * lane + 1] = b1 * kLog2e;
        s_beta[2 * lane] = be0; s_beta[2 * lane + 1] = be1;
        const float e0 = ex2_approx(b0 * kLog2e), e1 = ex2_approx(b1 * kLog2e);
        s_eb[2 * lane] = e0; s_eb[2 * lane + 1] = e1;
        s_bg[2 * lane] = be0 * e0; s_bg[2 * lane + 1] = be1 * e1;
        // decay vector of the record: e^{b_C - b_c}, then e^{b_C}
        float* dec = reinterpret_cast<float*>(rec + kRecDecay);
        dec[2 * lane] = ex2_approx((bC - b0) * kLog2e);
        dec[2 * lane + 1] = ex2_approx((bC - b1) * kLog2e);
        if (lane == 0) dec[kChunk] = ex2_approx(bC * kLog2e);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_base_s;
    // On a timeout: flag it, let thread 0 drain what it has in flight, free TMEM, leave.
    auto bail = [&](bool stores_pending) {
        if (tid == 0) {
            report(p.dev_status, kDevTimeout);
            if (stores_pending) bulk_wait_read_all();
        }
        if (warp == 0) tmem_dealloc(tmem, kIntraTmemCols);
    };

    if (warp == 0 && !warp_wait(&bar_tma, 0)) abort_flag = 1;      // one warp polls, the rest block
    __syncthreads();
    if (abort_flag) { bail(false); return; }
    tc_fence_after_sync();

    const uint32_t tG = tmem, tW = tmem, tU = tmem + 64;     // W reuses the Gram columns
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
    if (warp == 0 && !warp_wait(&bar_mma, 0)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) { bail(false); return; }
    tc_fence_after_sync();

    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    float* sA = reinterpret_cast<float*>(smem + kI_A);
    {
        // Accumulator row of this thread: TMEM lane 32 (warp % 4) + lane; lanes 0-63 hold q.k
        // rows (-> P), lanes 64-127 hold k.k rows (-> A).  The thread covers 32 of the 64 columns,
        // 16 at a time.
        const int row = (warp & 3) * 32 + (tid & 31);
        const int r = row & 63;
        const bool is_p = row < 64;
        const float br2 = s_b2[r];
        const float rowscale = is_p ? 1.f : s_beta[r];
        const int limit = is_p ? r : r - 1;              // keep columns i <= limit
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cbase = colhalf * 32 + step * 16;
            uint32_t x[16];
            tmem_ld16(tG + lane_base + cbase, x);
            tmem_wait_ld();
            float val[16];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                const float4 bb = *reinterpret_cast<const float4*>(s_b2 + cbase + 4 * q4);
                const float bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int jj = 4 * q4 + e;
                    const bool keep = cbase + jj <= limit;
                    const float dec = ex2_approx(keep ? br2 - bv[e] : 0.f);   // e^{b_r - b_i}
                    val[jj] = keep ? rowscale * dec * __uint_as_float(x[jj]) : 0.f;
                }
            }
            if (is_p) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    uint4 w;
                    w.x = pack_bf16(val[8 * h + 0], val[8 * h + 1]);
                    w.y = pack_bf16(val[8 * h + 2], val[8 * h + 3]);
                    w.z = pack_bf16(val[8 * h + 4], val[8 * h + 5]);
                    w.w = pack_bf16(val[8 * h + 6], val[8 * h + 7]);
                    *reinterpret_cast<uint4*>(smem + kI_P + sw128_offset(r, (cbase >> 3) + h)) = w;
                }
            } else {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<float4*>(sA + r * kLdA + cbase + 4 * q4) =
                        make_float4(val[4 * q4], val[4 * q4 + 1], val[4 * q4 + 2], val[4 * q4 + 3]);
            }
        }
    }
    {   // Q rows scaled by e^{b_r}, in place (the Gram product has consumed Q): this is the Qg image
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const int idx = tid + it * kIntraThreads;          // 1024 16-byte pieces
            const int halfq = idx >> 9, rem = idx & 511;
            const int r = rem >> 3;
            uint4* ptr = reinterpret_cast<uint4*>(smem + kI_QK + halfq * 16384 + rem * 16);
            const float f = s_eb[r];
            uint4 w = *ptr;
            w.x = scale_bf16x2(w.x, f); w.y = scale_bf16x2(w.y, f);
            w.z = scale_bf16x2(w.z, f); w.w = scale_bf16x2(w.w, f);
            *ptr = w;
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        // Qg and P are final: store them now; their shared memory is reused after the solve
        bulk_store(rec + kRecQg, smem + kI_QK, 8192);
        bulk_store(rec + kRecQg + 8192, smem + kI_QK + 16384, 8192);
        bulk_store(rec + kRecP, smem + kI_P, 8192);
        bulk_commit();
    }

    solve_unit_lower_64(sA, reinterpret_cast<float*>(smem + kI_Scr), tid);

    if (tid == 0) bulk_wait_read_all();      // the Q halves and the P image have been read out
    __syncthreads();

    {   // T (fp32, row-major) -> bf16 B operands T diag(beta e^b), T diag(beta) (hi, lo)
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int idx = tid + it * kIntraThreads;          // 512 pieces of 8 columns
            const int r = idx >> 3, c8 = idx & 7;
            const float4 t0 = *reinterpret_cast<const float4*>(sA + r * kLdA + 8 * c8);
            const float4 t1 = *reinterpret_cast<const float4*>(sA + r * kLdA + 8 * c8 + 4);
            const float4 g0 = *reinterpret_cast<const float4*>(s_bg + 8 * c8);
            const float4 g1 = *reinterpret_cast<const float4*>(s_bg + 8 * c8 + 4);
            const float4 e0 = *reinterpret_cast<const float4*>(s_beta + 8 * c8);
            const float4 e1 = *reinterpret_cast<const float4*>(s_beta + 8 * c8 + 4);
            const float tv[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const float ev[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};
            uint32_t w[4], hi[4], lo[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                w[j] = pack_bf16(tv[2 * j] * gv[2 * j], tv[2 * j + 1] * gv[2 * j + 1]);
                const float u0 = tv[2 * j] * ev[2 * j], u1 = tv[2 * j + 1] * ev[2 * j + 1];
                hi[j] = pack_bf16(u0, u1);
                lo[j] = pack_bf16(u0 - __uint_as_float(hi[j] << 16),
                                  u1 - __uint_as_float(hi[j] & 0xffff0000u));
            }
            const uint32_t off = sw128_offset(r, c8);
            *reinterpret_cast<uint4*>(smem + kI_Tw + off) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(smem + kI_Tu + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(smem + kI_TuLo + off) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
    }
    fence_proxy_async_smem();
    __syncthreads();

    const uint32_t sV = smem_u32(smem + kI_V);
    if (tid == 0) {
        // V into the space the solve has left; meanwhile W^T (dk x r) = K^T T_w^T with the raw K
        // tile read MN-major
        mbar_expect_tx(&bar_v, 16384);
        tma_load_2d(smem + kI_V, &maps.v, hv * kD, ci.t0, &bar_v);
        tma_load_2d(smem + kI_V + 8192, &maps.v, hv * kD + 64, ci.t0, &bar_v);
        const uint32_t idesc = make_idesc_bf16(128, 64, true, false);
        const uint32_t sTw = smem_u32(smem + kI_Tw);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            mma_ss(tW, make_sdesc_sw128(sQK + 8192 + ks * 2048, 16384, 1024),
                   make_sdesc_sw128(sTw + ks * 32, 16, 1024), idesc, ks > 0);
        mma_commit(&bar_mma);
    }
    if (warp == 0 && !warp_wait(&bar_mma, 1)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) { bail(false); return; }      // nothing of thread 0's stores is pending here
    tc_fence_after_sync();

    const int d = (warp & 3) * 32 + (tid & 31);   // TMEM lane of this thread: a dk / dv index
    {   // W^T[d][32 tokens] -> bf16 -> W image staged over the (now dead) K halves
        uint8_t* sW = smem + kI_QK + 8192 + (d >> 6) * 16384;
        const uint32_t wcol = ((d & 7) << 1);
        const uint32_t wchunk = (d & 63) >> 3;
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cbase = colhalf * 32 + step * 16;
            uint32_t x[16];
            tmem_ld16(tW + lane_base + cbase, x);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j)
                *reinterpret_cast<__nv_bfloat16*>(sW + sw128_offset(cbase + j, wchunk) + wcol) =
                    __float2bfloat16(__uint_as_float(x[j]));
        }
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    if (warp == 0 && !warp_wait(&bar_v, 0)) abort_flag = 1;        // V has landed
    __syncthreads();
    if (abort_flag) { bail(false); return; }
    tc_fence_after_sync();
    if (tid == 0) {
        bulk_store(rec + kRecW, smem + kI_QK + 8192, 8192);
        bulk_store(rec + kRecW + 8192, smem + kI_QK + 24576, 8192);
        bulk_commit();
        // U~^T (dv x r) = V^T T_u^T with T_u = hi + lo
        const uint32_t idesc = make_idesc_bf16(128, 64, true, false);
        const uint32_t sTu = smem_u32(smem + kI_Tu), sTuLo = smem_u32(smem + kI_TuLo);
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
    if (warp == 0 && !warp_wait(&bar_mma, 0)) abort_flag = 1;
    __syncthreads();
    if (abort_flag) { bail(true); return; }
    tc_fence_after_sync();

    {   // U~^T[d][32 tokens] -> record, [token group][dv][4 tokens] fp32
        float4* urec = reinterpret_cast<float4*>(rec + kRecU);
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cbase = colhalf * 32 + step * 16;
            uint32_t y[16];
            tmem_ld16(tU + lane_base + cbase, y);
            tmem_wait_ld();
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                urec[((cbase >> 2) + q4) * kD + d] =
                    make_float4(__uint_as_float(y[4 * q4]), __uint_as_float(y[4 * q4 + 1]),
                                __uint_as_float(y[4 * q4 + 2]), __uint_as_float(y[4 * q4 + 3]));
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) bulk_wait_read_all();
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
constexpr int kStateEpiWarps = 8;
constexpr int kStateEpiThreads = kStateEpiWarps * 32;
constexpr int kStateThreads = kStateEpiThreads + 32;
constexpr uint32_t kStateTmemCols = 512;
constexpr uint32_t kS_Rec = 0;                 // record image (74240 B, padded to 74752)
constexpr uint32_t kS_K = 74752;               // K tile, 2 halves [64 x 128 B]
constexpr uint32_t kStageBytes = 74752 + 16384;                 // 91136
constexpr uint32_t kS_Out = 2 * kStageBytes;   // o staging [64 tokens][128 dv] bf16
constexpr uint32_t kStateSmem = 2 * kStageBytes + 16384 + 1024;
// TMEM columns
constexpr uint32_t kT_D1 = 0, kT_Y = 64 /* two tiles of 64 */, kT_D4 = 192, kT_S = 320, kT_U = 384,
                   kT_Us = 416, kT_UsLo = 448;

// bounded wait that also gives up as soon as another role has flagged an abort
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

// Same, for a whole warp: lane 0 polls, every lane gets the verdict.
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = wait_or_abort(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__device__ __forceinline__ void epi_group_sync() {      // the 256 epilogue threads only
    asm volatile("bar.sync 1, %0;" ::"n"(kStateEpiThreads) : "memory");
}

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
                // base descriptors of both stages, built once; the loop only adds offsets
                const uint32_t sRec0 = smem_u32(smem + kS_Rec), sRec1 = sRec0 + kStageBytes;
                const uint64_t dW0 = make_sdesc_sw128(sRec0 + kRecW, 16, 1024);
                const uint64_t dQ0 = make_sdesc_sw128(sRec0 + kRecQg, 16, 1024);
                const uint64_t dP0 = make_sdesc_sw128(sRec0 + kRecP, 16, 1024);
                const uint64_t dK0 = make_sdesc_sw128(sRec0 + kS_K, 8192, 1024);
                const uint64_t dW1 = make_sdesc_sw128(sRec1 + kRecW, 16, 1024);
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
                    // D1 = S W^T  (on the chain); k-step ks reads 16 dk: 32 bytes inside a half
                    mma_ts_c<false>(tD1, tS, w, id64);
                    mma_ts_c<true>(tD1, tS + 8, sdesc_advance(w, 32), id64);
                    mma_ts_c<true>(tD1, tS + 16, sdesc_advance(w, 64), id64);
                    mma_ts_c<true>(tD1, tS + 24, sdesc_advance(w, 96), id64);
                    mma_ts_c<true>(tD1, tS + 32, sdesc_advance(w, 8192), id64);
                    mma_ts_c<true>(tD1, tS + 40, sdesc_advance(w, 8192 + 32), id64);
                    mma_ts_c<true>(tD1, tS + 48, sdesc_advance(w, 8192 + 64), id64);
                    mma_ts_c<true>(tD1, tS + 56, sdesc_advance(w, 8192 + 96), id64);
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
                    sO[(half * 32 + jj) * kD + dv] = __float2bfloat16(p.scale * __uint_as_float(x[jj]));
                    sO[(half * 32 + 16 + jj) * kD + dv] = __float2bfloat16(p.scale * __uint_as_float(y[jj]));
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
            for (int j = 0; j < nc; ++j) {
                const int st = j & 1;
                const uint8_t* base = smem + st * kStageBytes;
                if (j > 0) {     // part A of the previous chunk's outputs, while D1 is in flight
                    if (!warp_wait_or_abort(&bar_y, (j - 1) & 1, abortp)) { ok = false; break; }
                    tc_fence_after_sync();
                    epi_group_sync();
                    outputs_stage(j - 1);
                }
                if (!warp_wait_or_abort(&bar_full[st], (j >> 1) & 1, abortp)) { ok = false; break; }
                if (!warp_wait_or_abort(&bar_d1, j & 1, abortp)) { ok = false; break; }
                tc_fence_after_sync();

                const float* sdec = reinterpret_cast<const float*>(base + kS_Rec + kRecDecay);
                {   // U^T[dv][c] = U~^T - D1 for the thread's 32 tokens [32*half, 32*half+32)
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
                    outputs_flush(j - 1);
                }

                if (!warp_wait_or_abort(&bar_d4, j & 1, abortp)) { ok = false; break; }
                tc_fence_after_sync();
                {   // S <- e^{b_C} S + D4 on the thread's 64 dk columns; refresh the bf16 copy
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
            if (ok) {
                if (warp_wait_or_abort(&bar_y, (nc - 1) & 1, abortp)) {
                    tc_fence_after_sync();
                    epi_group_sync();
                    outputs_stage(nc - 1);
                    epi_group_sync();
                    outputs_flush(nc - 1);
                }
            }
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
