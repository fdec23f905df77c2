// Device-side building blocks shared by the chunked prefill kernels (the three-launch path and
// the fused single-launch path): shared-memory maps, the fp32 triangular solve, the intra-chunk
// item routine, and the bounded-wait helpers.  See gdn_prefill_chunk.cuh for the algebra.
#pragma once
#include "gdn_prefill_chunk.cuh"
#include "gdn_sm100.cuh"

namespace gdn {
using namespace sm100;

constexpr int kIntraThreads = 256;
constexpr uint32_t kIntraTmemCols = 128;    // the Gram accumulator, then W^T in the same columns; U~^T
constexpr int kLdA = 68;               // row stride (floats) of the fp32 A / T matrix
// Shared memory map (bytes from a 1024-aligned base).  Regions are reused as their contents die
// so that four CTAs fit on an SM:
//   R1  Q/K tiles.  Q half 0 -> Qg image (stored early) -> T_w -> T_u(lo);
//       Q half 1 -> Qg image -> T_u(hi);  K halves -> W image.
//   R2  A, then T, in fp32 -> V tile (loaded after the solve).
// The P image goes straight from registers to the record; T_u(lo) waits in registers until the
// product that reads T_w has retired.
constexpr uint32_t kI_QK = 0;          // 2 halves x [128 rows x 128 B]: rows 0-63 Q, 64-127 K
constexpr uint32_t kI_Tw = 0;          // over Q half 0: T diag(beta e^b) [64 r x 64 i] bf16, K-major
constexpr uint32_t kI_TuLo = 0;        // ... and later the bf16 remainder of T diag(beta)
constexpr uint32_t kI_Tu = 16384;      // over Q half 1: T diag(beta) rounded to bf16
constexpr uint32_t kI_A = 32768;       // A, then T in place: fp32 [64][kLdA]
constexpr uint32_t kI_V = 32768;       // over A: 2 halves x [64 x 128 B]
constexpr uint32_t kI_End = kI_A + 64 * kLdA * 4;      // 50176
constexpr uint32_t kIntraSmem = kI_End + 1024;         // + alignment slack
static_assert(kI_End % 1024 == 0 && 64 * kLdA * 4 >= 16384, "V tile must fit over A");

struct TensorMaps {
    CUtensorMap q, k, v;
};
// Host side: 2-D maps over the packed q, k, v (64 x 64 boxes, 128B swizzle); false on failure.
bool make_prefill_tensor_maps(TensorMaps* maps, const PrefillParams& p);
// Launch of the intra-chunk kernel over every (chunk, v-head) item of the batch.
// inline_tables: no table-building launch went before; every CTA finds its chunk from cu_seqlens and
// one CTA writes the per-sequence tables (first chunk, validity, rank) for the state pass.  Only
// for batches of few sequences: see prefill_tables_inline().
cudaError_t launch_prefill_intra(const TensorMaps& maps, const ChunkedParams& cp, cudaStream_t stream,
                                 bool inline_tables);
bool prefill_tables_inline(const ChunkedParams& cp);

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// One 16x8 output tile  C += A[16 x 8*ksteps] * B[8*ksteps x 8]  on mma.sync m16n8k8 with tf32
// operands (rounded to nearest, one product per k-step) and fp32 accumulation.  A, B: fp32
// row-major in shared memory; g = lane / 4, t = lane % 4.
// Accuracy: these products only form the OFF-diagonal blocks of T = (I + A)^-1 from blocks that
// are exact to fp32; an operand error of 2^-11 there moves the final state by about 1e-5 of its
// norm on random keys and 3e-4 when all keys coincide (the worst case for the solve), against
// 1.6e-4 and 1.4e-3 from the bf16 operands of the other products.  Split operands (three
// products per k-step) bought nothing measurable and cost 2.3x the instructions.
__device__ __forceinline__ uint32_t to_tf32(float x) {
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ void mma_m16n8k8_tf32(float (&c)[4], const uint32_t (&a)[4],
                                                 const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
template <int kSteps>
__device__ __forceinline__ void mma_tile_tf32(const float* A, int lda, const float* B, int ldb,
                                              float (&c)[4], int g, int t) {
    uint32_t a[kSteps][4], b[kSteps][2];
#pragma unroll
    for (int ks = 0; ks < kSteps; ++ks) {          // every load first, then the products
        const float* a_ = A + 8 * ks;
        const float* b_ = B + (8 * ks) * ldb;
        a[ks][0] = to_tf32(a_[g * lda + t]);
        a[ks][1] = to_tf32(a_[(g + 8) * lda + t]);
        a[ks][2] = to_tf32(a_[g * lda + t + 4]);
        a[ks][3] = to_tf32(a_[(g + 8) * lda + t + 4]);
        b[ks][0] = to_tf32(b_[t * ldb + g]);
        b[ks][1] = to_tf32(b_[(t + 4) * ldb + g]);
    }
#pragma unroll
    for (int ks = 0; ks < kSteps; ++ks) mma_m16n8k8_tf32(c, a[ks], b[ks]);
}

__device__ __forceinline__ uint32_t scale_bf16x2(uint32_t packed, float f) {
    return pack_bf16(__uint_as_float(packed << 16) * f, __uint_as_float(packed & 0xffff0000u) * f);
}

// Per-group statics of the intra-chunk work (one instance per concurrently processed item).
struct IntraStatics {
    uint64_t bar_tma, bar_v, bar_mma;
    int abort_flag;
    int item;                          // work-queue slot (persistent variant)
    alignas(16) float s_b2[kChunk];    // b_r log2(e): inclusive log-decay prefix
    alignas(16) float s_beta[kChunk];  // beta_r (0 past the chunk's length)
    alignas(16) float s_bg[kChunk];    // beta_r e^{b_r}
    alignas(16) float s_eb[kChunk];    // e^{b_r}
};

// T = (I + A)^{-1} for the strictly lower-triangular 64x64 A in sA (fp32, row-major, stride kLdA),
// in place, in two warp-local stages that need no barrier wider than a warp:
//   solve_blocks_16_32: a warp inverts two neighbouring diagonal 16x16 blocks by forward
//     substitution (thread (I, j) computes column j of (I + A_II)^{-1}, right-looking) and joins
//     them into the inverse of their 32x32 block,
//   solve_merge_64: a warp computes an 8-column block of the last off-diagonal 32x32 block,
// both by block elimination  [[Ta, 0], [X, Tb]],  X = -Tb (A_ba Ta),  whose small products run on
// the legacy mma.sync path (tcgen05 needs M >= 64).  The intermediate product A_ba Ta changes
// from accumulator to operand layout through the block of sA that mirrors X above the diagonal
// (zero in A and in T), which the warp clears again.
// Warp `pr` (0 or 1) of the group: diagonal blocks 2 pr, 2 pr + 1 and block (2 pr + 1, 2 pr).
__device__ __forceinline__ void solve_blocks_16_32(float* sA, const int pr, const int lane,
                                                   const int len) {
    {
        const int I = 2 * pr + (lane >> 4), j = lane & 15;
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
    if (len <= 32 * pr + 16) return;       // block (2 pr + 1, 2 pr) lies in rows past the chunk's length: zero
    __syncwarp();
    const int g = lane >> 2, t = lane & 3;
    const int I = 2 * pr + 1, J = 2 * pr;
    float* A_IJ = sA + (16 * I) * kLdA + 16 * J;
    float* X = sA + (16 * J) * kLdA + 16 * I;          // the mirror block, zero on entry
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) {                   // X = A_IJ T_JJ
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        mma_tile_tf32<2>(A_IJ, kLdA, sA + (16 * J) * kLdA + 16 * J + 8 * nb, kLdA, c, g, t);
        *reinterpret_cast<float2*>(X + g * kLdA + 8 * nb + 2 * t) = make_float2(c[0], c[1]);
        *reinterpret_cast<float2*>(X + (g + 8) * kLdA + 8 * nb + 2 * t) = make_float2(c[2], c[3]);
    }
    __syncwarp();
    float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)                     // T_IJ = -T_II X
        mma_tile_tf32<2>(sA + (16 * I) * kLdA + 16 * I, kLdA, X + 8 * nb, kLdA, c[nb], g, t);
    __syncwarp();                                      // every lane has read X and A_IJ
    {
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
        float* xr = X + (lane >> 1) * kLdA + 8 * (lane & 1);
        *reinterpret_cast<float4*>(xr) = zero;
        *reinterpret_cast<float4*>(xr + 4) = zero;
    }
#pragma unroll
    for (int nb = 0; nb < 2; ++nb) {
        float* dst = A_IJ + 8 * nb;
        *reinterpret_cast<float2*>(dst + g * kLdA + 2 * t) = make_float2(-c[nb][0], -c[nb][1]);
        *reinterpret_cast<float2*>(dst + (g + 8) * kLdA + 2 * t) = make_float2(-c[nb][2], -c[nb][3]);
    }
}

// Columns 8 nb .. 8 nb + 7 (nb = 0..3) of the 32x32 block (1, 0), by one warp, given the inverses
// of the two diagonal 32x32 blocks.  Called by four consecutive warps together: each reads all
// of A_ba for its first product and writes its columns of the result over A_ba afterwards, so
// the four meet at a barrier of their own (`bar_id`, 128 threads) in between.
__device__ __forceinline__ void solve_merge_64(float* sA, const int nb, const int lane,
                                               const int bar_id) {
    const int g = lane >> 2, t = lane & 3;
    float* Y = sA + 32 + 8 * nb;                       // rows 0-31 of the mirror block, zero on entry
#pragma unroll
    for (int mr = 0; mr < 2; ++mr) {                   // Y = A_ba Ta
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        mma_tile_tf32<4>(sA + (32 + 16 * mr) * kLdA, kLdA, sA + 8 * nb, kLdA, c, g, t);
        *reinterpret_cast<float2*>(Y + (16 * mr + g) * kLdA + 2 * t) = make_float2(c[0], c[1]);
        *reinterpret_cast<float2*>(Y + (16 * mr + g + 8) * kLdA + 2 * t) = make_float2(c[2], c[3]);
    }
    asm volatile("bar.sync %0, 128;" ::"r"(bar_id) : "memory");      // A_ba has been read by all four warps
    float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int mr = 0; mr < 2; ++mr)                     // X = -Tb Y
        mma_tile_tf32<4>(sA + (32 + 16 * mr) * kLdA + 32, kLdA, Y, kLdA, c[mr], g, t);
    __syncwarp();                                      // every lane has read Y and A_ba
    {
        const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
        *reinterpret_cast<float4*>(Y + lane * kLdA) = zero;
        *reinterpret_cast<float4*>(Y + lane * kLdA + 4) = zero;
    }
#pragma unroll
    for (int mr = 0; mr < 2; ++mr) {
        float* dst = sA + (32 + 16 * mr) * kLdA + 8 * nb;
        *reinterpret_cast<float2*>(dst + g * kLdA + 2 * t) = make_float2(-c[mr][0], -c[mr][1]);
        *reinterpret_cast<float2*>(dst + (g + 8) * kLdA + 2 * t) = make_float2(-c[mr][2], -c[mr][3]);
    }
}

// Lane 0 polls the mbarrier (bounded), the other lanes block at the warp barrier instead of
// competing for issue slots; returns the same verdict on every lane.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// The intra-chunk quantities of one (chunk, v-head) item, computed by a group of 256 threads
// (tid = 0..255 within the group; its warps must be CTA warps 0-3 mod 4 aligned, because a warp
// reaches TMEM lanes 32 (warp % 4) ...).  `smem` is the group's 1024-aligned slice of kI_End
// bytes, `tmem` its 128 TMEM columns, `sync` a barrier over exactly the group.  Writes the item's
// record; returns false after a bounded wait gave up (status word set, nothing left in flight).
template <class Sync>
__device__ __forceinline__ bool intra_item(const TensorMaps& maps, const PrefillParams& p,
                                           uint8_t* rec, const ChunkInfo ci, const int hqk,
                                           const int hv, uint8_t* smem, IntraStatics& st,
                                           const uint32_t tmem, const int tid, Sync sync,
                                           const uint32_t n_done = 0) {
    // `n_done` = items this group has processed before (persistent callers): the mbarriers are
    // initialised once and keep flipping phase, one completion of bar_tma and bar_v and three
    // of bar_mma per item.
    const uint32_t par1 = n_done & 1u;           // parity of this item's bar_tma / bar_v phase
    const uint32_t par3 = (3u * n_done) & 1u;    // parity of this item's first bar_mma phase
    const int warp = tid >> 5;
    const int colhalf = warp >> 2;                   // which 32 of the 64 accumulator columns
    if (tid == 0) {
        if (n_done == 0) {
            mbar_init(&st.bar_tma, 1);
            mbar_init(&st.bar_v, 1);
            mbar_init(&st.bar_mma, 1);
            fence_barrier_init();
        }
        st.abort_flag = 0;
        // Q and K first: everything below overlaps their flight (V comes later, over dead data)
        mbar_expect_tx(&st.bar_tma, 32768);
        tma_load_2d(smem + kI_QK, &maps.q, hqk * kD, ci.t0, &st.bar_tma);
        tma_load_2d(smem + kI_QK + 8192, &maps.k, hqk * kD, ci.t0, &st.bar_tma);
        tma_load_2d(smem + kI_QK + 16384, &maps.q, hqk * kD + 64, ci.t0, &st.bar_tma);
        tma_load_2d(smem + kI_QK + 24576, &maps.k, hqk * kD + 64, ci.t0, &st.bar_tma);
        // V has no room in shared memory until the solve is over; fetch it into L2 meanwhile, so
        // that its load then is not a DRAM round trip in front of the U~ product
        tma_prefetch_2d(&maps.v, hv * kD, ci.t0);
        tma_prefetch_2d(&maps.v, hv * kD + 64, ci.t0);
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
        st.s_b2[2 * lane] = b0 * kLog2e; st.s_b2[2 * lane + 1] = b1 * kLog2e;
        st.s_beta[2 * lane] = be0; st.s_beta[2 * lane + 1] = be1;
        const float e0 = ex2_approx(b0 * kLog2e), e1 = ex2_approx(b1 * kLog2e);
        st.s_eb[2 * lane] = e0; st.s_eb[2 * lane + 1] = e1;
        st.s_bg[2 * lane] = be0 * e0; st.s_bg[2 * lane + 1] = be1 * e1;
        // decay vector of the record: e^{b_C - b_c}, then e^{b_C}
        float* dec = reinterpret_cast<float*>(rec + kRecDecay);
        dec[2 * lane] = ex2_approx((bC - b0) * kLog2e);
        dec[2 * lane + 1] = ex2_approx((bC - b1) * kLog2e);
        if (lane == 0) dec[kChunk] = ex2_approx(bC * kLog2e);
    }
    sync();
    // On a timeout: flag it and let thread 0 drain what it has in flight; the caller unwinds.
    auto bail = [&](bool stores_pending) {
        if (tid == 0) {
            report(p.dev_status, kDevTimeout);
            if (stores_pending) bulk_wait_read_all();
        }
    };

    if (warp == 0 && !warp_wait(&st.bar_tma, par1)) st.abort_flag = 1;      // one warp polls, the rest block
    sync();
    if (st.abort_flag) { bail(false); return false; }
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
        mma_commit(&st.bar_mma);
    }
    if (warp == 0 && !warp_wait(&st.bar_mma, par3)) st.abort_flag = 1;
    sync();
    if (st.abort_flag) { bail(false); return false; }
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
        const float br2 = st.s_b2[r];
        const float rowscale = is_p ? p.scale : st.s_beta[r];      // the output scale rides on P and Qg
        const int limit = is_p ? r : r - 1;              // keep columns i <= limit
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cbase = colhalf * 32 + step * 16;
            float val[16];
            // a 16-column block that lies wholly above the diagonal for every row of the warp is
            // zero (warp-uniform test: no accumulator read, no exponentials)
            if (cbase > (row & 32) + 31) {
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) val[jj] = 0.f;
            } else {
                uint32_t x[16];
                tmem_ld16(tG + lane_base + cbase, x);
                tmem_wait_ld();
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const float4 bb = *reinterpret_cast<const float4*>(st.s_b2 + cbase + 4 * q4);
                    const float bv[4] = {bb.x, bb.y, bb.z, bb.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int jj = 4 * q4 + e;
                        const bool keep = cbase + jj <= limit;
                        const float dec = ex2_approx(keep ? br2 - bv[e] : 0.f);   // e^{b_r - b_i}
                        val[jj] = keep ? rowscale * dec * __uint_as_float(x[jj]) : 0.f;
                    }
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
                    *reinterpret_cast<uint4*>(rec + kRecP + sw128_offset(r, (cbase >> 3) + h)) = w;
                }
            } else {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<float4*>(sA + r * kLdA + cbase + 4 * q4) =
                        make_float4(val[4 * q4], val[4 * q4 + 1], val[4 * q4 + 2], val[4 * q4 + 3]);
            }
        }
    }
    tc_fence_before_sync();
    sync();
    // Two jobs side by side: warps 0-1 invert the two diagonal 32x32 blocks of I + A (serial
    // forward substitutions and two small products each, all inside the warp), warps 2-7 scale
    // the Q rows by scale * e^{b_r} in place (the Gram product has consumed Q): the Qg image.
    if (warp < 2) {
        solve_blocks_16_32(sA, warp, tid & 31, ci.len);
    } else {
#pragma unroll 2
        for (int idx = tid - 64; idx < 1024; idx += kIntraThreads - 64) {      // 1024 16-byte pieces
            const int halfq = idx >> 9, rem = idx & 511;
            const int r = rem >> 3;
            uint4* ptr = reinterpret_cast<uint4*>(smem + kI_QK + halfq * 16384 + rem * 16);
            const float f = st.s_eb[r] * p.scale;
            uint4 w = *ptr;
            w.x = scale_bf16x2(w.x, f); w.y = scale_bf16x2(w.y, f);
            w.z = scale_bf16x2(w.z, f); w.w = scale_bf16x2(w.w, f);
            *ptr = w;
        }
        fence_proxy_async_smem();
    }
    sync();
    if (tid == 0) {
        // Qg is final: store it now.  The T_w / T_u images are written over it next: wait for the
        // bulk store's reads (not for its writes to land) meanwhile.
        bulk_store(rec + kRecQg, smem + kI_QK, 8192);
        bulk_store(rec + kRecQg + 8192, smem + kI_QK + 16384, 8192);
        bulk_commit();
        bulk_wait_read_all();
    } else if (warp >= 4 && ci.len > 32) {
        // (rows past the length are zero: nothing to do then).  Barrier ids 4.. are this routine's:
        // one per group of 256 threads of the CTA.
        solve_merge_64(sA, warp - 4, tid & 31, 4 + (static_cast<int>(threadIdx.x) >> 8));
    }
    sync();

    uint32_t tu_lo[2][4];    // T diag(beta) - bf16(T diag(beta)), parked until T_w is dead
    {   // T (fp32, row-major) -> bf16 B operands T diag(beta e^b), T diag(beta) (hi, lo)
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int idx = tid + it * kIntraThreads;          // 512 pieces of 8 columns
            const int r = idx >> 3, c8 = idx & 7;
            const float4 t0 = *reinterpret_cast<const float4*>(sA + r * kLdA + 8 * c8);
            const float4 t1 = *reinterpret_cast<const float4*>(sA + r * kLdA + 8 * c8 + 4);
            const float4 g0 = *reinterpret_cast<const float4*>(st.s_bg + 8 * c8);
            const float4 g1 = *reinterpret_cast<const float4*>(st.s_bg + 8 * c8 + 4);
            const float4 e0 = *reinterpret_cast<const float4*>(st.s_beta + 8 * c8);
            const float4 e1 = *reinterpret_cast<const float4*>(st.s_beta + 8 * c8 + 4);
            const float tv[8] = {t0.x, t0.y, t0.z, t0.w, t1.x, t1.y, t1.z, t1.w};
            const float gv[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const float ev[8] = {e0.x, e0.y, e0.z, e0.w, e1.x, e1.y, e1.z, e1.w};
            uint32_t w[4], hi[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                w[j] = pack_bf16(tv[2 * j] * gv[2 * j], tv[2 * j + 1] * gv[2 * j + 1]);
                const float u0 = tv[2 * j] * ev[2 * j], u1 = tv[2 * j + 1] * ev[2 * j + 1];
                hi[j] = pack_bf16(u0, u1);
                tu_lo[it][j] = pack_bf16(u0 - __uint_as_float(hi[j] << 16),
                                         u1 - __uint_as_float(hi[j] & 0xffff0000u));
            }
            const uint32_t off = sw128_offset(r, c8);
            *reinterpret_cast<uint4*>(smem + kI_Tw + off) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(smem + kI_Tu + off) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
        }
    }
    fence_proxy_async_smem();
    sync();

    const uint32_t sV = smem_u32(smem + kI_V);
    if (tid == 0) {
        // V into the space the solve has left; meanwhile W^T (dk x r) = K^T T_w^T with the raw K
        // tile read MN-major
        mbar_expect_tx(&st.bar_v, 16384);
        tma_load_2d(smem + kI_V, &maps.v, hv * kD, ci.t0, &st.bar_v);
        tma_load_2d(smem + kI_V + 8192, &maps.v, hv * kD + 64, ci.t0, &st.bar_v);
        const uint32_t idesc = make_idesc_bf16(128, 64, true, false);
        const uint32_t sTw = smem_u32(smem + kI_Tw);
        // columns of T_w and T_u past the chunk's length are zero: their k-steps are left out
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            if (ks * 16 < ci.len)
                mma_ss(tW, make_sdesc_sw128(sQK + 8192 + ks * 2048, 16384, 1024),
                       make_sdesc_sw128(sTw + ks * 32, 16, 1024), idesc, ks > 0);
        mma_commit(&st.bar_mma);
    }
    if (warp == 0 && !warp_wait(&st.bar_mma, par3 ^ 1u)) st.abort_flag = 1;
    sync();
    if (st.abort_flag) { bail(false); return false; }      // nothing of thread 0's stores is pending here
    tc_fence_after_sync();

    const int d = (warp & 3) * 32 + (tid & 31);   // TMEM lane of this thread: a dk / dv index
    {   // W^T[d][32 tokens] -> bf16 -> W image staged over the (now dead) K halves.  The image
        // is MN-major for the state pass's product S W^T (one 128-byte row of 64 tokens per dk
        // index), so a thread writes its own row in 16-byte pieces.
        uint8_t* sW = smem + kI_QK + 8192 + (d >> 6) * 16384;
#pragma unroll
        for (int step = 0; step < 2; ++step) {
            const int cbase = colhalf * 32 + step * 16;
            uint32_t x[16];
            tmem_ld16(tW + lane_base + cbase, x);
            tmem_wait_ld();
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(x[8 * h + 0]), __uint_as_float(x[8 * h + 1]));
                w.y = pack_bf16(__uint_as_float(x[8 * h + 2]), __uint_as_float(x[8 * h + 3]));
                w.z = pack_bf16(__uint_as_float(x[8 * h + 4]), __uint_as_float(x[8 * h + 5]));
                w.w = pack_bf16(__uint_as_float(x[8 * h + 6]), __uint_as_float(x[8 * h + 7]));
                *reinterpret_cast<uint4*>(sW + sw128_offset(d & 63, (cbase >> 3) + h)) = w;
            }
        }
    }
    // the product that read T_w has retired: its place takes the remainder of T diag(beta)
#pragma unroll
    for (int it = 0; it < 2; ++it) {
        const int idx = tid + it * kIntraThreads;
        *reinterpret_cast<uint4*>(smem + kI_TuLo + sw128_offset(idx >> 3, idx & 7)) =
            make_uint4(tu_lo[it][0], tu_lo[it][1], tu_lo[it][2], tu_lo[it][3]);
    }
    fence_proxy_async_smem();
    tc_fence_before_sync();
    if (warp == 0 && !warp_wait(&st.bar_v, par1)) st.abort_flag = 1;        // V has landed
    sync();
    if (st.abort_flag) { bail(false); return false; }
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
            if (ks * 16 < ci.len)
                mma_ss(tU, make_sdesc_sw128(sV + ks * 2048, 8192, 1024),
                       make_sdesc_sw128(sTu + ks * 32, 16, 1024), idesc, ks > 0);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
            if (ks * 16 < ci.len)
                mma_ss(tU, make_sdesc_sw128(sV + ks * 2048, 8192, 1024),
                       make_sdesc_sw128(sTuLo + ks * 32, 16, 1024), idesc, true);
        mma_commit(&st.bar_mma);
    }
    if (warp == 0 && !warp_wait(&st.bar_mma, par3)) st.abort_flag = 1;
    sync();
    if (st.abort_flag) { bail(true); return false; }
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
    sync();
    if (tid == 0) bulk_wait_read_all();
    return true;
}

constexpr uint32_t kStateTmemCols = 512;
constexpr uint32_t kS_Rec = 0;                 // record image (74240 B, padded to 74752)
constexpr uint32_t kS_K = 74752;               // K tile, 2 halves [64 x 128 B]
constexpr uint32_t kStageBytes = 74752 + 16384;                 // 91136
constexpr uint32_t kS_Out = 2 * kStageBytes;   // o staging [64 tokens][128 dv] bf16
// TMEM columns
constexpr uint32_t kT_D1 = 0, kT_Y = 64 /* two tiles of 64 */, kT_D4 = 192, kT_S = 320, kT_U = 384,
                   kT_Us = 416, kT_UsLo = 448;

// bounded wait that also gives up as soon as another role has flagged an abort.  `reason` is what a
// wait that runs out writes into the flag: 1 = an error (reported as a timeout), 2 = give up
// without an error (the caller's work is finished by a later launch).
__device__ __forceinline__ bool wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                              const int reason = 1) {
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((i & 255u) == 255u && *abort_flag) return false;
    }
    if (*abort_flag == 0) *abort_flag = reason;      // keep an earlier, different reason
    return false;
}

// Same, for a whole warp: lane 0 polls, every lane gets the verdict.
__device__ __forceinline__ bool warp_wait_or_abort(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                   const int reason = 1) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = wait_or_abort(bar, parity, abort_flag, reason) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}


}  // namespace gdn
