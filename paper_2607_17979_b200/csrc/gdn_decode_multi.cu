// Decode of L >= 1 new tokens per sequence with the state tile held in registers across the
// tokens, for either orientation of the tile in memory.
//
//   per token:  S <- exp(g) S ;  u = S k ;  S <- S + beta (v - u) k^T ;  o = scale S q
//
// A tile is read once and written once however many tokens are applied, so the 128 KiB of
// traffic per (sequence, v-head) is amortised over L tokens.  The tokens' q, k, v, g, beta are
// staged in shared memory as fp32 while the tile's loads are in flight.
//
//   layout 0 ("vk"): tile [dv][dk], dk contiguous.  Same thread map as the one-token kernel:
//       eight lanes share a state row (a dv index), S k and S q are 8-lane shuffle sums.
//   layout 1 ("kv"): tile [dk][dv], dv contiguous.  A memory row is now a k index, so S k and
//       S q are sums DOWN the rows: every thread accumulates over the rows it holds, the eight
//       warps' partial sums meet in shared memory, and the per-column correction
//       w_j = beta (v_j - alpha (S k)_j) is broadcast back for the rank-1 update.
#include "gdn_common.cuh"

namespace gdn {

constexpr int kMultiThreads = 256;

namespace {

__device__ __forceinline__ float4 ldcs(const float4* p) {
    float4 r;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void stcs(float4* p, const float4& r) {
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "f"(r.x), "f"(r.y), "f"(r.z), "f"(r.w) : "memory");
}

// Packed pairs of fp32 (sm_100 issues one instruction for two lanes): d = a * b + c, d = a * b.
__device__ __forceinline__ float2 fma2(const float2 a, const float2 b, const float2 c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(d)
        : "l"(*reinterpret_cast<const unsigned long long*>(&a)),
          "l"(*reinterpret_cast<const unsigned long long*>(&b)),
          "l"(*reinterpret_cast<const unsigned long long*>(&c)));
    return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 mul2(const float2 a, const float2 b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;"
        : "=l"(d)
        : "l"(*reinterpret_cast<const unsigned long long*>(&a)),
          "l"(*reinterpret_cast<const unsigned long long*>(&b)));
    return *reinterpret_cast<float2*>(&d);
}
__device__ __forceinline__ float2 lo2(const float4& a) { return make_float2(a.x, a.y); }
__device__ __forceinline__ float2 hi2(const float4& a) { return make_float2(a.z, a.w); }
__device__ __forceinline__ float4 join(const float2 a, const float2 b) {
    return make_float4(a.x, a.y, b.x, b.y);
}

struct TokenStage {
    float k[kDecodeMaxTokens][kD];
    float q[kDecodeMaxTokens][kD];
    float v[kDecodeMaxTokens][kD];
    float alpha[kDecodeMaxTokens];
    float beta[kDecodeMaxTokens];
    float kq[kDecodeMaxTokens];
};

// q, k, v of the L tokens of entry i -> fp32 in shared memory; alpha = exp(g); kq = k.q.
// Ends with a __syncthreads().
__device__ __forceinline__ void stage_tokens(const DecodeMultiParams& mp, TokenStage& st, int i,
                                             int hv, int hqk) {
    const DecodeParams& p = mp.d;
    const int L = mp.L;
    for (int idx = threadIdx.x; idx < L * (kD / 4); idx += kMultiThreads) {
        const int t = idx / (kD / 4), c = (idx - t * (kD / 4)) * 4;
        const size_t tok = static_cast<size_t>(i) * L + t;
        *reinterpret_cast<float4*>(&st.k[t][c]) = load_bf16x4(p.k + (tok * p.Hqk + hqk) * kD + c);
        *reinterpret_cast<float4*>(&st.q[t][c]) = load_bf16x4(p.q + (tok * p.Hqk + hqk) * kD + c);
        *reinterpret_cast<float4*>(&st.v[t][c]) = load_bf16x4(p.v + (tok * p.Hv + hv) * kD + c);
    }
    if (threadIdx.x < L) {
        const size_t tok = static_cast<size_t>(i) * L + threadIdx.x;
        st.alpha[threadIdx.x] = expf(p.g[tok * p.Hv + hv]);
        st.beta[threadIdx.x] = p.beta[tok * p.Hv + hv];
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int t = warp; t < L; t += kMultiThreads / 32) {
        const float4 a = *reinterpret_cast<const float4*>(&st.k[t][lane * 4]);
        const float4 b = *reinterpret_cast<const float4*>(&st.q[t][lane * 4]);
        float x = dot4(a, b, 0.f);
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) x += __shfl_xor_sync(0xffffffffu, x, m);
        if (lane == 0) st.kq[t] = x;
    }
    __syncthreads();
}

// zero the o rows of a padding entry (all L tokens, this CTA's share of the dv range)
__device__ __forceinline__ void zero_outputs(const DecodeMultiParams& mp, int i, int hv, int first,
                                             int count) {
    for (int idx = threadIdx.x; idx < mp.L * count; idx += kMultiThreads) {
        const int t = idx / count, c = idx - t * count;
        mp.d.o[((static_cast<size_t>(i) * mp.L + t) * mp.d.Hv + hv) * kD + first + c] =
            __float2bfloat16(0.f);
    }
}

}  // namespace

// ---- layout 0: tile [dv][dk] -------------------------------------------------------------------
// kPasses = 4: one CTA per tile; kPasses = 1: a tile split over four CTAs of 32 dv rows each.
template <int kPasses>
__global__ void __launch_bounds__(kMultiThreads, kPasses == 4 ? 2 : 3)
decode_multi_vk_kernel(const DecodeMultiParams mp) {
    __shared__ __align__(16) TokenStage st;
    const DecodeParams& p = mp.d;
    constexpr int kSplit = 4 / kPasses;
    const int unit = blockIdx.x / kSplit;
    const int part = blockIdx.x - unit * kSplit;
    const int i = unit / p.Hv;
    const int hv = unit - i * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane & 7;
    const int rsel = lane >> 3;

    const int slot = p.slot_idx ? p.slot_idx[i] : i;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && threadIdx.x == 0 && part == 0) report(p.dev_status, kDevBadSlot);
        zero_outputs(mp, i, hv, part * (kD / kSplit), kD / kSplit);
        return;
    }

    float* tile = p.pool + (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD);
    const int row0 = part * (kD / kSplit) + warp * (4 * kPasses) + rsel;
    float4 s[kPasses][4];
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            s[ps][j] = ldcs(reinterpret_cast<const float4*>(
                tile + (row0 + ps * 4) * kD + sub * 4 + j * 32));

    stage_tokens(mp, st, i, hv, hqk);

    for (int t = 0; t < mp.L; ++t) {
        float4 kf[4], qf[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            kf[j] = *reinterpret_cast<const float4*>(&st.k[t][sub * 4 + j * 32]);
            qf[j] = *reinterpret_cast<const float4*>(&st.q[t][sub * 4 + j * 32]);
        }
        const float alpha = st.alpha[t], beta = st.beta[t], kq = st.kq[t];
        __nv_bfloat16* o_row = p.o + ((static_cast<size_t>(i) * mp.L + t) * p.Hv + hv) * kD;
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) {
            float2 pk2 = make_float2(0.f, 0.f), pq2 = pk2;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                pk2 = fma2(lo2(s[ps][j]), lo2(kf[j]), pk2);
                pk2 = fma2(hi2(s[ps][j]), hi2(kf[j]), pk2);
                pq2 = fma2(lo2(s[ps][j]), lo2(qf[j]), pq2);
                pq2 = fma2(hi2(s[ps][j]), hi2(qf[j]), pq2);
            }
            const float pk = sum8(pk2.x + pk2.y);
            const float pq = sum8(pq2.x + pq2.y);
            const int row = row0 + ps * 4;
            const float w = beta * (st.v[t][row] - alpha * pk);
            const float2 w2 = make_float2(w, w), a2 = make_float2(alpha, alpha);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                s[ps][j] = join(fma2(w2, lo2(kf[j]), mul2(a2, lo2(s[ps][j]))),
                                fma2(w2, hi2(kf[j]), mul2(a2, hi2(s[ps][j]))));
            if (sub == 0) o_row[row] = __float2bfloat16(p.scale * fmaf(w, kq, alpha * pq));
        }
    }

#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            stcs(reinterpret_cast<float4*>(tile + (row0 + ps * 4) * kD + sub * 4 + j * 32),
                 s[ps][j]);
}

// ---- layout 1: tile [dk][dv] -------------------------------------------------------------------
// kSplit = 1: one CTA per tile, a warp load covers one whole 512-byte row, a warp owns 16 rows.
// kSplit = 4: four CTAs per tile, each owning 32 dv columns (columns evolve independently); a warp
// load covers the 128-byte column share of four rows.  kSplit = 2: two CTAs of 64 columns.
template <int kSplit>
__global__ void __launch_bounds__(kMultiThreads, kSplit == 2 ? 3 : 2)
decode_multi_kv_kernel(const DecodeMultiParams mp) {
    __shared__ __align__(16) TokenStage st;
    constexpr int kCols = kD / kSplit;            // dv columns of this CTA
    constexpr int kLanesPerRow = kCols / 4;       // 32 or 8
    constexpr int kRowsPerLoad = 32 / kLanesPerRow;
    constexpr int kLoads = 16 / kRowsPerLoad;     // float4 per thread: 16 or 4
    __shared__ __align__(16) float red[kMultiThreads / 32][2][kCols];
    __shared__ __align__(16) float sw[kCols];

    const DecodeParams& p = mp.d;
    const int unit = blockIdx.x / kSplit;
    const int part = blockIdx.x - unit * kSplit;
    const int i = unit / p.Hv;
    const int hv = unit - i * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int cg = lane % kLanesPerRow;           // which float4 of the column share
    const int rsel = lane / kLanesPerRow;

    const int slot = p.slot_idx ? p.slot_idx[i] : i;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && threadIdx.x == 0 && part == 0) report(p.dev_status, kDevBadSlot);
        zero_outputs(mp, i, hv, part * kCols, kCols);
        return;
    }

    float* tile = p.pool + (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD);
    const int row0 = warp * 16 + rsel;
    const int col0 = part * kCols + cg * 4;
    float4 s[kLoads];
#pragma unroll
    for (int ld = 0; ld < kLoads; ++ld)
        s[ld] = ldcs(reinterpret_cast<const float4*>(
            tile + (row0 + ld * kRowsPerLoad) * kD + col0));

    stage_tokens(mp, st, i, hv, hqk);

    for (int t = 0; t < mp.L; ++t) {
        float2 akl = make_float2(0.f, 0.f), akh = akl, aql = akl, aqh = akl;
#pragma unroll
        for (int ld = 0; ld < kLoads; ++ld) {
            const float kr = st.k[t][row0 + ld * kRowsPerLoad];
            const float qr = st.q[t][row0 + ld * kRowsPerLoad];
            const float2 k2 = make_float2(kr, kr), q2 = make_float2(qr, qr);
            akl = fma2(lo2(s[ld]), k2, akl);
            akh = fma2(hi2(s[ld]), k2, akh);
            aql = fma2(lo2(s[ld]), q2, aql);
            aqh = fma2(hi2(s[ld]), q2, aqh);
        }
        float4 ak = join(akl, akh), aq = join(aql, aqh);
        if (kRowsPerLoad > 1) {
#pragma unroll
            for (int m = kLanesPerRow; m < 32; m <<= 1) {
                ak.x += __shfl_xor_sync(0xffffffffu, ak.x, m);
                ak.y += __shfl_xor_sync(0xffffffffu, ak.y, m);
                ak.z += __shfl_xor_sync(0xffffffffu, ak.z, m);
                ak.w += __shfl_xor_sync(0xffffffffu, ak.w, m);
                aq.x += __shfl_xor_sync(0xffffffffu, aq.x, m);
                aq.y += __shfl_xor_sync(0xffffffffu, aq.y, m);
                aq.z += __shfl_xor_sync(0xffffffffu, aq.z, m);
                aq.w += __shfl_xor_sync(0xffffffffu, aq.w, m);
            }
        }
        if (rsel == 0) {
            *reinterpret_cast<float4*>(&red[warp][0][cg * 4]) = ak;
            *reinterpret_cast<float4*>(&red[warp][1][cg * 4]) = aq;
        }
        __syncthreads();
        const float alpha = st.alpha[t];
        if (threadIdx.x < kCols) {
            float pk = 0.f, pq = 0.f;
#pragma unroll
            for (int w = 0; w < kMultiThreads / 32; ++w) {
                pk += red[w][0][threadIdx.x];
                pq += red[w][1][threadIdx.x];
            }
            const int col = part * kCols + threadIdx.x;
            const float w = st.beta[t] * (st.v[t][col] - alpha * pk);
            sw[threadIdx.x] = w;
            p.o[((static_cast<size_t>(i) * mp.L + t) * p.Hv + hv) * kD + col] =
                __float2bfloat16(p.scale * fmaf(w, st.kq[t], alpha * pq));
        }
        __syncthreads();
        const float4 wv = *reinterpret_cast<const float4*>(&sw[cg * 4]);
        const float2 a2 = make_float2(alpha, alpha);
#pragma unroll
        for (int ld = 0; ld < kLoads; ++ld) {
            const float kr = st.k[t][row0 + ld * kRowsPerLoad];
            const float2 k2 = make_float2(kr, kr);
            s[ld] = join(fma2(k2, lo2(wv), mul2(a2, lo2(s[ld]))),
                         fma2(k2, hi2(wv), mul2(a2, hi2(s[ld]))));
        }
    }

#pragma unroll
    for (int ld = 0; ld < kLoads; ++ld)
        stcs(reinterpret_cast<float4*>(tile + (row0 + ld * kRowsPerLoad) * kD + col0), s[ld]);
}

cudaError_t launch_decode_multi(const DecodeMultiParams& mp, cudaStream_t stream) {
    const long long units = static_cast<long long>(mp.d.B) * mp.d.Hv;
    if (units == 0) return cudaSuccess;
    DeviceInfo di;
    const int sms = device_info(&di) == cudaSuccess ? di.sms : 148;
    // fewer than two whole tiles per SM: quarter tiles spread the bytes over more SMs
    const bool split = units < 2LL * sms;
    const unsigned grid = static_cast<unsigned>(split ? units * 4 : units);
    if (mp.layout == 0) {
        if (split) decode_multi_vk_kernel<1><<<grid, kMultiThreads, 0, stream>>>(mp);
        // up to four tokens half tiles at three CTAs per SM overlap loads and arithmetic better;
        // beyond that the four independent row groups of a whole tile hide the per-token chain
        else if (mp.L <= 4) decode_multi_vk_kernel<2><<<grid * 2, kMultiThreads, 0, stream>>>(mp);
        else decode_multi_vk_kernel<4><<<grid, kMultiThreads, 0, stream>>>(mp);
    } else {
        if (split) decode_multi_kv_kernel<4><<<grid, kMultiThreads, 0, stream>>>(mp);
        else if (mp.L <= 2) decode_multi_kv_kernel<2><<<grid * 2, kMultiThreads, 0, stream>>>(mp);
        else decode_multi_kv_kernel<1><<<grid, kMultiThreads, 0, stream>>>(mp);
    }
    return cudaGetLastError();
}

}  // namespace gdn

// ---- in-place transpose of state tiles ([dv][dk] <-> [dk][dv]) ---------------------------------
// One CTA per (entry, v-head) tile.  The 128x128 tile is walked as 4x4 blocks of 32x32; a block
// pair (a, b) and (b, a) is read into two padded shared tiles and written back swapped and
// transposed, so the tile never needs a second copy in memory.
namespace gdn {

__global__ void __launch_bounds__(256)
state_transpose_kernel(float* pool, const int32_t* slot_idx, int32_t Hv, int32_t num_slots,
                       int32_t* dev_status) {
    __shared__ float ta[32][33], tb[32][33];
    const int i = blockIdx.x / Hv, hv = blockIdx.x - i * Hv;
    const int slot = slot_idx ? slot_idx[i] : i;
    if (slot < 0 || slot >= num_slots) {
        if (slot >= num_slots && threadIdx.x == 0) report(dev_status, kDevBadSlot);
        return;
    }
    float* tile = pool + (static_cast<size_t>(slot) * Hv + hv) * (kD * kD);
    const int c = threadIdx.x & 31, r0 = threadIdx.x >> 5;   // 8 rows per sweep
    for (int a = 0; a < 4; ++a)
        for (int b = a; b < 4; ++b) {
#pragma unroll
            for (int r = r0; r < 32; r += 8) {
                ta[r][c] = tile[(a * 32 + r) * kD + b * 32 + c];
                tb[r][c] = tile[(b * 32 + r) * kD + a * 32 + c];
            }
            __syncthreads();
#pragma unroll
            for (int r = r0; r < 32; r += 8) {
                tile[(b * 32 + r) * kD + a * 32 + c] = ta[c][r];
                if (a != b) tile[(a * 32 + r) * kD + b * 32 + c] = tb[c][r];
            }
            __syncthreads();
        }
}

cudaError_t launch_state_transpose(float* pool, const int32_t* slot_idx, int32_t n, int32_t Hv,
                                   int32_t num_slots, int32_t* dev_status, cudaStream_t stream) {
    const long long units = static_cast<long long>(n) * Hv;
    if (units == 0) return cudaSuccess;
    state_transpose_kernel<<<static_cast<unsigned>(units), 256, 0, stream>>>(pool, slot_idx, Hv,
                                                                             num_slots, dev_status);
    return cudaGetLastError();
}

}  // namespace gdn
