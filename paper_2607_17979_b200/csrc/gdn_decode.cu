// Decode: one gated-delta-rule token per (sequence, v-head) state tile.
//
//   S <- exp(g) S ;  u = S k ;  S <- S + beta (v - u) k^T ;  o = scale S q
//
// Bandwidth-bound: every 128x128 fp32 tile (64 KiB) is read once and written
// once, in place.  One CTA of 256 threads owns half a tile (64 rows; the rows
// evolve independently).  Eight lanes share a row (each holds 16 of its 128
// columns as four float4, interleaved so that a warp-wide load covers four
// 128-byte row segments); a warp owns 8 rows in two passes of four rows.  All
// float4 loads of a thread are issued before any arithmetic, so a CTA keeps its
// 32 KiB in flight, three CTAs (96 KiB) per SM.
// With p_k = S_old.k and p_q = S_old.q per row (two 8-lane shuffle sums):
//   u = alpha p_k,  w = beta (v_j - u),  S_new = alpha S_old + w k,
//   o_j = scale (alpha p_q + w (k.q)).
#include "gdn_common.cuh"

namespace gdn {

constexpr int kDecodeThreads = 256;

__device__ __forceinline__ float4 ld_stream(const float4* p) {
    float4 r;
    asm volatile("ld.global.cs.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ void st_stream(float4* p, const float4& r) {
    asm volatile("st.global.cs.v4.f32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "f"(r.x), "f"(r.y), "f"(r.z), "f"(r.w) : "memory");
}

// kPasses = 2: a tile is split over two CTAs of 64 rows each (rows evolve independently), three
// CTAs per SM: the default.  kPasses = 1: four CTAs of 32 rows per tile, used when there are too
// few tiles to fill the GPU.  (kPasses = 4, one CTA per tile at two CTAs per SM, also compiles.)
template <int kPasses>
__global__ void __launch_bounds__(kDecodeThreads, kPasses == 2 ? 3 : 2)
decode_kernel(const DecodeParams p) {
    constexpr int kSplit = 4 / kPasses;
    const int unit = blockIdx.x / kSplit;
    const int part = blockIdx.x - unit * kSplit;
    const int i = unit / p.Hv;
    const int hv = unit - i * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane & 7;        // which 16-column share of the row
    const int rsel = lane >> 3;      // which of the pass's four rows

    __nv_bfloat16* o_row = p.o + (static_cast<size_t>(i) * p.Hv + hv) * kD;
    const int slot = p.slot_idx ? p.slot_idx[i] : i;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && threadIdx.x == 0 && part == 0) report(p.dev_status, kDevBadSlot);
        if (threadIdx.x < kD / kSplit) o_row[part * (kD / kSplit) + threadIdx.x] = __float2bfloat16(0.f);
        return;
    }

    float* tile = p.pool + (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD);
    const int row0 = part * (kD / kSplit) + warp * (4 * kPasses) + rsel;
    float4 s[kPasses][4];
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps)
#pragma unroll
        for (int j = 0; j < 4; ++j)
            s[ps][j] = ld_stream(reinterpret_cast<const float4*>(
                tile + (row0 + ps * 4) * kD + sub * 4 + j * 32));

    const __nv_bfloat16* kp = p.k + (static_cast<size_t>(i) * p.Hqk + hqk) * kD;
    const __nv_bfloat16* qp = p.q + (static_cast<size_t>(i) * p.Hqk + hqk) * kD;
    const __nv_bfloat16* vp = p.v + (static_cast<size_t>(i) * p.Hv + hv) * kD;
    float4 kf[4], qf[4];
    float kq = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        kf[j] = load_bf16x4(kp + sub * 4 + j * 32);
        qf[j] = load_bf16x4(qp + sub * 4 + j * 32);
        kq = dot4(kf[j], qf[j], kq);
    }
    kq = sum8(kq);
    const float alpha = expf(p.g[static_cast<size_t>(i) * p.Hv + hv]);
    const float beta = p.beta[static_cast<size_t>(i) * p.Hv + hv];
    float vj[kPasses];
#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) vj[ps] = __bfloat162float(vp[row0 + ps * 4]);

#pragma unroll
    for (int ps = 0; ps < kPasses; ++ps) {
        float pk = 0.f, pq = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            pk = dot4(s[ps][j], kf[j], pk);
            pq = dot4(s[ps][j], qf[j], pq);
        }
        pk = sum8(pk);
        pq = sum8(pq);
        const float w = beta * (vj[ps] - alpha * pk);
        const int row = row0 + ps * 4;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            float4 r;
            r.x = fmaf(w, kf[j].x, alpha * s[ps][j].x);
            r.y = fmaf(w, kf[j].y, alpha * s[ps][j].y);
            r.z = fmaf(w, kf[j].z, alpha * s[ps][j].z);
            r.w = fmaf(w, kf[j].w, alpha * s[ps][j].w);
            st_stream(reinterpret_cast<float4*>(tile + row * kD + sub * 4 + j * 32), r);
        }
        if (sub == 0) o_row[row] = __float2bfloat16(p.scale * fmaf(w, kq, alpha * pq));
    }
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t stream) {
    const long long units = static_cast<long long>(p.B) * p.Hv;
    if (units == 0) return cudaSuccess;
    // below about two CTAs per SM of whole tiles, quarter tiles spread the same bytes over four
    // times as many SMs (the state rows are independent)
    DeviceInfo di;
    const int sms = device_info(&di) == cudaSuccess ? di.sms : 148;
    if (units < 2LL * sms)
        decode_kernel<1><<<static_cast<unsigned>(units * 4), kDecodeThreads, 0, stream>>>(p);
    else   // half tiles at three CTAs per SM: measured 0.5-1 % faster than whole tiles at two
        decode_kernel<2><<<static_cast<unsigned>(units * 2), kDecodeThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace gdn
