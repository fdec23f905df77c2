// Prefill, token by token, on the CUDA cores (no chunking).
//
// The rows of a state tile evolve independently under the gated delta rule
// (row j needs only v[j], k, g, beta), so a (sequence, v-head) tile is split
// into 8 CTAs of 16 rows; a warp carries 4 rows, 8 lanes per row, 16 columns
// per lane, in registers across all tokens of the sequence.  Next token's
// q, k, v, g, beta are fetched while the current token is computed.
#include "gdn_common.cuh"

namespace gdn {

constexpr int kRecThreads = 128;            // 4 warps x 4 rows = 16 rows per CTA
constexpr int kRecRowsPerCta = 16;
constexpr int kRecCtasPerTile = kD / kRecRowsPerCta;

struct TokenRegs {
    float4 k[4], q[4];
    float v, g, beta;
};

__device__ __forceinline__ void fetch_token(TokenRegs& r, const PrefillParams& p, int t, int hqk,
                                            int hv, int sub, int row) {
    const __nv_bfloat16* kp = p.k + (static_cast<size_t>(t) * p.Hqk + hqk) * kD;
    const __nv_bfloat16* qp = p.q + (static_cast<size_t>(t) * p.Hqk + hqk) * kD;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        r.k[j] = load_bf16x4(kp + sub * 4 + j * 32);
        r.q[j] = load_bf16x4(qp + sub * 4 + j * 32);
    }
    const size_t th = static_cast<size_t>(t) * p.Hv + hv;
    r.v = __bfloat162float(p.v[th * kD + row]);
    r.g = p.g[th];
    r.beta = p.beta[th];
}

__global__ void __launch_bounds__(kRecThreads)
prefill_recurrent_kernel(const PrefillParams p) {
    const int part = blockIdx.x % kRecCtasPerTile;
    const int unit = blockIdx.x / kRecCtasPerTile;
    const int n = unit / p.Hv;
    const int hv = unit - n * p.Hv;
    const int hqk = hv / (p.Hv / p.Hqk);
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int sub = lane & 7;
    const int row = part * kRecRowsPerCta + warp * 4 + (lane >> 3);

    const int t0 = p.cu_seqlens[n];
    const int t1 = p.cu_seqlens[n + 1];
    const bool first_ok = (n != 0) || (t0 == 0);
    const bool last_ok = (n != p.N - 1) || (t1 == p.T);
    if (t0 < 0 || t1 < t0 || t1 > p.T || !first_ok || !last_ok) {
        if (threadIdx.x == 0) report(p.dev_status, kDevBadCuSeqlens);
        return;
    }
    const int slot = p.slot_idx ? p.slot_idx[n] : n;
    if (slot < 0 || slot >= p.num_slots) {
        if (slot >= p.num_slots && threadIdx.x == 0) report(p.dev_status, kDevBadSlot);
        if (sub == 0)
            for (int t = t0; t < t1; ++t)
                p.o[(static_cast<size_t>(t) * p.Hv + hv) * kD + row] = __float2bfloat16(0.f);
        return;
    }

    const size_t tile_off = (static_cast<size_t>(slot) * p.Hv + hv) * (kD * kD) + row * kD;
    float4 s[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
        s[j] = p.init_state
                   ? *reinterpret_cast<const float4*>(p.init_state + tile_off + sub * 4 + j * 32)
                   : make_float4(0.f, 0.f, 0.f, 0.f);

    TokenRegs cur, nxt;
    if (t0 < t1) fetch_token(cur, p, t0, hqk, hv, sub, row);
    for (int t = t0; t < t1; ++t) {
        if (t + 1 < t1) fetch_token(nxt, p, t + 1, hqk, hv, sub, row);
        const float alpha = expf(cur.g);
        float pk = 0.f, pq = 0.f, kq = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            pk = dot4(s[j], cur.k[j], pk);
            pq = dot4(s[j], cur.q[j], pq);
            kq = dot4(cur.k[j], cur.q[j], kq);
        }
        pk = sum8(pk);
        pq = sum8(pq);
        kq = sum8(kq);
        const float w = cur.beta * (cur.v - alpha * pk);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            s[j].x = fmaf(w, cur.k[j].x, alpha * s[j].x);
            s[j].y = fmaf(w, cur.k[j].y, alpha * s[j].y);
            s[j].z = fmaf(w, cur.k[j].z, alpha * s[j].z);
            s[j].w = fmaf(w, cur.k[j].w, alpha * s[j].w);
        }
        if (sub == 0)
            p.o[(static_cast<size_t>(t) * p.Hv + hv) * kD + row] =
                __float2bfloat16(p.scale * fmaf(w, kq, alpha * pq));
        cur = nxt;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(p.final_state + tile_off + sub * 4 + j * 32) = s[j];
}

cudaError_t launch_prefill_recurrent(const PrefillParams& p, cudaStream_t stream) {
    const long long ctas = static_cast<long long>(p.N) * p.Hv * kRecCtasPerTile;
    if (ctas == 0 || p.T == 0) return cudaSuccess;
    prefill_recurrent_kernel<<<static_cast<unsigned>(ctas), kRecThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace gdn
