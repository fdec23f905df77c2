// Shared declarations of the CUDA side of the gated delta rule library.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

namespace gdn {

constexpr int kD = 128;          // dk == dv == 128 is the only supported head size
constexpr int kChunk = 64;       // prefill chunk length
constexpr int kDecodeMaxTokens = 16;  // most new tokens per sequence in one multi-token decode

// device status bits (mirror GDN_DEV_* of the public header)
constexpr int kDevBadSlot = 1;
constexpr int kDevBadCuSeqlens = 2;
constexpr int kDevTimeout = 4;

struct DecodeParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const float* g;
    const float* beta;
    float* pool;
    const int32_t* slot_idx;
    __nv_bfloat16* o;
    int32_t B, Hqk, Hv, num_slots;
    float scale;
    int32_t* dev_status;
};

struct DecodeMultiParams {
    DecodeParams d;      // q,k [B][L][Hqk][128]; v,o [B][L][Hv][128]; g,beta [B][L][Hv]
    int32_t L;           // new tokens per sequence, 1..kDecodeMaxTokens
    int32_t layout;      // 0: tile [dv][dk];  1: tile [dk][dv]
};

struct PrefillParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    const float* g;
    const float* beta;
    const int32_t* cu_seqlens;
    const float* init_state;
    float* final_state;
    const int32_t* slot_idx;
    __nv_bfloat16* o;
    int32_t T, N, Hqk, Hv, num_slots;
    float scale;
    int32_t* dev_status;
};

// The current device's SM count and cooperative-launch support, queried once per device.
struct DeviceInfo {
    int device, sms, cooperative;
};
cudaError_t device_info(DeviceInfo* out);
// Raises a kernel's dynamic shared memory limit on the current device, once per device.
cudaError_t ensure_dynamic_smem(const void* kernel, int bytes);
template <class K> inline cudaError_t ensure_dynamic_smem(K* kernel, int bytes) {
    return ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), bytes);
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t stream);
cudaError_t launch_decode_multi(const DecodeMultiParams& mp, cudaStream_t stream);
cudaError_t launch_gate(const __nv_bfloat16* a, const __nv_bfloat16* b, const float* A_log,
                        const float* dt_bias, float* g, float* beta, long long n, int Hv,
                        cudaStream_t stream);
cudaError_t launch_state_transpose(float* pool, const int32_t* slot_idx, int32_t n, int32_t Hv,
                                   int32_t num_slots, int32_t* dev_status, cudaStream_t stream);
cudaError_t launch_prefill_recurrent(const PrefillParams& p, cudaStream_t stream);

__device__ __forceinline__ void report(int32_t* dev_status, int bit) {
    if (dev_status) atomicOr(dev_status, bit);
}

// four consecutive bf16 -> four floats (8-byte aligned source)
__device__ __forceinline__ float4 load_bf16x4(const __nv_bfloat16* p) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    float4 r;
    r.x = __uint_as_float(raw.x << 16);
    r.y = __uint_as_float(raw.x & 0xffff0000u);
    r.z = __uint_as_float(raw.y << 16);
    r.w = __uint_as_float(raw.y & 0xffff0000u);
    return r;
}

__device__ __forceinline__ float dot4(const float4& a, const float4& b, float acc) {
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
    return acc;
}

// sum over the 8 lanes that share a state row (lanes differing in bits 0..2)
__device__ __forceinline__ float sum8(float x) {
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    x += __shfl_xor_sync(0xffffffffu, x, 4);
    return x;
}

}  // namespace gdn
