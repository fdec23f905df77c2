// Gate / beta preprocessing in front of prefill and decode: raw per-token projections to the
// log-domain gate g = ln(alpha) and the write strength beta the recurrence takes.
//
//   g[t][h]    = -exp(A_log[h]) * softplus(a[t][h] + dt_bias[h])      (<= 0, so alpha in (0, 1])
//   beta[t][h] = sigmoid(b[t][h])
//
// The paper names such a helper but prints no formula; this is the parametrisation of the
// published Gated DeltaNet layer.  Element-wise, fp32, one thread per (token, head).
#include "gdn_common.cuh"

namespace gdn {

__global__ void __launch_bounds__(256)
gate_kernel(const __nv_bfloat16* __restrict__ a, const __nv_bfloat16* __restrict__ b,
            const float* __restrict__ A_log, const float* __restrict__ dt_bias,
            float* __restrict__ g, float* __restrict__ beta, long long n, int Hv) {
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= n) return;
    const int h = static_cast<int>(idx % Hv);
    const float x = __bfloat162float(a[idx]) + dt_bias[h];
    const float softplus = fmaxf(x, 0.f) + log1pf(expf(-fabsf(x)));
    g[idx] = -expf(A_log[h]) * softplus;
    beta[idx] = 1.f / (1.f + expf(-__bfloat162float(b[idx])));
}

cudaError_t launch_gate(const __nv_bfloat16* a, const __nv_bfloat16* b, const float* A_log,
                        const float* dt_bias, float* g, float* beta, long long n, int Hv,
                        cudaStream_t stream) {
    if (n == 0) return cudaSuccess;
    gate_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, stream>>>(a, b, A_log, dt_bias, g,
                                                                           beta, n, Hv);
    return cudaGetLastError();
}

}  // namespace gdn
