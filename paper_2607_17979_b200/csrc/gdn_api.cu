// C-ABI entry points: argument validation and launch.  See include/gdn.h.
#include "gdn_common.cuh"
#include "gdn_prefill_chunk.cuh"
#include "../../include/gdn.h"

namespace {

thread_local cudaError_t g_last_cuda_error = cudaSuccess;

// remember the runtime's own code behind a GDN_ERR_CUDA return
inline int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return GDN_OK;
    g_last_cuda_error = e;
    return GDN_ERR_CUDA;
}

inline bool misaligned(const void* p, size_t a) {
    return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0;
}

int check_heads(int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv) {
    if (Hqk <= 0 || Hv <= 0) return GDN_ERR_SIZE;
    if (dk != gdn::kD || dv != gdn::kD || Hv % Hqk != 0) return GDN_ERR_SHAPE;
    return GDN_OK;
}

int check_prefill(const void* q, const void* k, const void* v, const float* g, const float* beta,
                  const int32_t* cu, const float* init_state, float* final_state, void* o,
                  int32_t T, int32_t N, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                  int32_t num_slots) {
    if (T < 0 || N < 0) return GDN_ERR_SIZE;
    const int rc = check_heads(Hqk, Hv, dk, dv);
    if (rc != GDN_OK) return rc;
    if (T == 0 || N == 0) return GDN_OK;
    if (num_slots <= 0) return GDN_ERR_SIZE;
    if (!q || !k || !v || !g || !beta || !cu || !final_state || !o) return GDN_ERR_NULL;
    if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
        misaligned(final_state, 16) || misaligned(init_state, 16) || misaligned(g, 4) ||
        misaligned(beta, 4) || misaligned(cu, 4))
        return GDN_ERR_ALIGN;
    return GDN_OK;
}

}  // namespace

extern "C" {

int gdn_decode(const void* q, const void* k, const void* v, const float* g, const float* beta,
               float* state_pool, const int32_t* slot_idx, void* o,
               int32_t B, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
               int32_t num_slots, float scale, int32_t* dev_status, void* stream) {
    if (B < 0) return GDN_ERR_SIZE;
    const int rc = check_heads(Hqk, Hv, dk, dv);
    if (rc != GDN_OK) return rc;
    if (B == 0) return GDN_OK;
    if (num_slots <= 0) return GDN_ERR_SIZE;
    if (!q || !k || !v || !g || !beta || !state_pool || !o) return GDN_ERR_NULL;
    if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
        misaligned(state_pool, 16) || misaligned(g, 4) || misaligned(beta, 4) ||
        misaligned(slot_idx, 4) || misaligned(dev_status, 4))
        return GDN_ERR_ALIGN;
    gdn::DecodeParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.g = g; p.beta = beta; p.pool = state_pool; p.slot_idx = slot_idx;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.B = B; p.Hqk = Hqk; p.Hv = Hv; p.num_slots = num_slots; p.scale = scale;
    p.dev_status = dev_status;
    return cuda_status(gdn::launch_decode(p, static_cast<cudaStream_t>(stream)));
}

int gdn_decode_multi(const void* q, const void* k, const void* v, const float* g,
                     const float* beta, float* state_pool, const int32_t* slot_idx, void* o,
                     int32_t B, int32_t L, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                     int32_t num_slots, float scale, int32_t state_layout, int32_t* dev_status,
                     void* stream) {
    if (B < 0 || L < 0) return GDN_ERR_SIZE;
    const int rc = check_heads(Hqk, Hv, dk, dv);
    if (rc != GDN_OK) return rc;
    if (state_layout != GDN_STATE_VK && state_layout != GDN_STATE_KV) return GDN_ERR_SHAPE;
    if (L > GDN_DECODE_MAX_TOKENS) return GDN_ERR_LIMIT;
    if (B == 0 || L == 0) return GDN_OK;
    if (num_slots <= 0) return GDN_ERR_SIZE;
    if (!q || !k || !v || !g || !beta || !state_pool || !o) return GDN_ERR_NULL;
    if (misaligned(q, 16) || misaligned(k, 16) || misaligned(v, 16) || misaligned(o, 16) ||
        misaligned(state_pool, 16) || misaligned(g, 4) || misaligned(beta, 4) ||
        misaligned(slot_idx, 4) || misaligned(dev_status, 4))
        return GDN_ERR_ALIGN;
    gdn::DecodeMultiParams mp;
    gdn::DecodeParams& p = mp.d;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.g = g; p.beta = beta; p.pool = state_pool; p.slot_idx = slot_idx;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.B = B; p.Hqk = Hqk; p.Hv = Hv; p.num_slots = num_slots; p.scale = scale;
    p.dev_status = dev_status;
    mp.L = L;
    mp.layout = state_layout;
    return cuda_status(gdn::launch_decode_multi(mp, static_cast<cudaStream_t>(stream)));
}

int gdn_gate(const void* a, const void* b, const float* A_log, const float* dt_bias,
             float* g, float* beta, int32_t T, int32_t Hv, void* stream) {
    if (T < 0 || Hv < 0) return GDN_ERR_SIZE;
    if (T == 0 || Hv == 0) return GDN_OK;
    if (!a || !b || !A_log || !dt_bias || !g || !beta) return GDN_ERR_NULL;
    if (misaligned(a, 2) || misaligned(b, 2) || misaligned(A_log, 4) || misaligned(dt_bias, 4) ||
        misaligned(g, 4) || misaligned(beta, 4))
        return GDN_ERR_ALIGN;
    return cuda_status(gdn::launch_gate(static_cast<const __nv_bfloat16*>(a),
                                        static_cast<const __nv_bfloat16*>(b), A_log, dt_bias, g,
                                        beta, static_cast<long long>(T) * Hv, Hv,
                                        static_cast<cudaStream_t>(stream)));
}

int gdn_state_transpose(float* state_pool, const int32_t* slot_idx, int32_t n, int32_t Hv,
                        int32_t dk, int32_t dv, int32_t num_slots, int32_t* dev_status,
                        void* stream) {
    if (n < 0 || Hv < 0) return GDN_ERR_SIZE;
    if (dk != gdn::kD || dv != gdn::kD) return GDN_ERR_SHAPE;
    if (n == 0 || Hv == 0) return GDN_OK;
    if (num_slots <= 0) return GDN_ERR_SIZE;
    if (!state_pool) return GDN_ERR_NULL;
    if (misaligned(state_pool, 16) || misaligned(slot_idx, 4) || misaligned(dev_status, 4))
        return GDN_ERR_ALIGN;
    return cuda_status(gdn::launch_state_transpose(state_pool, slot_idx, n, Hv, num_slots,
                                                   dev_status, static_cast<cudaStream_t>(stream)));
}

size_t gdn_prefill_workspace_bytes(int32_t T, int32_t N, int32_t Hqk, int32_t Hv,
                                   int32_t dk, int32_t dv, int32_t chunk) {
    if (T < 0 || N < 0 || chunk != gdn::kChunk || check_heads(Hqk, Hv, dk, dv) != GDN_OK) return 0;
    return gdn::workspace_layout(T, N, Hv).total;
}

int gdn_prefill_recurrent(const void* q, const void* k, const void* v, const float* g,
                          const float* beta, const int32_t* cu_seqlens, const float* init_state,
                          float* final_state, const int32_t* slot_idx, void* o,
                          int32_t T, int32_t N, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                          int32_t num_slots, float scale, int32_t* dev_status, void* stream) {
    const int rc = check_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, o,
                                 T, N, Hqk, Hv, dk, dv, num_slots);
    if (rc != GDN_OK || T == 0 || N == 0) return rc;
    gdn::PrefillParams p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.g = g; p.beta = beta; p.cu_seqlens = cu_seqlens; p.init_state = init_state;
    p.final_state = final_state; p.slot_idx = slot_idx;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.T = T; p.N = N; p.Hqk = Hqk; p.Hv = Hv; p.num_slots = num_slots; p.scale = scale;
    p.dev_status = dev_status;
    return cuda_status(gdn::launch_prefill_recurrent(p, static_cast<cudaStream_t>(stream)));
}

namespace {
enum PrefillRoute { kRouteChunked, kRouteFused, kRouteStream, kRouteOverlap };

int prefill_chunked_impl(PrefillRoute route, const void* q, const void* k, const void* v, const float* g,
                         const float* beta, const int32_t* cu_seqlens, const float* init_state,
                         float* final_state, const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                         int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                         int32_t num_slots, float scale, void* workspace, size_t workspace_bytes,
                         int32_t* dev_status, void* stream, int32_t split_permille = -1) {
    if (chunk != gdn::kChunk) return GDN_ERR_SHAPE;
    const int rc = check_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, o,
                                 T, N, Hqk, Hv, dk, dv, num_slots);
    if (rc != GDN_OK || T == 0 || N == 0) return rc;
    if (!workspace) return GDN_ERR_NULL;
    if (misaligned(workspace, 256)) return GDN_ERR_ALIGN;
    if (workspace_bytes < gdn_prefill_workspace_bytes(T, N, Hqk, Hv, dk, dv, chunk))
        return GDN_ERR_WORKSPACE;
    gdn::ChunkedParams cp;
    gdn::PrefillParams& p = cp.p;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k = static_cast<const __nv_bfloat16*>(k);
    p.v = static_cast<const __nv_bfloat16*>(v);
    p.g = g; p.beta = beta; p.cu_seqlens = cu_seqlens; p.init_state = init_state;
    p.final_state = final_state; p.slot_idx = slot_idx;
    p.o = static_cast<__nv_bfloat16*>(o);
    p.T = T; p.N = N; p.Hqk = Hqk; p.Hv = Hv; p.num_slots = num_slots; p.scale = scale;
    p.dev_status = dev_status;
    cp.ws = static_cast<uint8_t*>(workspace);
    cp.lay = gdn::workspace_layout(T, N, Hv);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return cuda_status(route == kRouteFused     ? gdn::launch_prefill_fused(cp, st)
                       : route == kRouteStream  ? gdn::launch_prefill_stream(cp, st)
                       : route == kRouteOverlap ? gdn::launch_prefill_overlap(cp, st, split_permille)
                                                : gdn::launch_prefill_chunked(cp, st));
}
}  // namespace

int gdn_prefill_chunked(const void* q, const void* k, const void* v, const float* g,
                        const float* beta, const int32_t* cu_seqlens, const float* init_state,
                        float* final_state, const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                        int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                        int32_t chunk, int32_t num_slots, float scale, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, void* stream) {
    (void)max_seqlen_hint;
    return prefill_chunked_impl(kRouteChunked, q, k, v, g, beta, cu_seqlens, init_state, final_state,
                                slot_idx, o, T, N, Hqk, Hv, dk, dv, chunk, num_slots, scale,
                                workspace, workspace_bytes, dev_status, stream);
}

int gdn_prefill_fused(const void* q, const void* k, const void* v, const float* g,
                      const float* beta, const int32_t* cu_seqlens, const float* init_state,
                      float* final_state, const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                      int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                      int32_t chunk, int32_t num_slots, float scale, void* workspace,
                      size_t workspace_bytes, int32_t* dev_status, void* stream) {
    (void)max_seqlen_hint;
    return prefill_chunked_impl(kRouteFused, q, k, v, g, beta, cu_seqlens, init_state, final_state,
                                slot_idx, o, T, N, Hqk, Hv, dk, dv, chunk, num_slots, scale,
                                workspace, workspace_bytes, dev_status, stream);
}

int gdn_prefill_stream(const void* q, const void* k, const void* v, const float* g,
                       const float* beta, const int32_t* cu_seqlens, const float* init_state,
                       float* final_state, const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                       int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                       int32_t chunk, int32_t num_slots, float scale, void* workspace,
                       size_t workspace_bytes, int32_t* dev_status, void* stream) {
    (void)max_seqlen_hint;
    return prefill_chunked_impl(kRouteStream, q, k, v, g, beta, cu_seqlens, init_state, final_state,
                                slot_idx, o, T, N, Hqk, Hv, dk, dv, chunk, num_slots, scale,
                                workspace, workspace_bytes, dev_status, stream);
}

int gdn_prefill_overlap(const void* q, const void* k, const void* v, const float* g,
                        const float* beta, const int32_t* cu_seqlens, const float* init_state,
                        float* final_state, const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                        int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                        int32_t chunk, int32_t num_slots, float scale, void* workspace,
                        size_t workspace_bytes, int32_t* dev_status, void* stream,
                        int32_t split_permille) {
    (void)max_seqlen_hint;
    return prefill_chunked_impl(kRouteOverlap, q, k, v, g, beta, cu_seqlens, init_state, final_state,
                                slot_idx, o, T, N, Hqk, Hv, dk, dv, chunk, num_slots, scale,
                                workspace, workspace_bytes, dev_status, stream, split_permille);
}

int gdn_prefill_route(int32_t T, int32_t N, int32_t max_seqlen_hint, int32_t Hv, int32_t sm_count,
                      int32_t cooperative_launch) {
    if (T <= 0 || N <= 0 || Hv <= 0 || sm_count <= 0) return GDN_ROUTE_NONE;
    // the length is known on the host only through the caller's hint or the bound T
    const int32_t longest = (max_seqlen_hint > 0 && max_seqlen_hint < T) ? max_seqlen_hint : T;
    // very short sequences: the token-by-token kernel (one launch, no workspace traffic)
    if (longest <= GDN_RECURRENT_MAX_SEQLEN) return GDN_ROUTE_RECURRENT;
    const long long units = static_cast<long long>(N) * Hv;
    // Few (sequence, v-head) units and long sequences: the serial state pass would occupy only a
    // few SMs while the rest idle, so run it next to the record producers in one cooperative launch.
    if (cooperative_launch && units <= sm_count / 3 && longest > 16 * gdn::kChunk) return GDN_ROUTE_FUSED;
    // More units than the cooperative launch takes but at most half as many as SMs, with long
    // chains (known only through the caller's hint): the state pass leaves half the machine free
    // from the start, so part of the records is produced beside it (two sequences of 4096 tokens
    // at 32 heads 261 -> 238 us, 4096 + 2048 230 -> 198 us, 8192 + 1024 382 -> 303 us; two chains of
    // 32 chunks were 4 % slower, hence 40).  That route wants two launches to run side by side,
    // which the device does but CUDA does not promise; if they do not, its last launch finishes
    // the work (same results, milliseconds lost), so choosing it is safe.  Below a third of the
    // SMs the cooperative launch is level with it or ahead; batches that fill the machine at
    // first and free it as their short chains end would gain 5-12 %, but the records produced late
    // are still dirty in L2 when the call ends and their write-back falls into whatever runs
    // next, and batches of equal chains lose up to 7 %: those stay with the persistent pass.
    if (max_seqlen_hint > 0 && units <= sm_count / 2 && longest >= 40 * gdn::kChunk)
        return GDN_ROUTE_OVERLAP;
    // Everything else: the three launches (table kernel, or none for small batches; the intra-chunk
    // kernel over all items; the persistent state pass).
    return GDN_ROUTE_STREAM;
}

int gdn_prefill(const void* q, const void* k, const void* v, const float* g, const float* beta,
                const int32_t* cu_seqlens, const float* init_state, float* final_state,
                const int32_t* slot_idx, void* o, int32_t T, int32_t N, int32_t max_seqlen_hint,
                int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                int32_t num_slots, float scale, void* workspace, size_t workspace_bytes,
                int32_t* dev_status, void* stream) {
    int sms = 148, coop = 0;
    gdn::DeviceInfo di;
    if (gdn::device_info(&di) == cudaSuccess) {
        sms = di.sms;
        coop = di.cooperative;
    }
    const int route_id = gdn_prefill_route(T, N, max_seqlen_hint, Hv, sms, coop);
    if (chunk == gdn::kChunk && route_id == GDN_ROUTE_RECURRENT) {
        // same validation of the workspace arguments as the chunked route, so that a call does
        // not start failing when its batch grows
        if (!workspace) {
            const int rc = check_prefill(q, k, v, g, beta, cu_seqlens, init_state, final_state, o,
                                         T, N, Hqk, Hv, dk, dv, num_slots);
            return rc != GDN_OK ? rc : GDN_ERR_NULL;
        }
        if (misaligned(workspace, 256)) return GDN_ERR_ALIGN;
        if (workspace_bytes < gdn_prefill_workspace_bytes(T, N, Hqk, Hv, dk, dv, chunk))
            return check_heads(Hqk, Hv, dk, dv) != GDN_OK ? check_heads(Hqk, Hv, dk, dv)
                                                          : GDN_ERR_WORKSPACE;
        return gdn_prefill_recurrent(q, k, v, g, beta, cu_seqlens, init_state, final_state,
                                     slot_idx, o, T, N, Hqk, Hv, dk, dv, num_slots, scale,
                                     dev_status, stream);
    }
    const PrefillRoute route = route_id == GDN_ROUTE_FUSED     ? kRouteFused
                               : route_id == GDN_ROUTE_STREAM  ? kRouteStream
                               : route_id == GDN_ROUTE_OVERLAP ? kRouteOverlap
                                                               : kRouteChunked;
    return prefill_chunked_impl(route, q, k, v, g, beta, cu_seqlens, init_state,
                                final_state, slot_idx, o, T, N, Hqk, Hv, dk, dv, chunk, num_slots,
                                scale, workspace, workspace_bytes, dev_status, stream);
}


// ---------------------------------------------------------------------------------------------
// Host-buffer variants: per-call tensors live in (preferably pinned) host memory; they are copied
// into a caller-provided device staging buffer, the device entry point runs, and o is copied
// back, all enqueued on `stream`.
// ---------------------------------------------------------------------------------------------
namespace {
struct Staging {
    size_t q, k, v, g, beta, idx, o, total;
};
inline size_t up256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }
Staging staging_layout(int64_t rows, int32_t Hqk, int32_t Hv, int64_t n_idx) {
    Staging s;
    size_t off = 0;
    s.q = off; off += up256(static_cast<size_t>(rows) * Hqk * gdn::kD * 2);
    s.k = off; off += up256(static_cast<size_t>(rows) * Hqk * gdn::kD * 2);
    s.v = off; off += up256(static_cast<size_t>(rows) * Hv * gdn::kD * 2);
    s.g = off; off += up256(static_cast<size_t>(rows) * Hv * 4);
    s.beta = off; off += up256(static_cast<size_t>(rows) * Hv * 4);
    s.idx = off; off += up256(static_cast<size_t>(n_idx) * 4);
    s.o = off; off += up256(static_cast<size_t>(rows) * Hv * gdn::kD * 2);
    s.total = off;
    return s;
}
}  // namespace

size_t gdn_decode_host_staging_bytes(int32_t B, int32_t Hqk, int32_t Hv) {
    if (B < 0 || Hqk <= 0 || Hv <= 0) return 0;
    return staging_layout(B, Hqk, Hv, B).total;
}

int gdn_decode_host(const void* q, const void* k, const void* v, const float* g, const float* beta,
                    float* state_pool, const int32_t* slot_idx, void* o,
                    int32_t B, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t num_slots,
                    float scale, void* staging, size_t staging_bytes, int32_t* dev_status,
                    void* stream) {
    if (B < 0) return GDN_ERR_SIZE;
    const int rc = check_heads(Hqk, Hv, dk, dv);
    if (rc != GDN_OK) return rc;
    if (B == 0) return GDN_OK;
    if (!q || !k || !v || !g || !beta || !state_pool || !o || !staging) return GDN_ERR_NULL;
    if (misaligned(staging, 256)) return GDN_ERR_ALIGN;
    const Staging s = staging_layout(B, Hqk, Hv, B);
    if (staging_bytes < s.total) return GDN_ERR_WORKSPACE;
    uint8_t* d = static_cast<uint8_t*>(staging);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qk = static_cast<size_t>(B) * Hqk * gdn::kD * 2, vo = static_cast<size_t>(B) * Hv * gdn::kD * 2;
    const size_t sc = static_cast<size_t>(B) * Hv * 4;
    cudaError_t e = cudaMemcpyAsync(d + s.q, q, qk, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.k, k, qk, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.v, v, vo, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.g, g, sc, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.beta, beta, sc, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && slot_idx)
        e = cudaMemcpyAsync(d + s.idx, slot_idx, static_cast<size_t>(B) * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_status(e);
    const int r = gdn_decode(d + s.q, d + s.k, d + s.v, reinterpret_cast<const float*>(d + s.g),
                             reinterpret_cast<const float*>(d + s.beta), state_pool,
                             slot_idx ? reinterpret_cast<const int32_t*>(d + s.idx) : nullptr,
                             d + s.o, B, Hqk, Hv, dk, dv, num_slots, scale, dev_status, stream);
    if (r != GDN_OK) return r;
    return cuda_status(cudaMemcpyAsync(o, d + s.o, vo, cudaMemcpyDeviceToHost, st));
}

size_t gdn_prefill_host_staging_bytes(int32_t T, int32_t N, int32_t Hqk, int32_t Hv) {
    if (T < 0 || N < 0 || Hqk <= 0 || Hv <= 0) return 0;
    return staging_layout(T, Hqk, Hv, 2 * static_cast<int64_t>(N) + 1).total;
}

int gdn_prefill_host(const void* q, const void* k, const void* v, const float* g, const float* beta,
                     const int32_t* cu_seqlens, const float* init_state, float* final_state,
                     const int32_t* slot_idx, void* o, int32_t T, int32_t N,
                     int32_t max_seqlen_hint, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                     int32_t chunk, int32_t num_slots, float scale, void* staging,
                     size_t staging_bytes, void* workspace, size_t workspace_bytes,
                     int32_t* dev_status, void* stream) {
    if (T < 0 || N < 0) return GDN_ERR_SIZE;
    const int rc = check_heads(Hqk, Hv, dk, dv);
    if (rc != GDN_OK) return rc;
    if (T == 0 || N == 0) return GDN_OK;
    if (!q || !k || !v || !g || !beta || !cu_seqlens || !final_state || !o || !staging)
        return GDN_ERR_NULL;
    if (misaligned(staging, 256)) return GDN_ERR_ALIGN;
    const Staging s = staging_layout(T, Hqk, Hv, 2 * static_cast<int64_t>(N) + 1);
    if (staging_bytes < s.total) return GDN_ERR_WORKSPACE;
    uint8_t* d = static_cast<uint8_t*>(staging);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t qk = static_cast<size_t>(T) * Hqk * gdn::kD * 2, vo = static_cast<size_t>(T) * Hv * gdn::kD * 2;
    const size_t sc = static_cast<size_t>(T) * Hv * 4;
    int32_t* d_cu = reinterpret_cast<int32_t*>(d + s.idx);
    int32_t* d_slot = d_cu + (N + 1);
    cudaError_t e = cudaMemcpyAsync(d + s.q, q, qk, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.k, k, qk, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.v, v, vo, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.g, g, sc, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(d + s.beta, beta, sc, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(d_cu, cu_seqlens, static_cast<size_t>(N + 1) * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && slot_idx)
        e = cudaMemcpyAsync(d_slot, slot_idx, static_cast<size_t>(N) * 4, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return cuda_status(e);
    const int r = gdn_prefill(d + s.q, d + s.k, d + s.v, reinterpret_cast<const float*>(d + s.g),
                              reinterpret_cast<const float*>(d + s.beta), d_cu, init_state,
                              final_state, slot_idx ? d_slot : nullptr, d + s.o, T, N,
                              max_seqlen_hint, Hqk, Hv, dk, dv, chunk, num_slots, scale, workspace,
                              workspace_bytes, dev_status, stream);
    if (r != GDN_OK) return r;
    return cuda_status(cudaMemcpyAsync(o, d + s.o, vo, cudaMemcpyDeviceToHost, st));
}

const char* gdn_status_string(int code) {
    switch (code) {
        case GDN_OK: return "ok";
        case GDN_ERR_NULL: return "a required pointer is NULL";
        case GDN_ERR_SIZE: return "a size is negative or num_slots is not positive";
        case GDN_ERR_SHAPE: return "unsupported shape (need dk = dv = 128, chunk = 64, Hv % Hqk = 0)";
        case GDN_ERR_ALIGN: return "a pointer is not aligned as required";
        case GDN_ERR_WORKSPACE: return "workspace too small";
        case GDN_ERR_CUDA: return "CUDA runtime error at launch or set-up";
        case GDN_ERR_LIMIT: return "a size exceeds the entry point's fixed maximum";
        default: return "unknown status";
    }
}

const char* gdn_last_cuda_error_string(void) { return cudaGetErrorString(g_last_cuda_error); }

int gdn_version(void) { return 100; }

}  // extern "C"
