// Chunked prefill on the sm_100a tensor cores (tcgen05 + TMEM, operands staged by TMA): the
// intra-chunk kernel and the host side shared by the launchers.
// The algebra and the record layout are described in gdn_prefill_chunk.cuh.
#include "gdn_prefill_device.cuh"

namespace gdn {

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

// The three-launch path: table-building launch (none for small batches), the intra-chunk kernel
// over all items, the persistent state pass.
cudaError_t launch_prefill_chunked(const ChunkedParams& cp, cudaStream_t stream) {
    return launch_prefill_stream(cp, stream);
}

}  // namespace gdn
