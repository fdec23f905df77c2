// Chunked prefill: shared layout of the workspace and of the per-(chunk, v-head) record.
//
// Inside a chunk of C = 64 tokens entering with state S0 (dv x dk), with
// b_r = sum_{i<=r} g_i (inclusive, chunk-local) the gated delta rule unrolls to
//
//   A_ri = beta_r e^{b_r-b_i} (k_r.k_i)  (i <  r),   T = (I + A)^{-1}
//   P_ri =        e^{b_r-b_i} (q_r.k_i)  (i <= r)
//   W  = T diag(beta e^b) K   (C x dk),   U~ = T diag(beta) V   (C x dv)
//   U  = U~ - W S0^T
//   O  = scale ( diag(e^b) Q S0^T + P U )  =  scale ( Qg S0^T + P U ),  Qg = diag(e^b) Q
//   S' = e^{b_C} S0 + U^T diag(e^{b_C-b}) K
//
// Three launches: a prep kernel builds the chunk table from cu_seqlens; the
// intra-chunk kernel (one CTA per chunk and v-head, all chunks in parallel)
// computes W, U~, P and b with tcgen05 GEMMs and an fp32 triangular solve and
// writes them as a record; the state-pass kernel (one CTA per sequence and
// v-head, or one persistent CTA per SM walking a list of them) walks the chunks
// in order carrying S in fp32 registers.  A fused variant runs the last two as
// one cooperative launch.
#pragma once
#include "gdn_common.cuh"
#include <cuda.h>

namespace gdn {

// One record per (chunk, v-head), written by the intra-chunk kernel in exactly the
// byte image the state-pass kernel wants in shared memory (one linear bulk copy):
//   [0, 16384)      W   as one MN-major 128B-swizzled tile [128 dk][64 tokens] bf16 (a row per dk)
//   [16384, 32768)  Qg  = diag(e^b) Q as two K-major 128B-swizzled halves [64 tokens][64 dk] bf16
//                   (the output's first term S0 Qg^T)
//   [32768, 40960)  P   as one K-major 128B-swizzled tile   [64 r][64 i]      bf16
//   [40960, 73728)  U~  as [16 token-groups][128 dv][4 tokens] fp32
//   [73728, 73984)  e^{b_C - b_c} for c = 0..63, fp32 (rows past the chunk's length hold 1)
//   [73984, 74240)  e^{b_C} in the first float, rest unused
constexpr uint32_t kRecW = 0;
constexpr uint32_t kRecQg = 16384;
constexpr uint32_t kRecP = 32768;
constexpr uint32_t kRecU = 40960;
constexpr uint32_t kRecDecay = 73728;
constexpr uint32_t kRecGammaC = 73984;
constexpr uint32_t kRecBytes = 74240;

// Small batches of at most this many sequences need no table-building launch: the intra-chunk
// kernel finds its chunks from cu_seqlens itself and writes the per-sequence tables for the state pass.
constexpr int kInlineTableSeqs = 16;
constexpr int kInlineTableItems = 2 * 148 * 4;     // and at most about two waves of (chunk, v-head) CTAs

struct ChunkInfo {      // 16 bytes
    int32_t seq;        // sequence the chunk belongs to
    int32_t t0;         // first packed token of the chunk
    int32_t len;        // valid tokens (1..64)
    int32_t pad;
};

// Workspace layout (all offsets multiples of 256 bytes):
//   [0,256)                      int32 header: [0] total_chunks, [1] total_items
//                                (= total_chunks * Hv), [2] item queue head, [3] unit queue head,
//                                [4] items produced before the state pass starts (two-part route)
//   seq_first[N+1]               int32: first chunk of each sequence (prefix sum); an invalid
//                                sequence has zero chunks and seq_bad[n] = 1
//   seq_bad[N]                   int32
//   chunks[max_chunks]           ChunkInfo
//   -- used by the fused single-launch path only --
//   seq_by_rank[N]               int32: sequences sorted by chunk count, longest first
//   rank_of[N]                   int32: the inverse (rank of each sequence)
//   order[max_chunks]            int32: chunk ids in processing order: by position inside the
//                                sequence first, by sequence rank second (so that the records
//                                every state-pass unit needs next are produced first)
//   hist, fill, cnt, pos[max_nc+2]  int32 scratch of the counting sort (max_nc = T/64 + 1)
//   flags[max_chunks][Hv]        uint32: 1 once the record is complete and visible
//   done[N][Hv]                  int32: 1 once the two-part route's state pass has finished the unit
//                                (rank-major, like the unit list); the rest is left to a last launch
//   -- both paths --
//   records[max_chunks][Hv]      kRecBytes each
struct WorkspaceLayout {
    size_t seq_first, seq_bad, chunks, seq_by_rank, rank_of, order, hist, fill, cnt, pos, flags,
        done, records, total;
    int32_t max_chunks, max_nc;
};

constexpr int kHdrTotalChunks = 0, kHdrTotalItems = 1, kHdrItemHead = 2, kHdrUnitHead = 3,
              kHdrSplit = 4;

inline size_t round256(size_t x) { return (x + 255) & ~static_cast<size_t>(255); }

inline WorkspaceLayout workspace_layout(int32_t T, int32_t N, int32_t Hv) {
    WorkspaceLayout w;
    w.max_chunks = T / kChunk + N;
    w.max_nc = T / kChunk + 1;
    const size_t nchunks = static_cast<size_t>(w.max_chunks ? w.max_chunks : 1);
    const size_t nbins = round256(sizeof(int32_t) * (static_cast<size_t>(w.max_nc) + 2));
    w.seq_first = 256;
    w.seq_bad = w.seq_first + round256(sizeof(int32_t) * (static_cast<size_t>(N) + 1));
    w.chunks = w.seq_bad + round256(sizeof(int32_t) * static_cast<size_t>(N ? N : 1));
    w.seq_by_rank = w.chunks + round256(sizeof(ChunkInfo) * nchunks);
    w.rank_of = w.seq_by_rank + round256(sizeof(int32_t) * static_cast<size_t>(N ? N : 1));
    w.order = w.rank_of + round256(sizeof(int32_t) * static_cast<size_t>(N ? N : 1));
    w.hist = w.order + round256(sizeof(int32_t) * nchunks);
    w.fill = w.hist + nbins;
    w.cnt = w.fill + nbins;
    w.pos = w.cnt + nbins;
    w.flags = w.pos + nbins;
    w.done = w.flags + round256(sizeof(uint32_t) * nchunks * Hv);
    w.records = w.done + round256(sizeof(int32_t) * static_cast<size_t>(N ? N : 1) * Hv);
    w.total = w.records + static_cast<size_t>(w.max_chunks) * Hv * kRecBytes;
    return w;
}

struct ChunkedParams {
    PrefillParams p;
    uint8_t* ws;
    WorkspaceLayout lay;
};

cudaError_t launch_prefill_chunked(const ChunkedParams& cp, cudaStream_t stream);
// One cooperative launch: some CTAs produce the records, the others run the state pass behind them.
cudaError_t launch_prefill_fused(const ChunkedParams& cp, cudaStream_t stream);
// Three launches with a persistent state pass: CTAs walk lists of (sequence, v-head) units and
// stream their records without draining between units (for batches with many more units than SMs).
cudaError_t launch_prefill_stream(const ChunkedParams& cp, cudaStream_t stream);
// Pieces shared by the launchers: the prep kernel that also ranks the sequences by chunk count
// (longest first) and, for the fused launch, orders the chunks and clears the queues and flags;
// the intra-chunk kernel over all items.
// mode 0: chunk table and ranking; 1: + processing order, cleared queue heads and flags (fused
// launch); 2: + the cut of the two-part production (split_permille < 0: the kernel's own model).
cudaError_t launch_prefill_ranked_prep(const ChunkedParams& cp, cudaStream_t stream, int mode,
                                       int split_permille = -1, int sms = 0);
// The intra-chunk kernel in two parts around a flag-gated persistent state pass: the second part
// of the records is produced beside the chains, on the SMs the state pass leaves free.
cudaError_t launch_prefill_overlap(const ChunkedParams& cp, cudaStream_t stream, int split_permille);

}  // namespace gdn
