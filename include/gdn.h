/*
 * gdn.h - C ABI of the B200 (sm_100a) gated delta rule library.
 *
 * Operator (paper, appendix "Operator Background and Mathematical Definitions",
 * subsection "Gated Delta Net", the gated delta rule):
 *
 *     S_t = S_{t-1} ( alpha_t ( I - beta_t k_t k_t^T ) ) + beta_t v_t k_t^T
 *     o_t = scale * S_t q_t                  (the paper writes it with scale = 1)
 *
 * S is a dv x dk matrix state per (sequence, v-head); alpha_t = exp(g_t) is the
 * log-domain ("natural-log") gate the same subsection describes.  The paper's
 * two execution regimes are the two entry points: decode (a prior state plus
 * one new token) and prefill (whole packed sequences, outputs plus final state,
 * evaluated through chunked matrix operations).
 *
 * Conventions fixed by this library (the paper leaves them open):
 *   - grouped heads: v-head hv uses q/k head  hv / (Hv / Hqk);  Hv % Hqk == 0.
 *   - a state tile is row-major [dv][dk], dk contiguous, fp32.
 *   - q, k, v, o are bf16 (raw 16-bit), g and beta fp32, all contiguous.
 *   - only dk == dv == 128 and chunk == 64 are supported.
 *
 * Common rules for every call below
 *   - Every pointer is DEVICE memory owned by the caller unless a comment says
 *     "host".  The library allocates nothing and keeps no state between calls
 *     except where an entry point's own comment says otherwise (and except a few
 *     facts about each device, looked up on first use and remembered: its SM
 *     count, whether it launches cooperatively, which kernels had their shared
 *     memory limit raised).
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return
 *     without synchronising.  No device data is read on the host.
 *   - Return value: 0 = enqueued; negative = rejected before any launch and
 *     nothing was written (see GDN_ERR_*).
 *   - Problems only the device can see set bits in *dev_status (device int32,
 *     may be NULL; bits are OR-ed in, never cleared by the library) and the
 *     offending unit is skipped; the kernels never trap.
 */
#ifndef GDN_B200_H_
#define GDN_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GDN_OK                 0
#define GDN_ERR_NULL          -1  /* a required pointer is NULL                              */
#define GDN_ERR_SIZE          -2  /* a negative size, or num_slots <= 0 with work to do       */
#define GDN_ERR_SHAPE         -3  /* dk, dv != 128, chunk != 64, Hv % Hqk != 0, ...           */
#define GDN_ERR_ALIGN         -4  /* q/k/v/o/state/workspace not 16-byte aligned              */
#define GDN_ERR_WORKSPACE     -5  /* workspace_bytes smaller than the size query answers      */
#define GDN_ERR_CUDA          -6  /* the CUDA runtime refused a launch or a set-up call       */
#define GDN_ERR_LIMIT         -7  /* a size exceeds a fixed maximum stated by the entry point */

#define GDN_DEV_BAD_SLOT       1  /* a slot index >= num_slots was skipped                    */
#define GDN_DEV_BAD_CU_SEQLENS 2  /* cu_seqlens not non-decreasing from 0 to T; unit skipped   */
#define GDN_DEV_TIMEOUT        4  /* a bounded wait inside a kernel gave up                   */

/*
 * gdn_decode - one token of the gated delta rule for each of B sequences
 * (paper, subsection "Gated Delta Net", the decode regime: a prior state plus a
 * few new updates; here exactly one update per sequence per call).
 *
 * For entry i and v-head hv, with slot = slot_idx ? slot_idx[i] : i and the
 * tile S = state_pool[slot][hv]:
 *     S <- exp(g) S ;  u = S k ;  S <- S + beta (v - u) k^T ;  o = scale S q
 * The tile is read once and written back in place; o is rounded to bf16.
 *
 *   q, k        bf16 [B][Hqk][dk]
 *   v           bf16 [B][Hv][dv]
 *   g, beta     fp32 [B][Hv]          g = ln(alpha)
 *   state_pool  fp32 [num_slots][Hv][dv][dk], updated in place
 *   slot_idx    int32 [B] or NULL.  A negative index is a padding entry: its
 *               o rows are zero and no state is touched.  An index >=
 *               num_slots does the same and sets GDN_DEV_BAD_SLOT.  Two
 *               entries naming the same slot in one call race (undefined).
 *   o           bf16 [B][Hv][dv], written
 * B == 0 is a no-op that returns 0.
 */
int gdn_decode(const void* q, const void* k, const void* v,
               const float* g, const float* beta,
               float* state_pool, const int32_t* slot_idx, void* o,
               int32_t B, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
               int32_t num_slots, float scale,
               int32_t* dev_status, void* stream);

/*
 * gdn_decode_multi - L >= 1 new tokens of the gated delta rule for each of B
 * sequences in one call, applied in order, with a choice of state orientation
 * (paper, same subsection: the decode regime applies a few new updates to a
 * prior state, and the paper's decode routes differ in how the state tile is
 * laid out, one of them working on the transposed tile).  The result equals L successive gdn_decode
 * calls; the state tile is read and written once for all L tokens.
 *
 *   q, k        bf16 [B][L][Hqk][dk]
 *   v           bf16 [B][L][Hv][dv]
 *   g, beta     fp32 [B][L][Hv]
 *   state_pool  fp32, updated in place:
 *                 state_layout == GDN_STATE_VK: [num_slots][Hv][dv][dk] (as gdn_decode)
 *                 state_layout == GDN_STATE_KV: [num_slots][Hv][dk][dv] (the transposed tile)
 *   slot_idx    int32 [B] or NULL, rules as in gdn_decode (a padding entry's
 *               L o rows are zero)
 *   o           bf16 [B][L][Hv][dv], written
 * L > GDN_DECODE_MAX_TOKENS returns GDN_ERR_LIMIT; another state_layout value
 * returns GDN_ERR_SHAPE; B == 0 or L == 0 is a no-op that returns 0.
 */
#define GDN_DECODE_MAX_TOKENS 16
#define GDN_STATE_VK 0
#define GDN_STATE_KV 1
int gdn_decode_multi(const void* q, const void* k, const void* v,
                     const float* g, const float* beta,
                     float* state_pool, const int32_t* slot_idx, void* o,
                     int32_t B, int32_t L, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                     int32_t num_slots, float scale, int32_t state_layout,
                     int32_t* dev_status, void* stream);

/*
 * gdn_gate - the scalar gate / beta preprocessing in front of the recurrence
 * (paper: the prefill route keeps a small fused helper that prepares the gate
 * and beta inputs; the paper prints no formula for it).  Reading taken: the
 * parametrisation of the published Gated DeltaNet layer,
 *     g[t][h]    = -exp(A_log[h]) * softplus(a[t][h] + dt_bias[h])
 *     beta[t][h] = sigmoid(b[t][h])
 * so that g <= 0 (alpha = exp(g) in (0, 1]) and beta in (0, 1).
 *
 *   a, b        bf16 [T][Hv]   raw per-token projections
 *   A_log       fp32 [Hv]      per-head log decay rate
 *   dt_bias     fp32 [Hv]      per-head bias
 *   g, beta     fp32 [T][Hv], written: the g and beta arguments of gdn_prefill /
 *               gdn_decode (T = B for a decode step)
 * T == 0 is a no-op that returns 0.
 */
int gdn_gate(const void* a, const void* b, const float* A_log, const float* dt_bias,
             float* g, float* beta, int32_t T, int32_t Hv, void* stream);

/*
 * gdn_state_transpose - transpose, in place, the 128 x 128 state tiles of n
 * entries (all Hv heads each): [dv][dk] becomes [dk][dv] and back.  It lets a
 * pool kept in the GDN_STATE_KV orientation go through gdn_prefill (which
 * reads and writes GDN_STATE_VK tiles): transpose the touched slots, prefill,
 * transpose again.  (The paper names the transposed-state decode route but no
 * such helper; this is this library's addition.)
 *
 *   state_pool  fp32 [num_slots][Hv][128][128], tiles transposed in place
 *   slot_idx    int32 [n] or NULL (= slots 0..n-1); negative entries are
 *               skipped, entries >= num_slots are skipped and set
 *               GDN_DEV_BAD_SLOT; a slot listed twice is undefined
 * n == 0 is a no-op that returns 0.
 */
int gdn_state_transpose(float* state_pool, const int32_t* slot_idx, int32_t n, int32_t Hv,
                        int32_t dk, int32_t dv, int32_t num_slots,
                        int32_t* dev_status, void* stream);

/*
 * gdn_prefill_workspace_bytes - device scratch gdn_prefill needs for a packed
 * batch of at most T tokens in at most N sequences.  Returns 0 for shapes
 * gdn_prefill would reject.
 */
size_t gdn_prefill_workspace_bytes(int32_t T, int32_t N, int32_t Hqk, int32_t Hv,
                                   int32_t dk, int32_t dv, int32_t chunk);

/*
 * gdn_prefill - the same recurrence over N packed variable-length sequences
 * (paper, subsection "Gated Delta Net", the prefill regime: whole sequences in,
 * outputs and final state out, the recurrence evaluated chunk by chunk as
 * matrix products with the gate kept in the log domain).  The result is
 * the token-by-token recurrence's; chunking only re-associates it.
 *
 * Sequence n owns tokens cu_seqlens[n] .. cu_seqlens[n+1]-1 and the state tile
 * slot = slot_idx ? slot_idx[n] : n.  Chunks of `chunk` tokens restart at every
 * sequence start; the last chunk of a sequence may be short; a sequence may be
 * empty (its final state is its initial state).
 *
 *   q, k         bf16 [T][Hqk][dk]     packed tokens
 *   v            bf16 [T][Hv][dv]
 *   g, beta      fp32 [T][Hv]
 *   cu_seqlens   int32 [N+1], cu[0] = 0, non-decreasing, cu[N] = T (checked on
 *                the device: a violating sequence is skipped and
 *                GDN_DEV_BAD_CU_SEQLENS is set)
 *   init_state   fp32 [num_slots][Hv][dv][dk] or NULL (= all-zero states)
 *   final_state  fp32 [num_slots][Hv][dv][dk], written for every slot a
 *                sequence maps to; may be the same buffer as init_state
 *   slot_idx     int32 [N] or NULL; negative = padding sequence (o rows zero,
 *                no state written); >= num_slots the same + GDN_DEV_BAD_SLOT
 *   o            bf16 [T][Hv][dv], written
 *   max_seqlen_hint  an upper bound on the longest sequence if the caller
 *                knows one, else 0; only steers launch geometry, never results
 *   workspace    device scratch of at least gdn_prefill_workspace_bytes(...)
 *                bytes, 256-byte aligned; contents are scratch before and after
 * T == 0 or N == 0 is a no-op that returns 0.
 */
int gdn_prefill(const void* q, const void* k, const void* v,
                const float* g, const float* beta, const int32_t* cu_seqlens,
                const float* init_state, float* final_state, const int32_t* slot_idx,
                void* o,
                int32_t T, int32_t N, int32_t max_seqlen_hint,
                int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                int32_t num_slots, float scale,
                void* workspace, size_t workspace_bytes,
                int32_t* dev_status, void* stream);

/*
 * gdn_prefill routes by shape: a batch whose longest sequence has at most
 * GDN_RECURRENT_MAX_SEQLEN tokens (by max_seqlen_hint if given, else by the
 * bound T) goes to the token-by-token kernel; anything longer to one of the
 * chunked variants (gdn_prefill_fused for a few long sequence-heads,
 * gdn_prefill_overlap when max_seqlen_hint tells of chains of at least 40
 * chunks and the sequence-heads number between a third and half of the SMs,
 * gdn_prefill_stream for everything else).  Each route can also be called
 * directly; arguments are gdn_prefill's.  gdn_prefill_chunked is the three
 * launches under their older name: it runs gdn_prefill_stream.
 * gdn_prefill_route answers which one gdn_prefill would take (host-only
 * arithmetic on the shapes; sm_count and cooperative_launch describe the
 * device, gdn_prefill itself queries them): one of GDN_ROUTE_* (never
 * GDN_ROUTE_CHUNKED any more), or GDN_ROUTE_NONE for an empty batch.
 */
#define GDN_RECURRENT_MAX_SEQLEN 16
#define GDN_ROUTE_NONE      0
#define GDN_ROUTE_RECURRENT 1
#define GDN_ROUTE_CHUNKED   2
#define GDN_ROUTE_FUSED     3
#define GDN_ROUTE_STREAM    4
#define GDN_ROUTE_OVERLAP   5
int gdn_prefill_route(int32_t T, int32_t N, int32_t max_seqlen_hint, int32_t Hv,
                      int32_t sm_count, int32_t cooperative_launch);
int gdn_prefill_chunked(const void* q, const void* k, const void* v,
                        const float* g, const float* beta, const int32_t* cu_seqlens,
                        const float* init_state, float* final_state, const int32_t* slot_idx,
                        void* o,
                        int32_t T, int32_t N, int32_t max_seqlen_hint,
                        int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                        int32_t num_slots, float scale,
                        void* workspace, size_t workspace_bytes,
                        int32_t* dev_status, void* stream);

/*
 * gdn_prefill_fused - the chunked algorithm in one cooperative launch (plus a
 * small table-building launch): some of the SMs walk the sequences' chunks
 * in order while the others produce the per-chunk quantities just ahead of
 * them.  Arguments, workspace and results are gdn_prefill_chunked's.
 */
int gdn_prefill_fused(const void* q, const void* k, const void* v,
                      const float* g, const float* beta, const int32_t* cu_seqlens,
                      const float* init_state, float* final_state, const int32_t* slot_idx,
                      void* o,
                      int32_t T, int32_t N, int32_t max_seqlen_hint,
                      int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                      int32_t num_slots, float scale,
                      void* workspace, size_t workspace_bytes,
                      int32_t* dev_status, void* stream);

/*
 * gdn_prefill_stream - the chunked algorithm in three launches whose state
 * pass is a persistent kernel: one CTA per SM walks a list of (sequence,
 * v-head) units and streams their chunks without draining its pipeline
 * between units.  Arguments, workspace and results are gdn_prefill_chunked's.
 */
int gdn_prefill_stream(const void* q, const void* k, const void* v,
                       const float* g, const float* beta, const int32_t* cu_seqlens,
                       const float* init_state, float* final_state, const int32_t* slot_idx,
                       void* o,
                       int32_t T, int32_t N, int32_t max_seqlen_hint,
                       int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                       int32_t num_slots, float scale,
                       void* workspace, size_t workspace_bytes,
                       int32_t* dev_status, void* stream);

/*
 * gdn_prefill_overlap - the chunked algorithm (same subsection of the paper as
 * gdn_prefill: the prefill regime of the gated delta rule) with the
 * intra-chunk work cut in two around the
 * persistent state pass: the records the chains need first are produced
 * before the state pass starts, the others beside it, on the SMs that hold no
 * live chain, each published through a flag the state pass waits for (bounded
 * wait).  For batches of few (sequence,
 * v-head) units of unequal length.  Arguments, workspace and results are
 * gdn_prefill_chunked's, plus
 *   split_permille  share of the (chunk, v-head) items, in the order the
 *                   chains consume them, produced before the state pass
 *                   starts: 0..1000, or negative = chosen on the device from
 *                   the sequence lengths.  With more units than the GPU has
 *                   SMs to spare everything is produced first (1000).
 *                   -2 = as negative, but the producers of the second part
 *                   are launched as an ordinary successor of the state pass
 *                   (serialised on purpose: the recovery path, for tests).
 * Five launches on `stream`; the call is complete when the last one is.  The
 * state pass waits for records of the launch behind it, so the two should run
 * at the same time, which programmatic dependent launch makes the device do
 * but which CUDA does not promise (and a tool that replays kernels one at a
 * time prevents).  If it does not happen the waits for records run out after
 * a few milliseconds, the state pass marks the (sequence, v-head) units it
 * has finished and the last launch runs the others once the records exist:
 * the results are the same, only time is lost (so profile gdn_prefill_stream
 * instead under such a tool).  With CUDA_LAUNCH_BLOCKING set everything is
 * produced first.
 */
int gdn_prefill_overlap(const void* q, const void* k, const void* v,
                        const float* g, const float* beta, const int32_t* cu_seqlens,
                        const float* init_state, float* final_state, const int32_t* slot_idx,
                        void* o,
                        int32_t T, int32_t N, int32_t max_seqlen_hint,
                        int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                        int32_t num_slots, float scale,
                        void* workspace, size_t workspace_bytes,
                        int32_t* dev_status, void* stream, int32_t split_permille);

/*
 * gdn_prefill_recurrent - the same operator and arguments as gdn_prefill,
 * evaluated token by token on the CUDA cores (no chunking, no workspace).  The
 * rows of a state tile evolve independently under the gated delta rule, so the
 * dv rows are spread over warps.  It is the route for very short batches and
 * an independent GPU cross-check of the chunked path.
 */
int gdn_prefill_recurrent(const void* q, const void* k, const void* v,
                          const float* g, const float* beta, const int32_t* cu_seqlens,
                          const float* init_state, float* final_state,
                          const int32_t* slot_idx, void* o,
                          int32_t T, int32_t N, int32_t Hqk, int32_t Hv,
                          int32_t dk, int32_t dv, int32_t num_slots, float scale,
                          int32_t* dev_status, void* stream);

/*
 * gdn_prefill_static - gdn_prefill for callers that cannot allocate device
 * memory.  (No counterpart in the paper: this is a deployment convenience of
 * this library.)  Some callers are not allowed to call cudaMalloc: code running
 * inside another framework's memory plan, a plugin that receives tensors but no
 * allocator, a serving loop whose HBM is already fully assigned.  For them the
 * scratch workspace comes from a fixed array inside the library's own device
 * image, GDN_STATIC_WORKSPACE_BYTES large, which every GPU that loads the
 * library holds until the process exits.
 *
 * Arguments and results are exactly gdn_prefill's, minus workspace and
 * workspace_bytes; inputs and outputs are still the caller's buffers.
 *   - A batch needing more scratch than the array holds
 *     (gdn_prefill_workspace_bytes(...) > GDN_STATIC_WORKSPACE_BYTES) returns
 *     GDN_ERR_LIMIT and nothing is launched.  The scratch is 74 240 bytes per
 *     chunk slot and v-head plus small tables, so with Hv = 32 the array covers
 *     14 chunk slots (floor(T/64) + N <= 14), e.g. 768 tokens in 2 sequences.
 *   - The call itself allocates and frees nothing.  The first call on each
 *     device looks up the array's device address (one cudaGetSymbolAddress, with
 *     that device current) and caches it; make that first call outside of any
 *     stream capture.
 *   - All calls on a device share the one array, and it keeps the previous
 *     call's contents; nothing in it needs to be zero on entry.  Calls that
 *     overlap on the GPU (two streams, two threads) race on it: serialise them.
 */
#define GDN_STATIC_WORKSPACE_BYTES (32u << 20)
size_t gdn_prefill_static_workspace_bytes(void);
int gdn_prefill_static(const void* q, const void* k, const void* v,
                       const float* g, const float* beta, const int32_t* cu_seqlens,
                       const float* init_state, float* final_state, const int32_t* slot_idx,
                       void* o,
                       int32_t T, int32_t N, int32_t max_seqlen_hint,
                       int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                       int32_t num_slots, float scale,
                       int32_t* dev_status, void* stream);

/*
 * Host-buffer variants (same operators; the paper has no counterpart: they are
 * the end-to-end form a caller without device tensors uses).  q, k, v, g, beta,
 * slot_idx / cu_seqlens and o are HOST pointers (pinned memory makes the copies
 * asynchronous); state_pool / init_state / final_state, staging, workspace and
 * dev_status stay DEVICE pointers.  The call enqueues the host->device copies
 * into `staging` (at least gdn_*_host_staging_bytes(...), 256-byte aligned),
 * the kernels, and the device->host copy of o on `stream`, and returns; o is
 * valid once the stream has been synchronised.  Errors as the device variants,
 * GDN_ERR_WORKSPACE also for a staging buffer that is too small.
 */
size_t gdn_decode_host_staging_bytes(int32_t B, int32_t Hqk, int32_t Hv);
int gdn_decode_host(const void* q, const void* k, const void* v,
                    const float* g, const float* beta,
                    float* state_pool, const int32_t* slot_idx, void* o,
                    int32_t B, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                    int32_t num_slots, float scale,
                    void* staging, size_t staging_bytes,
                    int32_t* dev_status, void* stream);
size_t gdn_prefill_host_staging_bytes(int32_t T, int32_t N, int32_t Hqk, int32_t Hv);
int gdn_prefill_host(const void* q, const void* k, const void* v,
                     const float* g, const float* beta, const int32_t* cu_seqlens,
                     const float* init_state, float* final_state, const int32_t* slot_idx,
                     void* o,
                     int32_t T, int32_t N, int32_t max_seqlen_hint,
                     int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                     int32_t num_slots, float scale,
                     void* staging, size_t staging_bytes,
                     void* workspace, size_t workspace_bytes,
                     int32_t* dev_status, void* stream);

/*
 * gdn_host_us_per_decode_call / gdn_host_us_per_prefill_call - measurement aids
 * (no counterpart in the paper, whose remark they serve: small-batch decode is
 * dominated by launch overhead and dispatch).  Each makes one untimed call, then
 * `reps` back-to-back calls of gdn_decode / gdn_prefill with the given arguments
 * on `stream`, and returns the mean HOST time per call in microseconds (argument
 * checks, tensor-map encoding and kernel launches; the stream is synchronised
 * before and after, outside the clock).  A negative return is the GDN_ERR_* code
 * of a rejected call.  The calls really run: the state pool / outputs are
 * updated reps + 1 times.  dev_status is not used.
 */
double gdn_host_us_per_decode_call(const void* q, const void* k, const void* v,
                                   const float* g, const float* beta,
                                   float* state_pool, const int32_t* slot_idx, void* o,
                                   int32_t B, int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv,
                                   int32_t num_slots, float scale, void* stream, int32_t reps);
double gdn_host_us_per_prefill_call(const void* q, const void* k, const void* v,
                                    const float* g, const float* beta, const int32_t* cu_seqlens,
                                    const float* init_state, float* final_state,
                                    const int32_t* slot_idx, void* o,
                                    int32_t T, int32_t N, int32_t max_seqlen_hint,
                                    int32_t Hqk, int32_t Hv, int32_t dk, int32_t dv, int32_t chunk,
                                    int32_t num_slots, float scale,
                                    void* workspace, size_t workspace_bytes,
                                    void* stream, int32_t reps);

/* Human-readable name of a return code (static storage, never NULL). */
const char* gdn_status_string(int code);

/*
 * The CUDA runtime's description of the error behind the calling thread's most
 * recent GDN_ERR_CUDA return ("no error" if there was none).  Static storage.
 */
const char* gdn_last_cuda_error_string(void);

/* Library version, major * 10000 + minor * 100 + patch. */
int gdn_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GDN_B200_H_ */
