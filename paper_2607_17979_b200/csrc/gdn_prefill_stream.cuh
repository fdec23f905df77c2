// Inter-chunk state pass as a PERSISTENT role: a CTA of 512 threads walks a fixed list of
// (sequence, v-head) units and streams their chunk records through one two-stage pipeline that
// does not drain between units.  Two kernels run it: the persistent state pass after the
// intra-chunk kernel (one CTA per SM), and the state CTAs of the fused cooperative launch, whose
// records are produced by other CTAs while the pass runs.
//
// The one-CTA-per-unit state kernel pays, for every unit, a launch slot, barrier and TMEM set-up,
// the first record's memory latency and the tail of its last chunk; with thousands of short
// units (many short sequences) that overhead is longer than the chunk steps themselves.  Here
//   * warp 13 (loader) copies records and K tiles in unit order, running up to two chunks ahead
//     of the consumers and straight across unit boundaries (in the fused launch it first waits
//     for each record's flag);
//   * warp 12 (issuer) issues every tcgen05.mma;
//   * warps 0-7 (chain) carry the dependent chain  U = U~ - S W^T  ->  D4 = (U decayed)^T K  ->
//     S = e^{b_C} S + D4  and nothing else; U~ is already in the accumulator of S W^T when the
//     product runs (negated B operand), so the chain warps read U itself;
//   * warps 8-11 (output) put U~ of the next chunk into that accumulator and turn
//     Y = S Qg^T + U P^T into o rows one chunk behind.  Whatever these warps issue comes out of
//     the chain warps' issue slots, so the rows are made with few instructions (fragment loads,
//     paired conversions, transposing matrix stores).
// The CTA is compiled for 512 threads (128 registers); the chain warps take 144 registers each
// from what the other groups hand back (setmaxnreg).
// The roles never meet at a CTA barrier inside the loop: each derives the same unit list
// (unit = cta + i * n_ctas over the rank-sorted units, longest sequences first) and the same
// running chunk count, from which every mbarrier parity follows.  Every barrier phase is consumed
// by its waiters before the next one can complete (a parity wait cannot tell a barrier that is two
// phases ahead), which is why the state hand-over after a unit's last chunk is omitted rather than
// left unconsumed.
//
// The fp32 master state lives in the chain threads' registers (64 per thread; TMEM lane = state
// row, two column halves), as in the one-CTA-per-unit state kernel.
#pragma once
#include "gdn_prefill_device.cuh"

namespace gdn {

constexpr int kSEpiWarps = 8;                 // warps 0-7: the dependent chain
constexpr int kSEpiThreads = kSEpiWarps * 32;
constexpr int kSOutWarp0 = 8;                 // warps 8-11: output rows (one per TMEM lane quadrant)
constexpr int kSOutThreads = 128;
constexpr int kSIssueWarp = 12;               // warp 12: tcgen05.mma issue
constexpr int kSLoadWarp = 13;                // warp 13: record and K-tile copies (14, 15 spare)
constexpr int kStreamThreads = 512;
constexpr uint32_t kStreamSmem = 2 * kStageBytes + 16384 + 1024;


// What every role needs to know about one unit; derived identically by each of them.
struct UnitInfo {
    int n, hv, hqk, c_first, nc, seq_t0, seq_len, slot;
    bool skip;          // invalid sequence, padding / out-of-range slot, or no chunks
    bool bad_seq, bad_slot;
    bool done;          // finished by an earlier launch (the two-part route's last launch only)
};

__device__ __forceinline__ UnitInfo unit_info(const PrefillParams& p, const uint8_t* ws,
                                              const WorkspaceLayout& lay, int unit,
                                              const int32_t* done = nullptr) {   // units to leave out
    const int32_t* seq_first = reinterpret_cast<const int32_t*>(ws + lay.seq_first);
    const int32_t* seq_bad = reinterpret_cast<const int32_t*>(ws + lay.seq_bad);
    const int32_t* seq_by_rank = reinterpret_cast<const int32_t*>(ws + lay.seq_by_rank);
    UnitInfo u;
    const int rank = unit / p.Hv;
    u.hv = unit - rank * p.Hv;
    u.n = seq_by_rank[rank];
    u.hqk = u.hv / (p.Hv / p.Hqk);
    u.c_first = seq_first[u.n];
    u.nc = seq_first[u.n + 1] - u.c_first;
    u.seq_t0 = p.cu_seqlens[u.n];
    u.seq_len = p.cu_seqlens[u.n + 1] - u.seq_t0;
    u.slot = p.slot_idx ? p.slot_idx[u.n] : u.n;
    u.bad_seq = seq_bad[u.n] != 0;
    u.bad_slot = u.slot < 0 || u.slot >= p.num_slots;
    u.skip = u.bad_seq || u.bad_slot || u.nc == 0;
    u.done = done != nullptr && done[unit] != 0;
    return u;
}

constexpr uint32_t kSpinFlagLimit = 1u << 22;
// a few milliseconds: far longer than the producers ever lag when they do run beside the state
// pass, far shorter than the other roles' mbarrier waits (which would report an error)
constexpr uint32_t kSpinFlagLimitSoft = 1u << 13;

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() {
    asm volatile("fence.proxy.async;" ::: "memory");
}

// The state pass of one CTA of 512 threads over the units cta, cta + n_ctas, ... of the rank-sorted
// list.  kGated = 0: every record exists (the intra-chunk kernel ran before).  kGated = 1:
// records are being produced by other CTAs of the same cooperative launch and the loading warp
// waits for each record's flag first.  kGated = 2: the records of the first hdr[kHdrSplit] items of
// the processing order exist, the others are being produced by a concurrent kernel and are waited
// for; a wait that runs out ends the CTA's work without an error (the units it has finished are
// marked in the done table, the others are left to a later launch).  kGated = 3: that later launch:
// every record exists, the units marked done are left out.  `tmem` = 512 allocated columns; ends
// with a CTA barrier.
template <int kGated>
__device__ __forceinline__ void state_stream_role(const TensorMaps& maps, const PrefillParams& p,
                                                  uint8_t* ws, const WorkspaceLayout& lay,
                                                  uint8_t* smem, const uint32_t tmem, const int cta,
                                                  const int n_ctas) {
    __shared__ uint64_t bar_full[2], bar_free_a[2], bar_free_b[2], bar_free_c[2], bar_y[2],
        bar_d1, bar_d4, bar_s, bar_u;
    __shared__ int abort_flag;
    __shared__ uint32_t armed_chunks;     // chunks of the CTA's stream whose copies the loader has started
    // kGated == 2 waits for records of a launch that may not be running beside this one: there no
    // wait that runs out is an error, whichever role it happens in (the loader's own wait for a
    // flag is the shortest, but the limits are counted in polls, not in time): the units this CTA
    // has not finished are left to the last launch, which reports real failures.
    constexpr int kWaitReason = kGated == 2 ? 2 : 1;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int half = (warp >> 2) & 1;                 // which half of the columns this thread owns
    const int dv = (warp & 3) * 32 + lane;            // TMEM lane = state row
    const uint32_t lane_base = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int total_units = p.N * p.Hv;
    int32_t* done_w = reinterpret_cast<int32_t*>(ws + lay.done);      // written by kGated == 2
    const int32_t* done_tab = kGated == 3 ? done_w : nullptr;         // read by kGated == 3
    (void)done_w;

    if (tid == 0) {
        mbar_init(&bar_full[0], 1);
        mbar_init(&bar_full[1], 1);
        // A stage is released in three parts as its readers finish with them, so that the next
        // record's copies start up to half a chunk step earlier (one chunk step of look-ahead is
        // shorter than a cold 74 KB copy): W and Qg once S W^T and S Qg^T have retired, U~ and the
        // decay vector once every chain warp has read them, P and the K tile once U P^T and the
        // state product have retired.
        for (int st = 0; st < 2; ++st) {
            mbar_init(&bar_free_a[st], 1);
            mbar_init(&bar_free_b[st], kSEpiWarps);
            mbar_init(&bar_free_c[st], 1);
        }
        mbar_init(&bar_d1, 1);
        mbar_init(&bar_d4, 1);
        mbar_init(&bar_y[0], 1);      // one per Y tile: with a single barrier the output warps could
        mbar_init(&bar_y[1], 1);      // find it two phases ahead, which a parity wait cannot tell
        // bar_s: everything the chunk's first product needs is in TMEM: the bf16 state (one arrival
        // per chain warp) and U~ in the accumulator (one per output warp).  The output warps copy
        // U~ only after they have seen the record land and have read the Y tile of two chunks
        // ago, so this one wait also tells the issuing warp that the record is in shared memory
        // and that the Y tile may be overwritten.
        mbar_init(&bar_s, kSEpiWarps + kSOutThreads / 32);
        mbar_init(&bar_u, kSEpiWarps);
        abort_flag = 0;
        armed_chunks = 0;
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    volatile int* abortp = &abort_flag;
    if constexpr (kGated == 0) pdl_wait();     // tables and records are the previous kernels'

    // gc = chunks of earlier units of this CTA; chunk j of the current unit is chunk g = gc + j of
    // the CTA's stream: stage g & 1, phase g >> 1 of bar_full / bar_free_* of that stage, phase g of
    // bar_d1 / bar_d4 / bar_y / bar_u and of bar_s (one state hand-over per chunk: the initial one
    // and one after every chunk but the unit's last).
    uint32_t gc = 0;

    // Register budget: setmaxnreg waits, unbounded, until the registers it asks for have been given
    // back by other warps of the same CTA, so keep room to spare and use multiples of 16.  The CTA
    // starts with 512 x 128; the issuing group gives back 128 x 64, the output warps 128 x 16, the
    // chain warps take 256 x 16.
    if (warp >= kSIssueWarp) {
    reg_dealloc<64>();
    if (warp == kSLoadWarp) {
        // ===================== loader: records and K tiles, in stream order
        if (lane == 0) {
            const size_t rec_stride = static_cast<size_t>(p.Hv) * kRecBytes;
            const uint32_t* flags = reinterpret_cast<const uint32_t*>(ws + lay.flags);
            (void)flags;
            bool live = true;
            // kGated == 2: chunk j of the sequence of rank r is item (pos[j] + r) * Hv + hv of
            // the processing order; items from `cut` on are waited for
            const int32_t* pos = reinterpret_cast<const int32_t*>(ws + lay.pos);
            const int32_t cut = kGated == 2 ? reinterpret_cast<const int32_t*>(ws)[kHdrSplit] : 0;
            (void)pos;
            (void)cut;
            // the next unit's table entries are fetched while the current unit is processed
            UnitInfo nxt = unit_info(p, ws, lay, min(cta, total_units - 1), done_tab);
            for (int unit = cta; unit < total_units && live; unit += n_ctas) {
                const UnitInfo u = nxt;
                nxt = unit_info(p, ws, lay, min(unit + n_ctas, total_units - 1), done_tab);
                if (u.skip || u.done) continue;
                const uint8_t* records =
                    ws + lay.records + (static_cast<size_t>(u.c_first) * p.Hv + u.hv) * kRecBytes;
                const int32_t rank = unit / p.Hv;
                int32_t pos_j = kGated == 2 ? pos[0] : 0;       // fetched one chunk ahead
                for (int j = 0; j < u.nc; ++j) {
                    const uint32_t g = gc + j;
                    const int st = g & 1;
                    // the stage held chunk g - 2; each part is refilled as soon as it is free
                    const uint32_t par_free = ((g - 2) >> 1) & 1u;
                    uint8_t* base = smem + st * kStageBytes;
                    const uint8_t* rec = records + j * rec_stride;
                    bool gated = kGated == 1;
                    if constexpr (kGated == 2) {
                        gated = (pos_j + rank) * p.Hv + u.hv >= cut;
                        pos_j = pos[j + 1];                     // pos has an entry past the longest chain
                    }
                    if (gated) {
                        // the record must have been published by its producer CTA
                        const uint32_t* f = flags + (static_cast<size_t>(u.c_first + j) * p.Hv + u.hv);
                        uint32_t v = 0;
                        // kGated == 2: a wait that runs out is no error (the producers' launch may
                        // not be running beside this one): give up soon, well before any of the
                        // other roles' waits, and leave the unit to the last launch
                        const uint32_t limit = kGated == 2 ? kSpinFlagLimitSoft : kSpinFlagLimit;
                        for (uint32_t i = 0; i < limit; ++i) {
                            v = ld_acquire_u32(f);
                            if (v != 0 || *abortp) break;
                            __nanosleep(64);
                        }
                        if (v != 1) {
                            if (*abortp == 0) *abortp = (kGated == 2 && v == 0) ? 2 : 1;
                            live = false;
                            break;
                        }
                        // No proxy fence here: the producer put one between its generic stores and
                        // the flag's release, which is on the path from those stores to the copies
                        // below; one here would also wait for this thread's copies in flight (3 %
                        // of a long sequence's run time).
                    }
                    if (g >= 2 && !wait_or_abort(&bar_free_a[st], par_free, abortp, kWaitReason)) { live = false; break; }
                    armed_chunks = g + 1;
                    mbar_expect_tx(&bar_full[st], kRecBytes + 16384);
                    bulk_load(base + kS_Rec + kRecW, rec + kRecW, kRecP - kRecW, &bar_full[st]);
                    if (g >= 2 && !wait_or_abort(&bar_free_b[st], par_free, abortp, kWaitReason)) { live = false; break; }
                    bulk_load(base + kS_Rec + kRecU, rec + kRecU, kRecBytes - kRecU, &bar_full[st]);
                    if (g >= 2 && !wait_or_abort(&bar_free_c[st], par_free, abortp, kWaitReason)) { live = false; break; }
                    bulk_load(base + kS_Rec + kRecP, rec + kRecP, kRecU - kRecP, &bar_full[st]);
                    tma_load_2d(base + kS_K, &maps.k, u.hqk * kD, u.seq_t0 + j * kChunk, &bar_full[st]);
                    tma_load_2d(base + kS_K + 8192, &maps.k, u.hqk * kD + 64, u.seq_t0 + j * kChunk,
                                &bar_full[st]);
                }
                gc += u.nc;
            }
        }
        __syncwarp();
    } else if (warp == kSIssueWarp) {
        // ===================== issuer: tensor-core instructions
        {   // the whole warp runs this warp-uniform code; one elected lane executes each tcgen05 instruction
            const uint32_t id64 = make_idesc_bf16(128, 64, false, false);
            const uint32_t id128mn = make_idesc_bf16(128, 128, false, true);
            const uint32_t id64mn = make_idesc_bf16(128, 64, false, true) | kIdescNegateB;
            const uint32_t sRec0 = smem_u32(smem + kS_Rec), sRec1 = sRec0 + kStageBytes;
            const uint64_t dW0 = make_sdesc_sw128(sRec0 + kRecW, 8192, 1024);
            const uint64_t dQ0 = make_sdesc_sw128(sRec0 + kRecQg, 16, 1024);
            const uint64_t dP0 = make_sdesc_sw128(sRec0 + kRecP, 16, 1024);
            const uint64_t dK0 = make_sdesc_sw128(sRec0 + kS_K, 8192, 1024);
            const uint64_t dW1 = make_sdesc_sw128(sRec1 + kRecW, 8192, 1024);
            const uint64_t dQ1 = make_sdesc_sw128(sRec1 + kRecQg, 16, 1024);
            const uint64_t dP1 = make_sdesc_sw128(sRec1 + kRecP, 16, 1024);
            const uint64_t dK1 = make_sdesc_sw128(sRec1 + kS_K, 8192, 1024);
            const uint32_t tS = tmem + kT_S, tD1 = tmem + kT_D1, tD4 = tmem + kT_D4;
            bool live = true;
            // the next unit's table entries are fetched while the current unit is processed
            UnitInfo nxt = unit_info(p, ws, lay, min(cta, total_units - 1), done_tab);
            for (int unit = cta; unit < total_units && live; unit += n_ctas) {
                const UnitInfo u = nxt;
                nxt = unit_info(p, ws, lay, min(unit + n_ctas, total_units - 1), done_tab);
                if (u.skip || u.done) continue;
                for (int j = 0; j < u.nc; ++j) {
                    const uint32_t g = gc + j;
                    const int st = g & 1;
                    const uint64_t w = st ? dW1 : dW0, qg = st ? dQ1 : dQ0, pp = st ? dP1 : dP0,
                                   kk = st ? dK1 : dK0;
                    const uint32_t tY = tmem + kT_Y + st * 64;
                    if (!wait_or_abort(&bar_s, g & 1u, abortp, kWaitReason)) {      // record landed, bf16 S and U~ in TMEM
                        live = false;
                        break;
                    }
                    tc_fence_after_sync();
                    // U = U~ - S W^T  (on the chain): the accumulator holds U~, the B operand is negated;
                    // W is MN-major: k-step ks reads 16 dk rows = 2048 bytes
                    if (elect_one()) mma_ts_c<true>(tD1, tS, w, id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 8, sdesc_advance(w, 2048), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 16, sdesc_advance(w, 4096), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 24, sdesc_advance(w, 6144), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 32, sdesc_advance(w, 8192), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 40, sdesc_advance(w, 10240), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 48, sdesc_advance(w, 12288), id64mn);
                    if (elect_one()) mma_ts_c<true>(tD1, tS + 56, sdesc_advance(w, 14336), id64mn);
                    if (elect_one()) mma_commit(&bar_d1);
                    // Y = S Qg^T  (off the chain) overwrites the tile the output warps read two chunks ago
                    if (elect_one()) mma_ts_c<false>(tY, tS, qg, id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 8, sdesc_advance(qg, 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 16, sdesc_advance(qg, 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 24, sdesc_advance(qg, 96), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 32, sdesc_advance(qg, 8192), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 40, sdesc_advance(qg, 8192 + 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 48, sdesc_advance(qg, 8192 + 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tS + 56, sdesc_advance(qg, 8192 + 96), id64);
                    if (elect_one()) mma_commit(&bar_free_a[st]);                          // W and Qg have been read
                    if (!wait_or_abort(&bar_u, g & 1u, abortp, kWaitReason)) {         // U operands in TMEM
                        live = false;
                        break;
                    }
                    tc_fence_after_sync();
                    // D4 = (U decayed, hi + lo) K   (K tile MN-major: 16 tokens = 2048 bytes)
                    if (elect_one()) mma_ts_c<false>(tD4, tmem + kT_Us, kk, id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 8, sdesc_advance(kk, 2048), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 16, sdesc_advance(kk, 4096), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_Us + 24, sdesc_advance(kk, 6144), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo, kk, id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 8, sdesc_advance(kk, 2048), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 16, sdesc_advance(kk, 4096), id128mn);
                    if (elect_one()) mma_ts_c<true>(tD4, tmem + kT_UsLo + 24, sdesc_advance(kk, 6144), id128mn);
                    if (elect_one()) mma_commit(&bar_d4);
                    // Y += U P^T
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U, pp, id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 8, sdesc_advance(pp, 32), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 16, sdesc_advance(pp, 64), id64);
                    if (elect_one()) mma_ts_c<true>(tY, tmem + kT_U + 24, sdesc_advance(pp, 96), id64);
                    if (elect_one()) mma_commit(&bar_y[st]);
                    if (elect_one()) mma_commit(&bar_free_c[st]);                          // P and the K tile have been read
                }
                gc += u.nc;
            }
        }
        __syncwarp();
    }
    } else if (warp < kSEpiWarps) {
        reg_alloc<144>();
        // ===================== chain warps: U and the state refresh (the dependent chain)
        auto hand_over = [&](uint64_t* bar) {     // after tcgen05.st: publish to the issuing lane
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar);
        };
        float S[64];      // the thread's 64 state columns [64*half, 64*half+64) of row dv, fp32 master
        auto store_state_bf16 = [&]() {           // S (fp32 regs) -> bf16 A operand in TMEM
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) pk[j] = pack_bf16(S[c0 + 2 * j], S[c0 + 2 * j + 1]);
                tmem_st16(tmem + kT_S + lane_base + half * 32 + (c0 >> 1), pk);
            }
        };
        bool ok = true;
        auto await = [&](uint64_t* bar, uint32_t parity) {   // bounded wait + tcgen05 fence
            if (ok && !warp_wait_or_abort(bar, parity, abortp, kWaitReason)) ok = false;
            tc_fence_after_sync();
        };
        // Every warp runs every group barrier and hand-over below, also after a wait has failed
        // (ok == false: later waits and all work are skipped), so that no warp is ever left alone
        // at a barrier.
        UnitInfo nxt = unit_info(p, ws, lay, min(cta, total_units - 1), done_tab);
        for (int unit = cta; unit < total_units; unit += n_ctas) {
            const UnitInfo u = nxt;
            nxt = unit_info(p, ws, lay, min(unit + n_ctas, total_units - 1), done_tab);
            const size_t tile_off = (static_cast<size_t>(u.bad_slot ? 0 : u.slot) * p.Hv + u.hv) * (kD * kD) +
                                    static_cast<size_t>(dv) * kD + half * 64;
            if (u.done) continue;
            if (u.skip) {
                if constexpr (kGated == 2) {
                    if (tid == 0) done_w[unit] = 1;
                }
                if (u.bad_seq) continue;
                if (u.bad_slot) {          // padding / out-of-range slot: zero rows, no state
                    if (u.slot >= p.num_slots && tid == 0) report(p.dev_status, kDevBadSlot);
                    const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
                    for (int idx = tid; idx < u.seq_len * 16; idx += kSEpiThreads)
                        *reinterpret_cast<uint4*>(p.o + (static_cast<size_t>(u.seq_t0 + (idx >> 4)) * p.Hv + u.hv) * kD +
                                                  (idx & 15) * 8) = zero;
                } else {                   // empty sequence: the state passes through untouched
#pragma unroll 4
                    for (int j = 0; j < 64; j += 4) {
                        const float4 x = p.init_state
                                             ? *reinterpret_cast<const float4*>(p.init_state + tile_off + j)
                                             : make_float4(0.f, 0.f, 0.f, 0.f);
                        *reinterpret_cast<float4*>(p.final_state + tile_off + j) = x;
                    }
                }
                continue;
            }
            const int nc = u.nc;
            // the unit's initial state
            if (p.init_state) {
#pragma unroll
                for (int j = 0; j < 64; j += 4) {
                    const float4 x = *reinterpret_cast<const float4*>(p.init_state + tile_off + j);
                    S[j] = x.x; S[j + 1] = x.y; S[j + 2] = x.z; S[j + 3] = x.w;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 64; ++j) S[j] = 0.f;
            }
            if (ok) store_state_bf16();
            hand_over(&bar_s);
            for (int j = 0; j < nc; ++j) {
                const uint32_t g = gc + j;
                const int st = g & 1;
                const uint8_t* base = smem + st * kStageBytes;
                await(&bar_full[st], (g >> 1) & 1u);
                await(&bar_d1, g & 1u);
                if (ok) {   // U^T[dv][c] (the accumulator holds U~ - S W^T) for the thread's 32 tokens [32*half, 32*half+32)
                    const float* sdec = reinterpret_cast<const float*>(base + kS_Rec + kRecDecay);
#pragma unroll
                    for (int c0 = 0; c0 < 32; c0 += 16) {
                        const int cb = half * 32 + c0;
                        uint32_t x[16];
                        tmem_ld16(tmem + kT_D1 + lane_base + cb, x);
                        tmem_wait_ld();
                        uint32_t pu[8], ph[8], pl[8];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const float4 dd = *reinterpret_cast<const float4*>(sdec + cb + 4 * q4);
                            const float u0 = __uint_as_float(x[4 * q4 + 0]);
                            const float u1 = __uint_as_float(x[4 * q4 + 1]);
                            const float u2 = __uint_as_float(x[4 * q4 + 2]);
                            const float u3 = __uint_as_float(x[4 * q4 + 3]);
                            const float s0 = u0 * dd.x, s1 = u1 * dd.y, s2 = u2 * dd.z, s3 = u3 * dd.w;
                            pu[2 * q4] = pack_bf16(u0, u1);
                            pu[2 * q4 + 1] = pack_bf16(u2, u3);
                            ph[2 * q4] = pack_bf16(s0, s1);
                            ph[2 * q4 + 1] = pack_bf16(s2, s3);
                            pl[2 * q4] = pack_bf16(s0 - __uint_as_float(ph[2 * q4] << 16),
                                                   s1 - __uint_as_float(ph[2 * q4] & 0xffff0000u));
                            pl[2 * q4 + 1] = pack_bf16(s2 - __uint_as_float(ph[2 * q4 + 1] << 16),
                                                       s3 - __uint_as_float(ph[2 * q4 + 1] & 0xffff0000u));
                        }
                        tmem_st8(tmem + kT_Us + lane_base + (cb >> 1), ph);
                        tmem_st8(tmem + kT_UsLo + lane_base + (cb >> 1), pl);
                        tmem_st8(tmem + kT_U + lane_base + (cb >> 1), pu);
                    }
                }
                const float gC = reinterpret_cast<const float*>(base + kS_Rec + kRecGammaC)[0];
                hand_over(&bar_u);
                if (lane == 0) mbar_arrive(&bar_free_b[st]);    // this warp has read U~, decay, e^{b_C}
                const bool last = j + 1 == nc;
                await(&bar_d4, g & 1u);
                if (ok) {   // S <- e^{b_C} S + D4 on the thread's 64 dk columns
#pragma unroll
                    for (int c0 = 0; c0 < 64; c0 += 32) {
                        uint32_t xa[16], xb[16];
                        tmem_ld16(tmem + kT_D4 + lane_base + half * 64 + c0, xa);
                        tmem_ld16(tmem + kT_D4 + lane_base + half * 64 + c0 + 16, xb);
                        tmem_wait_ld();
#pragma unroll
                        for (int jj = 0; jj < 16; ++jj) {
                            S[c0 + jj] = fmaf(gC, S[c0 + jj], __uint_as_float(xa[jj]));
                            S[c0 + 16 + jj] = fmaf(gC, S[c0 + 16 + jj], __uint_as_float(xb[jj]));
                        }
                    }
                    if (!last) {
                        store_state_bf16();          // the next chunk's A operand
                    } else {
#pragma unroll
                        for (int j4 = 0; j4 < 64; j4 += 4)
                            *reinterpret_cast<float4*>(p.final_state + tile_off + j4) =
                                make_float4(S[j4], S[j4 + 1], S[j4 + 2], S[j4 + 3]);
                        // (every record of the unit has been loaded by now: no flag wait can
                        // fail after this point, and any other failure is reported as an error)
                        if constexpr (kGated == 2) {
                            if (tid == 0) done_w[unit] = 1;
                        }
                    }
                }
                if (!last) hand_over(&bar_s);
            }
            gc += nc;
        }
    } else {
        reg_dealloc<112>();
        // ===================== output warps: Y = S Qg^T + U P^T (fp32, TMEM) -> o rows.  Warp 8 + q
        // reads TMEM lanes 32 q .. 32 q + 31 (dv indices), scales and rounds, transposes through
        // shared memory, and the four warps write whole rows in 16-byte pieces.
        const int q4 = warp & 3;
        const uint32_t olane = static_cast<uint32_t>(q4 * 32) << 16;
        const int ot = tid - kSOutWarp0 * 32;
        const size_t tok_stride = static_cast<size_t>(p.Hv) * kD;
        __nv_bfloat16* sO = reinterpret_cast<__nv_bfloat16*>(smem + kS_Out);
        auto out_sync = [] { asm volatile("bar.sync 1, %0;" ::"n"(kSOutThreads) : "memory"); };
        bool ok = true;
        // U~ (fp32, 32 KB per chunk) reaches the chain through the accumulator of S W^T: this group
        // copies it from the record into TMEM one chunk ahead, the product then subtracts S W^T
        // from it (negated B operand), and the chain warps read U itself.  (Read by the chain warps
        // from shared memory, the 32 KB took 300 of the 3700 cycles of a chunk step.)
        const int odv = q4 * 32 + lane;
        auto preload = [&](uint32_t gq) {       // chunk gq of the CTA's stream -> accumulator
            const int sq = gq & 1;
            if (ok && !warp_wait_or_abort(&bar_full[sq], (gq >> 1) & 1u, abortp, kWaitReason)) ok = false;
            if (ok) {
                const float4* sU = reinterpret_cast<const float4*>(smem + sq * kStageBytes + kS_Rec + kRecU);
#pragma unroll
                for (int c0 = 0; c0 < 64; c0 += 16) {
                    uint32_t r[16];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const float4 v = sU[((c0 >> 2) + q) * kD + odv];
                        r[4 * q] = __float_as_uint(v.x); r[4 * q + 1] = __float_as_uint(v.y);
                        r[4 * q + 2] = __float_as_uint(v.z); r[4 * q + 3] = __float_as_uint(v.w);
                    }
                    tmem_st16(tmem + kT_D1 + olane + c0, r);
                }
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bar_s);
        };
        bool preloaded = false;     // U~ of the chunk about to be processed is already in place
        UnitInfo nxt = unit_info(p, ws, lay, min(cta, total_units - 1), done_tab);
        for (int unit = cta; unit < total_units; unit += n_ctas) {
            const UnitInfo u = nxt;
            nxt = unit_info(p, ws, lay, min(unit + n_ctas, total_units - 1), done_tab);
            if (u.skip || u.done) continue;
            for (int j = 0; j < u.nc; ++j) {
                const uint32_t g = gc + j;
                const int buf = g & 1;
                // k = 0: this chunk's U~ (first chunk of the stream, or after a skipped unit).
                // k = 1: once the chain warps have read U of this chunk the accumulator is free for
                // the next chunk's U~ (when the next chunk is known without looking past a skipped
                // unit), which is then in place long before the chain warps hand the state over.
                const bool ahead = j + 1 < u.nc || (unit + n_ctas < total_units && !nxt.skip && !nxt.done);
#pragma unroll 1
                for (int k = preloaded ? 1 : 0; k < 2; ++k) {
                    if (k == 1) {
                        if (ok && !warp_wait_or_abort(&bar_u, g & 1u, abortp, kWaitReason)) ok = false;
                        tc_fence_after_sync();
                        if (!ahead) break;
                    }
                    preload(g + k);
                }
                preloaded = ahead;
                // every warp runs both group barriers of every chunk, also after a failed wait
                if (ok && !warp_wait_or_abort(&bar_y[buf], (g >> 1) & 1u, abortp, kWaitReason)) ok = false;
                tc_fence_after_sync();
                // The Y tile (lanes = dv, columns = tokens) is read as accumulator fragments, rounded
                // in pairs and stored transposed, 8 dv of one token per 16 bytes, into a [token][dv]
                // tile of two 128B-swizzled halves of 64 dv: 2 loads, 32 conversions and 8 stores
                // per thread instead of 64 scalar conversions and 64 two-byte stores (what these
                // warps issue comes out of the chain warps' issue slots).
                uint32_t pa[16], pb[16];     // packed pairs: lanes 0-15 / 16-31 of the quadrant
                if (ok) {
                    const uint32_t tY = tmem + kT_Y + buf * 64;
                    uint32_t y[32];
                    tmem_ld_16x256b_x8(tY + olane, y);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        pa[i] = pack_bf16(__uint_as_float(y[2 * i]), __uint_as_float(y[2 * i + 1]));
                    tmem_ld_16x256b_x8(tY + olane + (16u << 16), y);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        pb[i] = pack_bf16(__uint_as_float(y[2 * i]), __uint_as_float(y[2 * i + 1]));
                }
                if (ok) {
                    const int dv0 = q4 * 32 + 8 * (lane >> 3);         // the 8 dv this lane's address covers
                    const uint32_t dst = smem_u32(sO) + (dv0 >> 6) * 8192;
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        stmatrix_x4_trans(dst + sw128_offset(8 * i + (lane & 7), (dv0 & 63) >> 3),
                                          pa[2 * i], pa[2 * i + 1], pb[2 * i], pb[2 * i + 1]);
                }
                out_sync();
                if (ok) {
                    const int len = min(kChunk, u.seq_len - j * kChunk);
                    __nv_bfloat16* og = p.o + (static_cast<size_t>(u.seq_t0 + j * kChunk) * p.Hv + u.hv) * kD;
                    const uint8_t* src = reinterpret_cast<const uint8_t*>(sO) + ((ot & 15) >> 3) * 8192;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int row = it * 8 + (ot >> 4), piece = ot & 15;
                        if (row < len)
                            *reinterpret_cast<uint4*>(og + row * tok_stride + piece * 8) =
                                *reinterpret_cast<const uint4*>(src + sw128_offset(row, piece & 7));
                    }
                }
                out_sync();
            }
            gc += u.nc;
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (abort_flag != 0 && warp == kSIssueWarp && lane == 0) {
        if (abort_flag == 1) report(p.dev_status, kDevTimeout);     // 2: a record not produced yet, no error
        // let copies already in flight land before the CTA's shared memory goes away: the last two
        // chunks the loader started, each on its stage's barrier at that chunk's own parity
        const uint32_t armed = *reinterpret_cast<volatile uint32_t*>(&armed_chunks);
        for (uint32_t back = 1; back <= 2 && back <= armed; ++back) {
            const uint32_t gq = armed - back;
            mbar_wait(&bar_full[gq & 1], (gq >> 1) & 1u, 1u << 12);
        }
    }
}

}  // namespace gdn
