// Gated delta rule (Gated DeltaNet) reference oracle: plain, slow, fp64, CPU only.
//
// THIS IS TEST INFRASTRUCTURE. Only the tests, the smoke check and the
// benchmark's CPU-baseline leg may call it. It shares no code with the CUDA
// library and the CUDA library never calls it.
//
// What it computes (paper, appendix "Operator Background and Mathematical
// Definitions", subsection "Gated Delta Net", the gated delta rule):
//
//     S_t = S_{t-1} ( alpha_t ( I - beta_t k_t k_t^T ) ) + beta_t v_t k_t^T
//     o_t = scale * S_t q_t                   (the paper's o_t has scale = 1)
//
// with S in R^{dv x dk}, alpha_t = exp(g_t) (the paper's natural-log gate),
// one independent recurrence per (sequence, v-head).  The token loop below
// takes the steps in exactly that order, one token at a time:
//
//   (1) decay:        S <- alpha_t * S
//   (2) read-out:     u <- S k_t                      (dv-vector)
//   (3) delta write:  S <- S + beta_t (v_t - u) k_t^T
//   (4) output:       o_t <- scale * S q_t            (uses the UPDATED state)
//
// (1)-(3) is the bracketed product multiplied out:
//   alpha S (I - beta k k^T) + beta v k^T = alpha S + beta (v - alpha S k) k^T.
//
// Conventions the paper leaves open and this library fixes:
//   * q,k heads map to v heads by  hqk = hv / (Hv / Hqk)   (grouped heads).
//   * a state tile is stored row-major [dv][dk] (dk contiguous).
//   * bf16 inputs arrive as raw 16-bit patterns and are widened exactly.
//   * slot index < 0 marks a padding entry: its outputs are zero and no state
//     is touched; an index >= num_slots is reported and skipped the same way.
//
// Threads only split the independent (sequence, v-head) units; there is no
// blocking, fusion or re-association of the arithmetic.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <thread>
#include <vector>
#include <atomic>
#include <algorithm>

namespace {

inline double bf16_to_double(uint16_t bits) {
    uint32_t w = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &w, sizeof(f));
    return static_cast<double>(f);
}

// One token of the recurrence for one (sequence, v-head) unit.
// S: [dv][dk] fp64, updated in place.  o: [dv] fp64.
void gated_delta_step(double* S, const uint16_t* q, const uint16_t* k, const uint16_t* v,
                      float g, float beta_f, double scale, int dk, int dv,
                      double* o, double* kd, double* qd) {
    const double alpha = std::exp(static_cast<double>(g));
    const double beta = static_cast<double>(beta_f);
    for (int c = 0; c < dk; ++c) {
        kd[c] = bf16_to_double(k[c]);
        qd[c] = bf16_to_double(q[c]);
    }
    for (int j = 0; j < dv; ++j) {
        double* row = S + static_cast<size_t>(j) * dk;
        // (1) decay
        for (int c = 0; c < dk; ++c) row[c] *= alpha;
        // (2) read-out of the value currently stored under key k_t
        double u = 0.0;
        for (int c = 0; c < dk; ++c) u += row[c] * kd[c];
        // (3) delta write
        const double w = beta * (bf16_to_double(v[j]) - u);
        for (int c = 0; c < dk; ++c) row[c] += w * kd[c];
        // (4) output from the updated state
        double acc = 0.0;
        for (int c = 0; c < dk; ++c) acc += row[c] * qd[c];
        o[j] = scale * acc;
    }
}

template <class F>
void parallel_units(int64_t n_units, int n_threads, F&& body) {
    int hw = static_cast<int>(std::thread::hardware_concurrency());
    if (hw <= 0) hw = 1;
    int nt = n_threads > 0 ? n_threads : hw;
    nt = static_cast<int>(std::min<int64_t>(nt, std::max<int64_t>(n_units, 1)));
    if (nt <= 1) {
        for (int64_t u = 0; u < n_units; ++u) body(u);
        return;
    }
    std::atomic<int64_t> next{0};
    std::vector<std::thread> pool;
    pool.reserve(nt);
    for (int t = 0; t < nt; ++t) {
        pool.emplace_back([&]() {
            for (;;) {
                int64_t u = next.fetch_add(1);
                if (u >= n_units) break;
                body(u);
            }
        });
    }
    for (auto& th : pool) th.join();
}

}  // namespace

extern "C" {

// Number of worker threads a call with n_threads <= 0 would use at most.
int gdn_oracle_default_threads(void) {
    int hw = static_cast<int>(std::thread::hardware_concurrency());
    return hw > 0 ? hw : 1;
}

// Decode: one token per sequence, state pool updated in place.
//   q,k   bf16 bits [B][Hqk][dk]      v bf16 bits [B][Hv][dv]
//   g,beta fp32 [B][Hv]               pool fp64 [num_slots][Hv][dv][dk] (in/out)
//   slot_idx int32 [B] or NULL (identity)        o fp64 [B][Hv][dv]
// Returns the number of (entry, v-head) units skipped because their slot was
// out of range (>= num_slots); negative slots are padding and are not counted.  -1 = bad
// arguments.
int gdn_oracle_decode(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                      const float* g, const float* beta, double* pool,
                      const int32_t* slot_idx, double* o,
                      int B, int Hqk, int Hv, int dk, int dv, int num_slots,
                      double scale, int n_threads) {
    if (B < 0 || Hqk <= 0 || Hv <= 0 || dk <= 0 || dv <= 0 || Hv % Hqk != 0) return -1;
    const int G = Hv / Hqk;
    std::atomic<int> bad{0};
    parallel_units(static_cast<int64_t>(B) * Hv, n_threads, [&](int64_t unit) {
        const int i = static_cast<int>(unit / Hv);
        const int hv = static_cast<int>(unit % Hv);
        const int hqk = hv / G;
        double* o_row = o + (static_cast<size_t>(i) * Hv + hv) * dv;
        const int slot = slot_idx ? slot_idx[i] : i;
        if (slot < 0 || slot >= num_slots) {
            if (slot >= num_slots) bad.fetch_add(1);
            for (int j = 0; j < dv; ++j) o_row[j] = 0.0;
            return;
        }
        std::vector<double> kd(dk), qd(dk);
        double* S = pool + (static_cast<size_t>(slot) * Hv + hv) * dv * dk;
        gated_delta_step(S,
                         q + (static_cast<size_t>(i) * Hqk + hqk) * dk,
                         k + (static_cast<size_t>(i) * Hqk + hqk) * dk,
                         v + (static_cast<size_t>(i) * Hv + hv) * dv,
                         g[static_cast<size_t>(i) * Hv + hv],
                         beta[static_cast<size_t>(i) * Hv + hv],
                         scale, dk, dv, o_row, kd.data(), qd.data());
    });
    return bad.load();
}

// Prefill: packed variable-length sequences, token by token.
//   q,k bf16 bits [T][Hqk][dk]   v bf16 bits [T][Hv][dv]   g,beta fp32 [T][Hv]
//   cu_seqlens int32 [N+1] (cu[0]=0, non-decreasing, cu[N]=T)
//   init_state fp64 [num_slots][Hv][dv][dk] or NULL (= zero state)
//   final_state fp64 [num_slots][Hv][dv][dk] (may be the same array as init)
//   slot_idx int32 [N] or NULL (identity); negative = padding sequence
//   o fp64 [T][Hv][dv]
// Returns count of (sequence, v-head) units skipped for an out-of-range slot, -1 bad args,
// -2 inconsistent cu_seqlens.
int gdn_oracle_prefill(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                       const float* g, const float* beta, const int32_t* cu_seqlens,
                       const double* init_state, double* final_state,
                       const int32_t* slot_idx, double* o,
                       int T, int N, int Hqk, int Hv, int dk, int dv, int num_slots,
                       double scale, int n_threads) {
    if (T < 0 || N < 0 || Hqk <= 0 || Hv <= 0 || dk <= 0 || dv <= 0 || Hv % Hqk != 0) return -1;
    if (N > 0) {
        if (cu_seqlens[0] != 0 || cu_seqlens[N] != T) return -2;
        for (int n = 0; n < N; ++n)
            if (cu_seqlens[n + 1] < cu_seqlens[n]) return -2;
    }
    const int G = Hv / Hqk;
    const size_t tile = static_cast<size_t>(dv) * dk;
    std::atomic<int> bad{0};
    parallel_units(static_cast<int64_t>(N) * Hv, n_threads, [&](int64_t unit) {
        const int n = static_cast<int>(unit / Hv);
        const int hv = static_cast<int>(unit % Hv);
        const int hqk = hv / G;
        const int t0 = cu_seqlens[n], t1 = cu_seqlens[n + 1];
        const int slot = slot_idx ? slot_idx[n] : n;
        if (slot < 0 || slot >= num_slots) {
            if (slot >= num_slots) bad.fetch_add(1);
            for (int t = t0; t < t1; ++t) {
                double* o_row = o + (static_cast<size_t>(t) * Hv + hv) * dv;
                for (int j = 0; j < dv; ++j) o_row[j] = 0.0;
            }
            return;
        }
        std::vector<double> S(tile, 0.0), kd(dk), qd(dk);
        if (init_state) {
            const double* src = init_state + (static_cast<size_t>(slot) * Hv + hv) * tile;
            std::copy(src, src + tile, S.begin());
        }
        for (int t = t0; t < t1; ++t) {
            gated_delta_step(S.data(),
                             q + (static_cast<size_t>(t) * Hqk + hqk) * dk,
                             k + (static_cast<size_t>(t) * Hqk + hqk) * dk,
                             v + (static_cast<size_t>(t) * Hv + hv) * dv,
                             g[static_cast<size_t>(t) * Hv + hv],
                             beta[static_cast<size_t>(t) * Hv + hv],
                             scale, dk, dv,
                             o + (static_cast<size_t>(t) * Hv + hv) * dv,
                             kd.data(), qd.data());
        }
        double* dst = final_state + (static_cast<size_t>(slot) * Hv + hv) * tile;
        std::copy(S.begin(), S.end(), dst);
    });
    return bad.load();
}

}  // extern "C"
