// Shared declarations of the sr_gate CUDA library (internal; the public boundary is include/sr_gate.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "sr_gate.h"

namespace sr {

// Records the text of a failed CUDA call for sr_last_cuda_error().
void note_cuda_error(cudaError_t e, const char* where);

#define SR_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t e__ = (expr);                           \
        if (e__ != cudaSuccess) {                           \
            ::sr::note_cuda_error(e__, #expr);              \
            return SR_ERR_CUDA;                             \
        }                                                   \
    } while (0)

// Launch-error check that does not synchronise.
#define SR_LAUNCH_CHECK(name)                               \
    do {                                                    \
        cudaError_t e__ = cudaGetLastError();               \
        if (e__ != cudaSuccess) {                           \
            ::sr::note_cuda_error(e__, name);               \
            return SR_ERR_CUDA;                             \
        }                                                   \
    } while (0)

struct GateArgs {
    const int32_t* seqs;
    const int32_t* lens;
    int32_t n_groups, N, stride, K;
    double threshold;
    int32_t norm_mode;
    int32_t* pair_dist;
    int32_t* pair_sum;
    double* mean;
    uint8_t* stop;
    int32_t* status;
};

__host__ __device__ inline int pairs_of(int N) { return N * (N - 1) / 2; }

// Index of pair (a, b), a < b, in the order (0,1),(0,2),...,(N-2,N-1).
__host__ __device__ inline int pair_index(int a, int b, int N) {
    return a * N - a * (a + 1) / 2 + (b - a - 1);
}

// Inverse of pair_index.
__device__ inline void pair_from_index(int p, int N, int& a, int& b) {
    int i = 0, rem = p, row = N - 1;
    while (rem >= row) { rem -= row; --row; ++i; }
    a = i;
    b = i + 1 + rem;
}

__device__ __forceinline__ uint32_t low_mask(int m) {   // m in 0..32
    return m >= 32 ? 0xFFFFFFFFu : ((1u << m) - 1u);
}

// One term of the d_K sum (Section 3.2): the pair distance divided by the longer
// prefix length, 0 for two empty prefixes; the raw distance in SR_NORM_NONE.
__device__ __forceinline__ double pair_term(int d, int mi, int mj, int norm_mode) {
    if (norm_mode == SR_NORM_NONE) return (double)d;
    const int longer = mi > mj ? mi : mj;
    return longer > 0 ? __ddiv_rn((double)d, (double)longer) : 0.0;
}

// d / L for 0 <= d, L <= 32 (0 when L == 0), correctly rounded: the compiler's constant
// evaluation of an IEEE division equals the device's __ddiv_rn.  Terms of d_K for
// prefixes of at most 32 symbols come from this table instead of a run-time division.
struct QuotientTable {
    double v[33 * 33];
    constexpr QuotientTable() : v() {
        for (int d = 0; d <= 32; ++d)
            for (int l = 0; l <= 32; ++l) v[d * 33 + l] = l > 0 ? (double)d / (double)l : 0.0;
    }
};
__device__ const QuotientTable kQuot = QuotientTable();

// (i, j) of pair p, as i | j << 8, for every group size: filled in at compile time.
struct PairTable {
    uint16_t v[SR_MAX_N + 1][SR_MAX_N * (SR_MAX_N - 1) / 2];
    constexpr PairTable() : v() {
        for (int n = 2; n <= SR_MAX_N; ++n) {
            int p = 0;
            for (int i = 0; i < n; ++i)
                for (int j = i + 1; j < n; ++j) v[n][p++] = (uint16_t)(i | (j << 8));
        }
    }
};
__device__ const PairTable kPairs = PairTable();

// One column of the bit-vector edit-distance recurrence on a single 32-bit word of
// vertical deltas (Pv: +1, Mv: -1), horizontal input +1 at row 0.  `Ph` / `Mh` return the
// horizontal delta words BEFORE the shift (bit r = delta leaving row r).
__device__ __forceinline__ void word_column(uint32_t Eq, uint32_t& Pv, uint32_t& Mv,
                                            uint32_t& Ph, uint32_t& Mh) {
    const uint32_t Xv = Eq | Mv;
    const uint32_t Xh = (((Eq & Pv) + Pv) ^ Pv) | Eq;
    Ph = Mv | ~(Xh | Pv);
    Mh = Pv & Xh;
    const uint32_t Phs = (Ph << 1) | 1u;
    const uint32_t Mhs = Mh << 1;
    Pv = Mhs | ~(Xv | Phs);
    Mv = Phs & Xv;
}

// Ordered fp64 sum of the P terms of a group (pair order), the integer sum of the raw
// distances, the division by P and the strict comparison of Eq. 2, by one thread.  The
// loads run eight ahead of the (necessarily sequential) additions.
__device__ __forceinline__ void group_sum_and_gate(const double* term, const int32_t* dist, int P,
                                                   const GateArgs& a, size_t g) {
    double s = 0.0;
    int isum = 0, p = 0;
    for (; p + 8 <= P; p += 8) {
        double t[8];
        int d[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) { t[u] = term[p + u]; d[u] = dist[p + u]; }
#pragma unroll
        for (int u = 0; u < 8; ++u) { s = __dadd_rn(s, t[u]); isum += d[u]; }
    }
    for (; p < P; ++p) { s = __dadd_rn(s, term[p]); isum += dist[p]; }
    const double dk = __ddiv_rn(s, (double)P);
    if (a.pair_sum) a.pair_sum[g] = isum;
    if (a.mean) a.mean[g] = dk;
    a.stop[g] = dk < a.threshold ? 1 : 0;
}

size_t align_up(size_t x, size_t a);

// api.cu: the argument rules shared by every gate entry point (SR_OK or an SR_ERR_* code).
int check_gate_args(const int32_t* seqs, int32_t n_groups, int32_t N, int32_t stride, int32_t K,
                    int32_t norm_mode, const uint8_t* stop);

// Device arena of the host-buffer entry points (api.cu): staged inputs, outputs, gate workspace.
struct HostArena {
    size_t off_seqs, off_lens, off_dist, off_sum, off_mean, off_stop, off_status, off_ws, total;
};
HostArena host_arena(int32_t n_groups, int32_t N, int32_t stride, int32_t K);

// gate_single.cu: prefixes of at most 32 symbols, one 32-bit word per pair.
int launch_gate_single(const GateArgs& a, cudaStream_t s);
// gate_multi.cu: prefixes of up to SR_MAX_K symbols, blocked multi-word.
size_t gate_multi_workspace_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K);
// `ev`: NULL, or 5 events recorded before prep / after prep / after scan+scatter /
// after dp / after finish.
// `decide`: finish groups whose lower-bounded d_K already reaches the threshold without
// running their pairs; `exact` (may be NULL) then receives 1 per group computed exactly.
// `feed`: NULL, or the groups become ready on the stream in `pieces` pieces: before the
// per-group pass of piece [g0, g1) is enqueued, `before(ctx, g0, g1, s)` is called to
// enqueue what makes those groups' inputs valid (a wait on a copy, an unpacking kernel).
struct GroupFeed {
    int pieces;
    int (*before)(void* ctx, int g0, int g1, cudaStream_t s);
    void* ctx;
};
int launch_gate_multi(const GateArgs& a, void* ws, size_t ws_bytes, cudaStream_t s,
                      const cudaEvent_t* ev = nullptr, bool decide = false, uint8_t* exact = nullptr,
                      const GroupFeed* feed = nullptr);
// incremental.cu
size_t incr_state_bytes(int32_t n_groups, int32_t N, int32_t max_steps);
int launch_incr_init(void* state, size_t bytes, int32_t n_groups, int32_t N, int32_t max_steps,
                     cudaStream_t s);
int launch_incr_step(void* state, size_t bytes, const int32_t* new_actions, int32_t n_groups,
                     int32_t N, double threshold, int32_t norm_mode, int32_t* pair_dist,
                     int32_t* pair_sum, double* mean, uint8_t* stop, int32_t* status,
                     cudaStream_t s);
// advantage.cu
int launch_advantage(const float* rewards, const uint8_t* drop_mask, int32_t n_groups, int32_t N,
                     float eps, float* adv, uint8_t* zero_var, cudaStream_t s);

// signals.cu
int launch_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                   int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                   uint8_t* stop, cudaStream_t s);

int launch_group_signals(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                         int32_t stride, int32_t K, double* upr, double* uar, double* ent,
                         double* jac, cudaStream_t s);
int launch_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                       int64_t* counts, double* sumsq, cudaStream_t s);

// compact.cu
size_t kept_groups_workspace_bytes(int32_t n_groups);
int launch_kept_groups(const uint8_t* stop, const uint8_t* zero_var, int32_t n_groups,
                       int32_t* index, int32_t* count, void* ws, cudaStream_t s);

}  // namespace sr
