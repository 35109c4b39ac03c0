// extern "C" boundary of the sr_gate library: argument validation and dispatch.
// Every argument check runs on the host before anything is enqueued, so a validation
// error guarantees that no buffer was touched; only SR_ERR_CUDA (a failed CUDA call or
// launch) can arrive after earlier work of the same call is already on the stream.
#include <stdio.h>
#include <string.h>

#include "common.cuh"
#include "sr_probe.h"

namespace sr {

static thread_local char g_cuda_error[256] = "no CUDA error recorded";

void note_cuda_error(cudaError_t e, const char* where) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s (%s)", where, cudaGetErrorName(e),
             cudaGetErrorString(e));
}

int check_gate_args(const int32_t* seqs, int32_t n_groups, int32_t N, int32_t stride,
                           int32_t K, int32_t norm_mode, const uint8_t* stop) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (stride < 0 || K < 0 || K > stride || K > SR_MAX_K) return SR_ERR_BAD_K;
    if (norm_mode != SR_NORM_MAXLEN && norm_mode != SR_NORM_NONE) return SR_ERR_BAD_MODE;
    if (n_groups > 0 && (seqs == nullptr || stop == nullptr)) return SR_ERR_NULL;
    if ((stride & 3) != 0 || (reinterpret_cast<uintptr_t>(seqs) & 15) != 0) return SR_ERR_ALIGN;
    return SR_OK;
}

HostArena host_arena(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    HostArena h;
    const size_t P = pairs_of(N);
    size_t off = 0;
    h.off_seqs = off;   off = align_up(off + (size_t)n_groups * N * stride * 4, 256);
    h.off_lens = off;   off = align_up(off + (size_t)n_groups * N * 4, 256);
    h.off_dist = off;   off = align_up(off + (size_t)n_groups * P * 4, 256);
    h.off_sum = off;    off = align_up(off + (size_t)n_groups * 4, 256);
    h.off_mean = off;   off = align_up(off + (size_t)n_groups * 8, 256);
    h.off_stop = off;   off = align_up(off + (size_t)n_groups, 256);
    h.off_status = off; off = align_up(off + 4, 256);
    h.off_ws = off;     off += sr_gate_workspace_bytes(n_groups, N, stride, K);
    h.total = align_up(off, 256);
    return h;
}

}  // namespace sr

using namespace sr;

extern "C" {

int sr_version(void) { return SR_VERSION; }

const char* sr_strerror(int code) {
    switch (code) {
        case SR_OK: return "ok";
        case SR_ERR_NULL: return "a required pointer is NULL";
        case SR_ERR_BAD_N: return "N outside 2..32 or negative group count";
        case SR_ERR_BAD_K: return "K / stride / max_steps out of range";
        case SR_ERR_ALIGN: return "seqs must be 16-byte aligned and stride a multiple of 4";
        case SR_ERR_STATE_SIZE: return "incremental state buffer too small";
        case SR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case SR_ERR_CUDA: return "a CUDA call failed (see sr_last_cuda_error)";
        case SR_ERR_BAD_MODE: return "unknown norm_mode";
        case SR_ERR_SCRATCH_LIMIT: return "problem needs more scratch than sr_gate_noalloc's built-in array";
        case SR_ERR_BAD_OFFSETS: return "row_start does not begin at 0, decreases, or exceeds rows x stride symbols";
        default: return "unknown error code";
    }
}

const char* sr_last_cuda_error(void) { return g_cuda_error; }

size_t sr_gate_workspace_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N || K < 0 || K > stride || K > SR_MAX_K) return 0;
    if (K <= 32) return 0;
    return gate_multi_workspace_bytes(n_groups, N, stride, K);
}

int sr_gate(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N, int32_t stride,
            int32_t K, double threshold, int32_t norm_mode, int32_t* pair_dist, int32_t* pair_sum,
            double* mean, uint8_t* stop, int32_t* status, void* workspace, size_t workspace_bytes,
            void* stream) {
    const int rc = check_gate_args(seqs, n_groups, N, stride, K, norm_mode, stop);
    if (rc != SR_OK) return rc;
    GateArgs a{seqs, lens, n_groups, N, stride, K, threshold, norm_mode,
               pair_dist, pair_sum, mean, stop, status};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (K <= 32) return launch_gate_single(a, s);
    if (n_groups > 0) {
        const size_t need = gate_multi_workspace_bytes(n_groups, N, stride, K);
        if (workspace == nullptr || workspace_bytes < need ||
            (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
            return SR_ERR_WORKSPACE;
    }
    return launch_gate_multi(a, workspace, workspace_bytes, s);
}

int sr_gate_decide(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                   int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                   int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                   uint8_t* exact, int32_t* status, void* workspace, size_t workspace_bytes,
                   void* stream) {
    const int rc = check_gate_args(seqs, n_groups, N, stride, K, norm_mode, stop);
    if (rc != SR_OK) return rc;
    GateArgs a{seqs, lens, n_groups, N, stride, K, threshold, norm_mode,
               pair_dist, pair_sum, mean, stop, status};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (K <= 32 || n_groups == 0) {
        if (exact && n_groups > 0) SR_CUDA_TRY(cudaMemsetAsync(exact, 1, (size_t)n_groups, s));
        return K <= 32 ? launch_gate_single(a, s) : SR_OK;
    }
    const size_t need = gate_multi_workspace_bytes(n_groups, N, stride, K);
    if (workspace == nullptr || workspace_bytes < need ||
        (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
        return SR_ERR_WORKSPACE;
    return launch_gate_multi(a, workspace, workspace_bytes, s, nullptr, true, exact);
}

int sr_gate_stages(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                   int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                   int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                   int32_t* status, void* workspace, size_t workspace_bytes, void* stream,
                   void* const* events) {
    if (events == nullptr) return SR_ERR_NULL;
    for (int k = 0; k < 5; ++k)
        if (events[k] == nullptr) return SR_ERR_NULL;
    const int rc = check_gate_args(seqs, n_groups, N, stride, K, norm_mode, stop);
    if (rc != SR_OK) return rc;
    GateArgs a{seqs, lens, n_groups, N, stride, K, threshold, norm_mode,
               pair_dist, pair_sum, mean, stop, status};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaEvent_t ev[5];
    for (int k = 0; k < 5; ++k) ev[k] = static_cast<cudaEvent_t>(events[k]);
    if (K <= 32 || n_groups == 0) {
        SR_CUDA_TRY(cudaEventRecord(ev[0], s));
        const int r = (K <= 32) ? launch_gate_single(a, s) : SR_OK;
        if (r != SR_OK) return r;
        for (int k = 1; k < 5; ++k) SR_CUDA_TRY(cudaEventRecord(ev[k], s));
        return SR_OK;
    }
    const size_t need = gate_multi_workspace_bytes(n_groups, N, stride, K);
    if (workspace == nullptr || workspace_bytes < need ||
        (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
        return SR_ERR_WORKSPACE;
    return launch_gate_multi(a, workspace, workspace_bytes, s, ev);
}

size_t sr_gate_host_arena_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N || stride < 0 || K < 0 || K > stride || K > SR_MAX_K)
        return 0;
    return host_arena(n_groups, N, stride, K).total;
}

int sr_gate_host(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                 int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                 int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                 int32_t* status, void* arena, size_t arena_bytes, void* stream,
                 void* copy_stream) {
    // the alignment rule applies to the device copy, which the arena guarantees
    const int32_t* aligned_stand_in = seqs ? reinterpret_cast<const int32_t*>(uintptr_t(256)) : nullptr;
    int rc = check_gate_args(aligned_stand_in, n_groups, N, stride, K, norm_mode, stop);
    if (rc != SR_OK) return rc;
    if (n_groups == 0) return SR_OK;
    const HostArena h = host_arena(n_groups, N, stride, K);
    if (arena == nullptr || arena_bytes < h.total || (reinterpret_cast<uintptr_t>(arena) & 255) != 0)
        return SR_ERR_WORKSPACE;
    unsigned char* d = static_cast<unsigned char*>(arena);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
    const size_t P = pairs_of(N);
    // With a copy stream the batch goes over in chunks: the input copy of chunk c+1
    // overlaps the kernels of chunk c (which run one after the other on `stream` and so
    // can share the workspace).
    const bool overlap = cs != nullptr && cs != s && n_groups >= 64;
    const int chunks = overlap ? 4 : 1;
    cudaStream_t in_stream = overlap ? cs : s;
    if (status)
        SR_CUDA_TRY(cudaMemcpyAsync(d + h.off_status, status, 4, cudaMemcpyHostToDevice, s));
    cudaEvent_t ev = nullptr;
    if (overlap) {       // the copies must not overtake earlier work on `stream` that uses the arena
        SR_CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
        SR_CUDA_TRY(cudaEventRecord(ev, s));
        SR_CUDA_TRY(cudaStreamWaitEvent(cs, ev, 0));
        SR_CUDA_TRY(cudaEventDestroy(ev));               // released once it has completed
    }
    for (int c = 0; c < chunks; ++c) {
        const int32_t g0 = (int32_t)((long long)n_groups * c / chunks);
        const int32_t g1 = (int32_t)((long long)n_groups * (c + 1) / chunks);
        const int32_t ng = g1 - g0;
        if (ng == 0) continue;
        const size_t row0 = (size_t)g0 * N;
        SR_CUDA_TRY(cudaMemcpyAsync(d + h.off_seqs + row0 * stride * 4, seqs + row0 * stride,
                                    (size_t)ng * N * stride * 4, cudaMemcpyHostToDevice, in_stream));
        if (lens)
            SR_CUDA_TRY(cudaMemcpyAsync(d + h.off_lens + row0 * 4, lens + row0, (size_t)ng * N * 4,
                                        cudaMemcpyHostToDevice, in_stream));
        if (overlap) {
            SR_CUDA_TRY(cudaEventCreateWithFlags(&ev, cudaEventDisableTiming));
            SR_CUDA_TRY(cudaEventRecord(ev, cs));
            SR_CUDA_TRY(cudaStreamWaitEvent(s, ev, 0));
            SR_CUDA_TRY(cudaEventDestroy(ev));
        }
        rc = sr_gate(reinterpret_cast<const int32_t*>(d + h.off_seqs) + row0 * stride,
                     lens ? reinterpret_cast<const int32_t*>(d + h.off_lens) + row0 : nullptr, ng, N,
                     stride, K, threshold, norm_mode,
                     pair_dist ? reinterpret_cast<int32_t*>(d + h.off_dist) + (size_t)g0 * P : nullptr,
                     pair_sum ? reinterpret_cast<int32_t*>(d + h.off_sum) + g0 : nullptr,
                     mean ? reinterpret_cast<double*>(d + h.off_mean) + g0 : nullptr,
                     d + h.off_stop + g0,
                     status ? reinterpret_cast<int32_t*>(d + h.off_status) : nullptr, d + h.off_ws,
                     h.total - h.off_ws, stream);
        if (rc != SR_OK) return rc;
    }
    if (pair_dist)
        SR_CUDA_TRY(cudaMemcpyAsync(pair_dist, d + h.off_dist, (size_t)n_groups * P * 4,
                                    cudaMemcpyDeviceToHost, s));
    if (pair_sum)
        SR_CUDA_TRY(cudaMemcpyAsync(pair_sum, d + h.off_sum, (size_t)n_groups * 4,
                                    cudaMemcpyDeviceToHost, s));
    if (mean)
        SR_CUDA_TRY(cudaMemcpyAsync(mean, d + h.off_mean, (size_t)n_groups * 8,
                                    cudaMemcpyDeviceToHost, s));
    SR_CUDA_TRY(cudaMemcpyAsync(stop, d + h.off_stop, (size_t)n_groups, cudaMemcpyDeviceToHost, s));
    if (status)
        SR_CUDA_TRY(cudaMemcpyAsync(status, d + h.off_status, 4, cudaMemcpyDeviceToHost, s));
    return SR_OK;
}

size_t sr_incr_state_bytes(int32_t n_groups, int32_t N, int32_t max_steps) {
    return incr_state_bytes(n_groups, N, max_steps);
}

int sr_incr_init(void* state, size_t state_bytes, int32_t n_groups, int32_t N, int32_t max_steps,
                 void* stream) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (max_steps < 1 || max_steps > SR_MAX_INCR_STEPS) return SR_ERR_BAD_K;
    if (state == nullptr) return SR_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(state) & 15) != 0) return SR_ERR_ALIGN;
    return launch_incr_init(state, state_bytes, n_groups, N, max_steps,
                            static_cast<cudaStream_t>(stream));
}

int sr_gate_step_incremental(void* state, size_t state_bytes, const int32_t* new_actions,
                             int32_t n_groups, int32_t N, double threshold, int32_t norm_mode,
                             int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                             int32_t* status, void* stream) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (norm_mode != SR_NORM_MAXLEN && norm_mode != SR_NORM_NONE) return SR_ERR_BAD_MODE;
    if (state == nullptr) return SR_ERR_NULL;
    if (n_groups > 0 && (new_actions == nullptr || stop == nullptr)) return SR_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(state) & 15) != 0) return SR_ERR_ALIGN;
    return launch_incr_step(state, state_bytes, new_actions, n_groups, N, threshold, norm_mode,
                            pair_dist, pair_sum, mean, stop, status,
                            static_cast<cudaStream_t>(stream));
}

int sr_gate_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                    int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                    uint8_t* stop, void* stream) {
    if (n_groups < 0 || N < 1 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (K < 0) return SR_ERR_BAD_K;
    if (n_groups > 0 && (mean == nullptr || stop == nullptr || (lens == nullptr && done == nullptr)))
        return SR_ERR_NULL;
    return launch_or_rule(mean, lens, done, n_groups, N, K, threshold, tau_high, tau, stop,
                          static_cast<cudaStream_t>(stream));
}

int sr_group_signals(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                     int32_t stride, int32_t K, double* unique_prefix_ratio,
                     double* unique_action_ratio, double* action_entropy,
                     double* bigram_jaccard_mean, void* stream) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (stride < 0 || K < 0 || K > stride || K > 32) return SR_ERR_BAD_K;
    if (n_groups > 0 && seqs == nullptr) return SR_ERR_NULL;
    if ((stride & 3) != 0 || (reinterpret_cast<uintptr_t>(seqs) & 15) != 0) return SR_ERR_ALIGN;
    return launch_group_signals(seqs, lens, n_groups, N, stride, K, unique_prefix_ratio,
                                unique_action_ratio, action_entropy, bigram_jaccard_mean,
                                static_cast<cudaStream_t>(stream));
}

int sr_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                   int64_t* counts, double* sumsq, void* stream) {
    if (n_groups < 0 || N < 1 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (counts == nullptr || sumsq == nullptr || (n_groups > 0 && adv == nullptr)) return SR_ERR_NULL;
    return launch_batch_stats(adv, stop, n_groups, N, counts, sumsq, static_cast<cudaStream_t>(stream));
}

size_t sr_kept_groups_workspace_bytes(int32_t n_groups) {
    if (n_groups < 0) return 0;
    return kept_groups_workspace_bytes(n_groups);
}

int sr_kept_groups(const uint8_t* stop, const uint8_t* zero_var, int32_t n_groups, int32_t* index,
                   int32_t* count, void* workspace, size_t workspace_bytes, void* stream) {
    if (n_groups < 0) return SR_ERR_BAD_N;
    if (count == nullptr || (n_groups > 0 && index == nullptr)) return SR_ERR_NULL;
    if (n_groups > 0 && (workspace == nullptr || workspace_bytes < kept_groups_workspace_bytes(n_groups) ||
                         (reinterpret_cast<uintptr_t>(workspace) & 15) != 0))
        return SR_ERR_WORKSPACE;
    return launch_kept_groups(stop, zero_var, n_groups, index, count, workspace,
                              static_cast<cudaStream_t>(stream));
}

double sr_savings_fraction(int64_t cut, int64_t n_groups, int32_t T_max, int32_t K) {
    if (n_groups <= 0 || T_max <= 0) return 0.0;
    return (double)(cut * (int64_t)(T_max - K)) / (double)(n_groups * (int64_t)T_max);
}

double sr_dilution_gain(double zero_frac_before, double zero_frac_after) {
    return (1.0 - zero_frac_after) / (1.0 - zero_frac_before);
}

int sr_grpo_advantage(const float* rewards, const uint8_t* drop_mask, int32_t n_groups, int32_t N,
                      float eps, float* adv, uint8_t* zero_var, void* stream) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (n_groups > 0 && (rewards == nullptr || adv == nullptr)) return SR_ERR_NULL;
    return launch_advantage(rewards, drop_mask, n_groups, N, eps, adv, zero_var,
                            static_cast<cudaStream_t>(stream));
}

}  // extern "C"
