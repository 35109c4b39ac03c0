// Further per-group signals of the paper's Appendix B and the OR-rule extension.
#include "common.cuh"

namespace sr {
namespace {

// tau_K and Cut = [d_K < d_L] or [tau_K >= tau_H] (Eq. 3): one thread per group, N <= 32
// flags or lengths each.  A few bytes per rollout: bound by HBM bandwidth / launch latency.
__global__ void __launch_bounds__(256)
or_rule_kernel(const double* __restrict__ mean, const int32_t* __restrict__ lens,
               const uint8_t* __restrict__ done, int n_groups, int N, int K, double threshold,
               double tau_high, double* __restrict__ tau, uint8_t* __restrict__ stop) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_groups) return;
    int finished = 0;
    for (int i = 0; i < N; ++i) {
        const size_t idx = (size_t)g * N + i;
        finished += done ? (done[idx] != 0) : (lens[idx] < K);
    }
    const double t = __ddiv_rn((double)finished, (double)N);
    if (tau) tau[g] = t;
    stop[g] = (mean[g] < threshold || t >= tau_high) ? 1 : 0;
}

// Batch reductions (Section 4.5 dilution, Section 3.4 norm kept): grid-stride over the
// trajectories, fp64 partial sums per thread, warp shuffles, one atomic per warp.
__global__ void __launch_bounds__(256)
batch_stats_kernel(const float* __restrict__ adv, const uint8_t* __restrict__ stop, long long n_traj,
                   int N, int n_groups, unsigned long long* counts, double* sumsq) {
    double ss_all = 0.0, ss_kept = 0.0;
    unsigned z_all = 0, z_kept = 0, kept_groups = 0;
    const long long stride = (long long)gridDim.x * blockDim.x;
    const long long t0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (long long t = t0; t < n_traj; t += stride) {
        const int g = (int)(t / N);
        const bool kept = !(stop && stop[g]);
        const double a = (double)__ldg(adv + t);
        const bool zero = a == 0.0;
        const double sq = __dmul_rn(a, a);
        ss_all += sq;
        z_all += zero;
        if (kept) { ss_kept += sq; z_kept += zero; }
    }
    for (long long g = t0; g < n_groups; g += stride) kept_groups += !(stop && stop[g]);
    for (int off = 16; off > 0; off >>= 1) {
        ss_all += __shfl_xor_sync(0xFFFFFFFFu, ss_all, off);
        ss_kept += __shfl_xor_sync(0xFFFFFFFFu, ss_kept, off);
        z_all += __shfl_xor_sync(0xFFFFFFFFu, z_all, off);
        z_kept += __shfl_xor_sync(0xFFFFFFFFu, z_kept, off);
        kept_groups += __shfl_xor_sync(0xFFFFFFFFu, kept_groups, off);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicAdd(&sumsq[0], ss_all);
        atomicAdd(&sumsq[1], ss_kept);
        atomicAdd(&counts[0], (unsigned long long)z_all);
        atomicAdd(&counts[1], (unsigned long long)z_kept);
        atomicAdd(&counts[2], (unsigned long long)kept_groups);
    }
}

}  // namespace

int launch_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                       int64_t* counts, double* sumsq, cudaStream_t s) {
    SR_CUDA_TRY(cudaMemsetAsync(counts, 0, 3 * sizeof(int64_t), s));
    SR_CUDA_TRY(cudaMemsetAsync(sumsq, 0, 2 * sizeof(double), s));
    if (n_groups == 0) return SR_OK;
    const long long n_traj = (long long)n_groups * N;
    int dev = 0, sms = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    SR_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    long long want = (n_traj + 255) / 256;
    const long long cap = (long long)sms * 8;
    const int blocks = (int)(want < cap ? want : cap);
    batch_stats_kernel<<<blocks, 256, 0, s>>>(adv, stop, n_traj, N, n_groups,
                                              reinterpret_cast<unsigned long long*>(counts), sumsq);
    SR_LAUNCH_CHECK("batch_stats_kernel");
    return SR_OK;
}

int launch_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                   int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                   uint8_t* stop, cudaStream_t s) {
    if (n_groups == 0) return SR_OK;
    or_rule_kernel<<<(n_groups + 255) / 256, 256, 0, s>>>(mean, lens, done, n_groups, N, K, threshold,
                                                          tau_high, tau, stop);
    SR_LAUNCH_CHECK("or_rule_kernel");
    return SR_OK;
}

}  // namespace sr
