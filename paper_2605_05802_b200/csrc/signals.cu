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

// The other action-only signals of Appendix B.  One CTA per group: the prefixes are
// staged once in shared memory (rows of 33 words); one thread per (rollout, position)
// marks the first occurrence of every bigram of a rollout; one thread per rollout does
// the prefix / step-K-action comparisons; one thread per pair counts the common bigrams;
// thread 0 adds everything up in a fixed order.
__global__ void __launch_bounds__(512)
group_signals_kernel(const int32_t* __restrict__ seqs, const int32_t* __restrict__ lens, int N,
                     int stride, int K, double* upr, double* uar, double* ent, double* jac) {
    __shared__ int32_t s_sym[SR_MAX_N * 33];
    __shared__ int32_t s_len[SR_MAX_N], s_raw[SR_MAX_N];
    __shared__ uint32_t s_first[SR_MAX_N];          // bit t: bigram (t, t+1) is new in its rollout
    __shared__ int32_t s_fp[SR_MAX_N], s_fa[SR_MAX_N], s_same[SR_MAX_N];
    __shared__ double s_term[SR_MAX_N * (SR_MAX_N - 1) / 2];
    const int g = blockIdx.x, tid = threadIdx.x, nthr = blockDim.x;
    const int P = pairs_of(N);
    for (int i = tid; i < N; i += nthr) {
        const int raw = lens ? lens[(size_t)g * N + i] : K;
        s_raw[i] = raw;
        s_len[i] = min(max(raw, 0), K);
        s_first[i] = 0u;
    }
    const int q4 = (K + 3) >> 2;
    for (int e = tid; e < N * 8; e += nthr) {
        const int i = e >> 3, q = e & 7;
        if (q < q4) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(seqs + ((size_t)g * N + i) * stride) + q);
            int32_t* d = s_sym + i * 33 + 4 * q;
            d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
        }
    }
    __syncthreads();
    for (int e = tid; e < N * 32; e += nthr) {
        const int i = e >> 5, t = e & 31;
        const int32_t* a = s_sym + i * 33;
        if (t + 1 < s_len[i]) {
            bool seen = false;
            for (int u = 0; u < t; ++u) seen |= (a[u] == a[t]) & (a[u + 1] == a[t + 1]);
            if (!seen) atomicOr(&s_first[i], 1u << t);
        }
    }
    for (int i = tid; i < N; i += nthr) {
        const int mi = s_len[i];
        const bool has_i = s_raw[i] >= K && K >= 1;
        const int32_t* a = s_sym + i * 33;
        int first_p = 1, first_a = 1, same_a_cnt = 0;
        for (int j = 0; j < N; ++j) {
            const int32_t* b = s_sym + j * 33;
            bool same_p = mi == s_len[j];
            for (int r = 0; same_p && r < mi; ++r) same_p = a[r] == b[r];
            const bool has_j = s_raw[j] >= K && K >= 1;
            const bool same_a = has_i == has_j && (!has_i || a[K - 1] == b[K - 1]);
            if (j < i && same_p) first_p = 0;
            if (j < i && same_a) first_a = 0;
            same_a_cnt += same_a;
        }
        s_fp[i] = first_p; s_fa[i] = first_a; s_same[i] = same_a_cnt;
    }
    __syncthreads();
    if (jac) {
        for (int p = tid; p < P; p += nthr) {
            int i, j;
            pair_from_index(p, N, i, j);
            const int32_t* a = s_sym + i * 33;
            const int32_t* b = s_sym + j * 33;
            const int nbj = s_len[j] - 1;
            int both = 0;
            uint32_t todo = s_first[i];
            while (todo) {
                const int t = __ffs(todo) - 1;
                todo &= todo - 1;
                bool hit = false;
                for (int u = 0; u < nbj; ++u) hit |= (b[u] == a[t]) & (b[u + 1] == a[t + 1]);
                both += hit;
            }
            const int uni = __popc(s_first[i]) + __popc(s_first[j]) - both;
            s_term[p] = uni > 0 ? __dsub_rn(1.0, __ddiv_rn((double)both, (double)uni)) : 0.0;
        }
    }
    __syncthreads();
    if (tid == 0) {
        int dp = 0, da = 0;
        double h = 0.0;
        for (int i = 0; i < N; ++i) {
            dp += s_fp[i];
            da += s_fa[i];
            if (s_fa[i]) {
                const double pr = __ddiv_rn((double)s_same[i], (double)N);
                h = __dsub_rn(h, __dmul_rn(pr, log(pr)));
            }
        }
        if (upr) upr[g] = __ddiv_rn((double)dp, (double)N);
        if (uar) uar[g] = __ddiv_rn((double)da, (double)N);
        if (ent) ent[g] = __ddiv_rn(h, log((double)N));
        if (jac) {
            double s = 0.0;
            for (int p = 0; p < P; ++p) s = __dadd_rn(s, s_term[p]);
            jac[g] = __ddiv_rn(s, (double)P);
        }
    }
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

int launch_group_signals(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                         int32_t stride, int32_t K, double* upr, double* uar, double* ent,
                         double* jac, cudaStream_t s) {
    if (n_groups == 0) return SR_OK;
    int threads = (max(pairs_of(N), N * 8) + 31) & ~31;
    if (threads < 64) threads = 64;
    if (threads > 512) threads = 512;
    group_signals_kernel<<<n_groups, threads, 0, s>>>(seqs, lens, N, stride, K, upr, uar, ent, jac);
    SR_LAUNCH_CHECK("group_signals_kernel");
    return SR_OK;
}

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
