// Group-relative advantages, Eq. 1 of the paper, with the zero-variance flag of
// Section 2.1.  One thread per group: the N rewards are read with vector loads,
// mean and population variance are accumulated in fp64 in index order (explicit
// round-to-nearest adds and multiplies, no fused multiply-add), every centred reward is
// multiplied by the fp64 reciprocal of sigma + eps, and the result is rounded once to fp32.  The kernel moves 8 bytes per rollout plus 1-2 per group and
// is bound by HBM bandwidth.
#include "common.cuh"

namespace sr {
namespace {

template <int NT>   // NT > 0: compile-time N; NT == 0: runtime N
__global__ void __launch_bounds__(256)
advantage_kernel(const float* __restrict__ rewards, const uint8_t* __restrict__ drop_mask,
                 int n_groups, int n_rt, float eps, float* __restrict__ adv,
                 uint8_t* __restrict__ zero_var) {
    const int N = NT > 0 ? NT : n_rt;
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_groups) return;
    float r[NT > 0 ? NT : SR_MAX_N];
    const float* src = rewards + (size_t)g * N;
    if (NT > 0 && NT % 4 == 0) {
#pragma unroll
        for (int q = 0; q < NT / 4; ++q) {
            const float4 v = __ldg(reinterpret_cast<const float4*>(src) + q);
            r[4 * q] = v.x; r[4 * q + 1] = v.y; r[4 * q + 2] = v.z; r[4 * q + 3] = v.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < (NT > 0 ? NT : SR_MAX_N); ++i)
            if (i < N) r[i] = __ldg(src + i);
    }
    bool equal = (r[0] == r[0]);
#pragma unroll
    for (int i = 1; i < (NT > 0 ? NT : SR_MAX_N); ++i)
        if (i < N) equal = equal && (r[i] == r[0]);
    if (zero_var) zero_var[g] = equal ? 1 : 0;
    const bool zero = equal || (drop_mask && drop_mask[g]);
    double rbar = 0.0, inv = 1.0;
    if (!zero) {
        double sum = 0.0;
#pragma unroll
        for (int i = 0; i < (NT > 0 ? NT : SR_MAX_N); ++i)
            if (i < N) sum = __dadd_rn(sum, (double)r[i]);
        rbar = __ddiv_rn(sum, (double)N);
        double ss = 0.0;
#pragma unroll
        for (int i = 0; i < (NT > 0 ? NT : SR_MAX_N); ++i)
            if (i < N) {
                const double d = __dsub_rn((double)r[i], rbar);
                ss = __dadd_rn(ss, __dmul_rn(d, d));
            }
        // one reciprocal of sigma + eps, then a multiplication per rollout: the fp64 product is
        // within one fp64 rounding of the quotient, far inside the fp32 result's own rounding
        inv = __ddiv_rn(1.0, __dadd_rn(__dsqrt_rn(__ddiv_rn(ss, (double)N)), (double)eps));
    }
    float out[NT > 0 ? NT : SR_MAX_N];
#pragma unroll
    for (int i = 0; i < (NT > 0 ? NT : SR_MAX_N); ++i)
        if (i < N) out[i] = zero ? 0.0f : (float)__dmul_rn(__dsub_rn((double)r[i], rbar), inv);
    float* dst = adv + (size_t)g * N;
    if (NT > 0 && NT % 4 == 0) {
#pragma unroll
        for (int q = 0; q < NT / 4; ++q)
            reinterpret_cast<float4*>(dst)[q] =
                make_float4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < (NT > 0 ? NT : SR_MAX_N); ++i)
            if (i < N) dst[i] = out[i];
    }
}

}  // namespace

int launch_advantage(const float* rewards, const uint8_t* drop_mask, int32_t n_groups, int32_t N,
                     float eps, float* adv, uint8_t* zero_var, cudaStream_t s) {
    if (n_groups == 0) return SR_OK;
    const int threads = 256;
    const int blocks = (n_groups + threads - 1) / threads;
    // the vector path needs 16-byte aligned rows
    const bool aligned = ((reinterpret_cast<uintptr_t>(rewards) | reinterpret_cast<uintptr_t>(adv)) & 15) == 0;
    if (N == 8 && aligned)
        advantage_kernel<8><<<blocks, threads, 0, s>>>(rewards, drop_mask, n_groups, N, eps, adv, zero_var);
    else if (N == 16 && aligned)
        advantage_kernel<16><<<blocks, threads, 0, s>>>(rewards, drop_mask, n_groups, N, eps, adv, zero_var);
    else
        advantage_kernel<0><<<blocks, threads, 0, s>>>(rewards, drop_mask, n_groups, N, eps, adv, zero_var);
    SR_LAUNCH_CHECK("advantage_kernel");
    return SR_OK;
}

}  // namespace sr
