// Further per-group signals of the paper's Appendix B and the OR-rule extension.
#include <math.h>

#include "common.cuh"

namespace sr {
namespace {

// tau_K and Cut = [d_K < d_L] or [tau_K >= tau_H] (Eq. 3): one thread per group, N <= 32
// flags or lengths each.  A few bytes per rollout: bound by HBM bandwidth / launch latency.
__global__ void __launch_bounds__(256)
or_rule_kernel(const double* __restrict__ mean, const int32_t* __restrict__ lens,
               const uint8_t* __restrict__ done, int n_groups, int N, int K, double threshold,
               double tau_high, bool vec4, double* __restrict__ tau, uint8_t* __restrict__ stop) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_groups) return;
    const double dk = mean[g];
    int finished = 0;
    if (vec4) {                                   // lengths only, rows 16-byte aligned
        const int4* row = reinterpret_cast<const int4*>(lens + (size_t)g * N);
        for (int q = 0; q < N / 4; ++q) {
            const int4 v = __ldg(row + q);
            finished += (v.x < K) + (v.y < K) + (v.z < K) + (v.w < K);
        }
    } else {
        for (int i = 0; i < N; ++i) {
            const size_t idx = (size_t)g * N + i;
            finished += done ? (done[idx] != 0) : (lens[idx] < K);
        }
    }
    const double t = __ddiv_rn((double)finished, (double)N);
    if (tau) tau[g] = t;
    stop[g] = (dk < threshold || t >= tau_high) ? 1 : 0;
}

// The other action-only signals of Appendix B.  One CTA per group: the prefixes are
// staged once in shared memory (rows of 33 words).  The bigrams of all rollouts are
// renamed to dense ids through an open-addressing table (as the gate does for symbols),
// every rollout gets a bit set over those ids, and the Jaccard term of a pair is a few
// popcounts of AND-ed words instead of K^2 comparisons.  One thread per rollout does
// the prefix / step-K-action comparisons; thread 0 adds everything up in a fixed order.
constexpr int kBgWords = 31;                    // 32 * 31 = 992 distinct bigrams at most
constexpr int kSymPitch = 36;                   // words per staged prefix: 32 + pad, rows 16-byte aligned

// Shared memory of a group, sized for the call's N and K (the arrays for 32 rollouts would
// keep an SM at 8 CTAs whatever the group size): byte offsets into dynamic shared memory.
struct SignalLayout {
    int off_term, off_plogp, off_sym, off_owner, off_bits, off_small, off_bid, off_slot;
    int words;                                  // words of a rollout's bigram bit set
    int total;
};

__global__ void __launch_bounds__(512)
group_signals_kernel(const int32_t* __restrict__ seqs, const int32_t* __restrict__ lens, int N,
                     int stride, int K, int slots, int slot_shift, double ln_n, SignalLayout L,
                     double* upr, double* uar, double* ent, double* jac) {
    extern __shared__ __align__(16) unsigned char smem[];
    double* s_term = reinterpret_cast<double*>(smem + L.off_term);          // [P]
    double* s_plogp = reinterpret_cast<double*>(smem + L.off_plogp);        // [N]
    int32_t* s_sym = reinterpret_cast<int32_t*>(smem + L.off_sym);          // [N][kSymPitch]
    uint32_t* s_owner = reinterpret_cast<uint32_t*>(smem + L.off_owner);    // [slots] element (i * 32 + t) + 1 that claimed the slot
    uint32_t* s_bits = reinterpret_cast<uint32_t*>(smem + L.off_bits);      // [N][kBgWords]
    int32_t* s_len = reinterpret_cast<int32_t*>(smem + L.off_small);        // 6 arrays of [N] and a counter
    int32_t* s_raw = s_len + N;
    int32_t* s_fp = s_raw + N;
    int32_t* s_fa = s_fp + N;
    int32_t* s_same = s_fa + N;
    int32_t* s_card = s_same + N;
    int& s_nbig = *(s_card + N);
    uint16_t* s_bid = reinterpret_cast<uint16_t*>(smem + L.off_bid);        // [slots] dense bigram id of a claimed slot
    uint16_t* s_slot = reinterpret_cast<uint16_t*>(smem + L.off_slot);      // [N * 32] slot of every element's bigram
    const int g = blockIdx.x, tid = threadIdx.x, nthr = blockDim.x;
    const int P = pairs_of(N);
    for (int i = tid; i < N; i += nthr) {
        const int raw = lens ? lens[(size_t)g * N + i] : K;
        s_raw[i] = raw;
        s_len[i] = min(max(raw, 0), K);
        s_fp[i] = 1; s_fa[i] = 1; s_same[i] = 1;     // every rollout equals itself
    }
    if (tid == 0) s_nbig = 0;
    const int q4 = (K + 3) >> 2;
    for (int e = tid; e < N * 8; e += nthr) {
        const int i = e >> 3, q = e & 7;
        if (q < q4) {
            const int4 v = __ldg(reinterpret_cast<const int4*>(seqs + ((size_t)g * N + i) * stride) + q);
            *reinterpret_cast<int4*>(s_sym + i * kSymPitch + 4 * q) = v;
        }
    }
    if (jac) {                                   // 16-byte stores: both regions are padded to 16 bytes
        uint4* o4 = reinterpret_cast<uint4*>(s_owner);
        for (int e = tid; e < slots / 4; e += nthr) o4[e] = make_uint4(0u, 0u, 0u, 0u);
        uint4* b4 = reinterpret_cast<uint4*>(s_bits);
        for (int e = tid; e < (N * kBgWords + 3) / 4; e += nthr) b4[e] = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    if (jac) {                                   // bigram (a[t], a[t+1]) of rollout i -> slot
        for (int e = tid; e < N * 32; e += nthr) {
            const int i = e >> 5, t = e & 31;
            if (t + 1 >= s_len[i]) continue;
            const int32_t x = s_sym[i * kSymPitch + t], y = s_sym[i * kSymPitch + t + 1];
            uint32_t h = (((uint32_t)x * 0x9E3779B1u) ^ ((uint32_t)y * 0x85EBCA77u)) >> slot_shift;
            for (int probe = 0; probe < slots; ++probe) {         // at most half of the slots fill up
                uint32_t o = s_owner[h];
                if (o == 0u) o = atomicCAS(&s_owner[h], 0u, (uint32_t)e + 1u);
                if (o == 0u) { s_bid[h] = (uint16_t)atomicAdd(&s_nbig, 1); break; }
                const int oi = (int)(o - 1u) >> 5, ot = (int)(o - 1u) & 31;
                if (s_sym[oi * kSymPitch + ot] == x && s_sym[oi * kSymPitch + ot + 1] == y) break;
                h = (h + 1u) & (uint32_t)(slots - 1);
            }
            s_slot[e] = (uint16_t)h;
        }
    }
    // one thread per unordered pair: equal prefixes / equal step-K actions knock out the
    // later rollout as a "first occurrence" and count towards the action's multiplicity
    for (int p = tid; p < P; p += nthr) {
        const int pr = kPairs.v[N][p];
        const int i = pr & 0xFF, j = pr >> 8;
        const int32_t* a = s_sym + i * kSymPitch;
        const int32_t* b = s_sym + j * kSymPitch;
        const int mi = s_len[i];
        bool same_p = mi == s_len[j];
        for (int q = 0; same_p && 4 * q < mi; ++q) {          // four symbols per 16-byte load
            const int4 u = reinterpret_cast<const int4*>(a)[q], v = reinterpret_cast<const int4*>(b)[q];
            const int left = mi - 4 * q;                     // symbols of this quad inside the prefix
            same_p = u.x == v.x && (left < 2 || u.y == v.y) && (left < 3 || u.z == v.z) && (left < 4 || u.w == v.w);
        }
        const bool has_i = s_raw[i] >= K && K >= 1, has_j = s_raw[j] >= K && K >= 1;
        const bool same_a = has_i == has_j && (!has_i || a[K - 1] == b[K - 1]);
        if (same_p) s_fp[j] = 0;
        if (same_a) { s_fa[j] = 0; atomicAdd(&s_same[i], 1); atomicAdd(&s_same[j], 1); }
    }
    __syncthreads();
    if (jac) {                                   // bit sets of bigram ids, one per rollout
        for (int e = tid; e < N * 32; e += nthr) {
            const int i = e >> 5, t = e & 31;
            if (t + 1 >= s_len[i]) continue;
            const uint32_t id = s_bid[s_slot[e]];
            atomicOr(&s_bits[i * kBgWords + (id >> 5)], 1u << (id & 31));
        }
        __syncthreads();
        const int words = (s_nbig + 31) >> 5;
        for (int i = tid; i < N; i += nthr) {
            int c = 0;
            for (int w = 0; w < words; ++w) c += __popc(s_bits[i * kBgWords + w]);
            s_card[i] = c;
        }
        __syncthreads();
        for (int p = tid; p < P; p += nthr) {
            const int pr = kPairs.v[N][p];
            const int i = pr & 0xFF, j = pr >> 8;
            int both = 0;
            for (int w = 0; w < words; ++w) both += __popc(s_bits[i * kBgWords + w] & s_bits[j * kBgWords + w]);
            const int uni = s_card[i] + s_card[j] - both;
            s_term[p] = uni > 0 ? __dsub_rn(1.0, __ddiv_rn((double)both, (double)uni)) : 0.0;
        }
    }
    // entropy terms side by side (the logarithms are the long part); added up in order below
    if (tid < N) {
        const double pr = __ddiv_rn((double)s_same[tid], (double)N);
        s_plogp[tid] = s_fa[tid] ? __dmul_rn(pr, log(pr)) : 0.0;
    }
    __syncthreads();
    if (tid == 0) {
        int dp = 0, da = 0;
        double h = 0.0;
        for (int i = 0; i < N; ++i) {
            dp += s_fp[i];
            da += s_fa[i];
            if (s_fa[i]) h = __dsub_rn(h, s_plogp[i]);
        }
        if (upr) upr[g] = __ddiv_rn((double)dp, (double)N);
        if (uar) uar[g] = __ddiv_rn((double)da, (double)N);
        if (ent) ent[g] = __ddiv_rn(h, ln_n);        // ln N comes from the host: one fp64 logarithm less in this serial tail
        if (jac) {
            double s = 0.0;
            for (int p = 0; p < P; ++p) s = __dadd_rn(s, s_term[p]);
            jac[g] = __ddiv_rn(s, (double)P);
        }
    }
}

// Batch reductions (Section 4.5 dilution, Section 3.4 norm kept): grid-stride over the
// groups, fp64 partial sums per thread, warp shuffles, one set of atomics per CTA.
// N = 8 (the paper's G): four groups per trip, a grid stride apart (so that consecutive
// lanes read consecutive 32-byte rows), their eight 16-byte loads and four decision bytes
// issued before any arithmetic; the last trip takes whatever is left of the four with
// predicated loads.  Measured at 0.59 of the copy bandwidth: the warps wait on loads (17
// stall cycles per issue) while the fp32 -> fp64 conversions of the exact squares keep the
// conversion unit a third busy.  Tried and not faster: four consecutive groups per thread
// (uncoalesced 16-byte loads), eight groups per trip, larger CTAs, more CTAs (the five
// atomics per CTA start to cost from about 5000 CTAs on).
__global__ void __launch_bounds__(256)
batch_stats_kernel(const float* __restrict__ adv, const uint8_t* __restrict__ stop, int N,
                   int n_groups, bool vec4, unsigned long long* counts, double* sumsq) {
    double ss_all = 0.0, ss_kept = 0.0;
    unsigned z_all = 0, z_kept = 0, kept_groups = 0;
    const int stride = gridDim.x * blockDim.x;
    long long g = blockIdx.x * blockDim.x + threadIdx.x;     // 64-bit: g + 4 * stride may pass 2^31
    if (vec4 && N == 8) {
        for (; g < n_groups; g += 4LL * stride) {
            float4 v[4][2];
            unsigned char st[4];
            bool have[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const long long gg = g + (long long)u * stride;
                have[u] = gg < n_groups;
                v[u][0] = v[u][1] = make_float4(1.f, 1.f, 1.f, 1.f);
                st[u] = 0;
                if (have[u]) {
                    const float4* row = reinterpret_cast<const float4*>(adv + (size_t)gg * 8);
                    v[u][0] = __ldg(row);
                    v[u][1] = __ldg(row + 1);
                    st[u] = stop ? stop[gg] : 0;
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (!have[u]) continue;
                const float f[8] = {v[u][0].x, v[u][0].y, v[u][0].z, v[u][0].w,
                                    v[u][1].x, v[u][1].y, v[u][1].z, v[u][1].w};
                double ss = 0.0;
                unsigned z = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) {        // zero tests in fp32 (exact), squares in fp64
                    const double a = (double)f[i];
                    ss += __dmul_rn(a, a);
                    z += f[i] == 0.0f;
                }
                const bool kept = st[u] == 0;
                kept_groups += kept;
                ss_all += ss;
                z_all += z;
                if (kept) { ss_kept += ss; z_kept += z; }
            }
        }
    }
    for (; g < n_groups; g += stride) {            // any other group size: one group per trip
        const bool kept = !(stop && stop[g]);
        kept_groups += kept;
        const float* row = adv + (size_t)g * N;
        double ss = 0.0;
        unsigned z = 0;
        if (vec4) {
            for (int q = 0; q < N / 4; ++q) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(row) + q);
                const double a0 = v.x, a1 = v.y, a2 = v.z, a3 = v.w;
                ss += __dmul_rn(a0, a0); ss += __dmul_rn(a1, a1); ss += __dmul_rn(a2, a2); ss += __dmul_rn(a3, a3);
                z += (a0 == 0.0) + (a1 == 0.0) + (a2 == 0.0) + (a3 == 0.0);
            }
        } else {
            for (int i = 0; i < N; ++i) {
                const double a = (double)__ldg(row + i);
                ss += __dmul_rn(a, a);
                z += a == 0.0;
            }
        }
        ss_all += ss;
        z_all += z;
        if (kept) { ss_kept += ss; z_kept += z; }
    }
    for (int off = 16; off > 0; off >>= 1) {
        ss_all += __shfl_xor_sync(0xFFFFFFFFu, ss_all, off);
        ss_kept += __shfl_xor_sync(0xFFFFFFFFu, ss_kept, off);
        z_all += __shfl_xor_sync(0xFFFFFFFFu, z_all, off);
        z_kept += __shfl_xor_sync(0xFFFFFFFFu, z_kept, off);
        kept_groups += __shfl_xor_sync(0xFFFFFFFFu, kept_groups, off);
    }
    // warp results -> shared memory -> one set of atomics per CTA
    __shared__ double s_ss[2][8];
    __shared__ unsigned s_cnt[3][8];
    const int w = threadIdx.x >> 5;
    if ((threadIdx.x & 31) == 0) {
        s_ss[0][w] = ss_all; s_ss[1][w] = ss_kept;
        s_cnt[0][w] = z_all; s_cnt[1][w] = z_kept; s_cnt[2][w] = kept_groups;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        double a = 0.0, k = 0.0;
        unsigned long long c0 = 0, c1 = 0, c2 = 0;
        for (int i = 0; i < 8; ++i) {
            a += s_ss[0][i]; k += s_ss[1][i];
            c0 += s_cnt[0][i]; c1 += s_cnt[1][i]; c2 += s_cnt[2][i];
        }
        atomicAdd(&sumsq[0], a);
        atomicAdd(&sumsq[1], k);
        atomicAdd(&counts[0], c0);
        atomicAdd(&counts[1], c1);
        atomicAdd(&counts[2], c2);
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
    int slots = 64;                                  // >= 2 * N * (K - 1) bigrams: at most 2048
    while (slots < 2 * N * (K > 1 ? K - 1 : 1)) slots <<= 1;
    int slot_shift = 32;
    while ((1 << (32 - slot_shift)) < slots) --slot_shift;
    SignalLayout L;
    int off = 0;
    auto take = [&](int bytes) { int o = off; off = (off + bytes + 15) & ~15; return o; };
    L.off_term = take(pairs_of(N) * 8);
    L.off_plogp = take(N * 8);
    L.off_sym = take(N * kSymPitch * 4);
    L.off_owner = take(slots * 4);
    L.off_bits = take(N * kBgWords * 4);
    L.off_small = take((6 * N + 1) * 4);
    L.off_bid = take(slots * 2);
    L.off_slot = take(N * 32 * 2);
    L.words = kBgWords;
    L.total = off;
    group_signals_kernel<<<n_groups, threads, L.total, s>>>(seqs, lens, N, stride, K, slots, slot_shift,
                                                            log((double)N), L, upr, uar, ent, jac);
    SR_LAUNCH_CHECK("group_signals_kernel");
    return SR_OK;
}

int launch_batch_stats(const float* adv, const uint8_t* stop, int32_t n_groups, int32_t N,
                       int64_t* counts, double* sumsq, cudaStream_t s) {
    SR_CUDA_TRY(cudaMemsetAsync(counts, 0, 3 * sizeof(int64_t), s));
    SR_CUDA_TRY(cudaMemsetAsync(sumsq, 0, 2 * sizeof(double), s));
    if (n_groups == 0) return SR_OK;
    int dev = 0, sms = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    SR_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const bool vec4 = (N % 4 == 0) && (reinterpret_cast<uintptr_t>(adv) & 15) == 0;
    const int want = (n_groups + 255) / 256;
    const int cap = sms * 16;
    const int blocks = want < cap ? want : cap;
    batch_stats_kernel<<<blocks, 256, 0, s>>>(adv, stop, N, n_groups, vec4,
                                              reinterpret_cast<unsigned long long*>(counts), sumsq);
    SR_LAUNCH_CHECK("batch_stats_kernel");
    return SR_OK;
}

int launch_or_rule(const double* mean, const int32_t* lens, const uint8_t* done, int32_t n_groups,
                   int32_t N, int32_t K, double threshold, double tau_high, double* tau,
                   uint8_t* stop, cudaStream_t s) {
    if (n_groups == 0) return SR_OK;
    const bool vec4 = done == nullptr && (N % 4 == 0) && (reinterpret_cast<uintptr_t>(lens) & 15) == 0;
    or_rule_kernel<<<(n_groups + 255) / 256, 256, 0, s>>>(mean, lens, done, n_groups, N, K, threshold,
                                                          tau_high, vec4, tau, stop);
    SR_LAUNCH_CHECK("or_rule_kernel");
    return SR_OK;
}

}  // namespace sr
