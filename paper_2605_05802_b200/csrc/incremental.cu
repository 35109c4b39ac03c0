// Incremental gate: one new action per rollout per environment step, gate
// re-evaluated after every step (the paper gates at one fixed K, Appendix C.1; a
// per-step evaluation is what its "adaptive K" follow-up needs, Section 5).
//
// Per pair (i, j), i < j, with current lengths m = len_i (rows) and n = len_j
// (columns) of the edit-distance matrix D, the state keeps
//   VP / VN : bit r-1 set iff D[r][n] - D[r-1][n] is +1 / -1   (last column)
//   HP / HN : bit c-1 set iff D[m][c] - D[m][c-1] is +1 / -1   (last row)
// and D[m][n] = n + popc(VP) - popc(VN) is never stored.  When j appends y, one
// bit-parallel column step over the rows gives the new last column and the
// horizontal delta of the bottom row; when i appends x, the same step on the
// transposed roles gives the new last row; when both append, both steps start from
// the OLD state and the new corner D[m+1][n+1] is the usual three-way minimum.
//
// State buffer layout (position independent, byte-copyable):
//   [0, 256)        header: magic, n_groups, N, max_steps, steps taken so far (an upper
//                   bound of every rollout's length, known without reading the lengths)
//   lens   int32 [n_groups][N]
//   hist   int32 [n_groups][8][N][4]      actions emitted so far: action r of rollout i
//                                         sits at [r / 4][i][r % 4], so that the first
//                                         quads of all rollouts of a group (what a step
//                                         reads) are contiguous
//   pairs  uint4 [n_groups][P]            (VP, VN, HP, HN)
// every section starts on a 256-byte boundary.
#include "common.cuh"

namespace sr {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

namespace {

constexpr uint32_t kMagic = 0x53524731u;   // "SRG1"
constexpr int kHistPitch = 32;

struct IncrLayout {
    size_t off_lens, off_hist, off_pairs, total;
};

IncrLayout incr_layout(int32_t n_groups, int32_t N) {
    IncrLayout L;
    size_t off = 256;
    L.off_lens = off;
    off = align_up(off + (size_t)n_groups * N * 4, 256);
    L.off_hist = off;
    off = align_up(off + (size_t)n_groups * N * kHistPitch * 4, 256);
    L.off_pairs = off;
    off = align_up(off + (size_t)n_groups * pairs_of(N) * 16, 256);
    L.total = off;
    return L;
}

__global__ void incr_init_kernel(unsigned char* state, IncrLayout L, int n_groups, int N,
                                 int max_steps) {
    const size_t tid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t nthr = (size_t)gridDim.x * blockDim.x;
    uint32_t* hdr = reinterpret_cast<uint32_t*>(state);
    if (tid < 64) {
        uint32_t v = 0;
        if (tid == 0) v = kMagic;
        if (tid == 1) v = (uint32_t)n_groups;
        if (tid == 2) v = (uint32_t)N;
        if (tid == 3) v = (uint32_t)max_steps;
        hdr[tid] = v;
    }
    // lengths and pair state start at zero; the history needs no clearing (only the
    // first len entries of a row are ever read)
    uint32_t* lens = reinterpret_cast<uint32_t*>(state + L.off_lens);
    for (size_t e = tid; e < (size_t)n_groups * N; e += nthr) lens[e] = 0u;
    uint4* pairs = reinterpret_cast<uint4*>(state + L.off_pairs);
    for (size_t e = tid; e < (size_t)n_groups * pairs_of(N); e += nthr)
        pairs[e] = make_uint4(0u, 0u, 0u, 0u);
}

// One bit-parallel column step over `m` rows (m >= 1) with horizontal input +1 at
// row 0; returns the horizontal delta leaving the bottom row.  Bits of Eq at or above m
// are harmless: carries and shifts only move upwards, and the result is masked.
__device__ __forceinline__ int column_step(uint32_t Eq, uint32_t& Pv, uint32_t& Mv, int m) {
    uint32_t Ph, Mh;
    word_column(Eq, Pv, Mv, Ph, Mh);
    const int hout = (int)((Ph >> (m - 1)) & 1u) - (int)((Mh >> (m - 1)) & 1u);
    const uint32_t msk = low_mask(m);
    Pv &= msk;
    Mv &= msk;
    return hout;
}

struct IncrArgs {
    unsigned char* state;
    IncrLayout L;
    const int32_t* new_actions;
    int n_groups, N;
    double threshold;
    int norm_mode;
    int32_t* pair_dist;
    int32_t* pair_sum;
    double* mean;
    uint8_t* stop;
    int32_t* status;
    int gpb;                                               // groups per CTA
    uint32_t inv_P, inv_N;                                 // ceil(2^20 / P), ceil(2^20 / N): thread -> group by multiply-shift (exact below 512)
    int off_dist, off_term;                                // shared-memory offsets
    uint32_t one;                                          // 1, as a run-time value
};

// Match masks of a pair's two new actions against the stored actions of the other
// rollout: bit r of eq_y set iff action r of rollout ri equals y, bit c of eq_x set iff
// action c of rollout rj equals x, over the first 4 * kQuads positions.  Positions at or
// past a rollout's length hold whatever the buffer holds; the caller's column step
// ignores those bits (carries and shifts only move upwards, the result is masked).
// `quads` points at the group's stored actions ([8][N] int4): one 16-byte load and four
// compare / set-bit pairs per quad, both rows' loads issued before the comparisons.
template <int kQuads>
__device__ __forceinline__ void match_masks(const int4* quads, int N, int ri, int rj, int32_t y,
                                            int32_t x, uint32_t one, uint32_t& eq_y, uint32_t& eq_x) {
    int4 vi[kQuads], vj[kQuads];
#pragma unroll
    for (int q = 0; q < kQuads; ++q) { vi[q] = quads[q * N + ri]; vj[q] = quads[q * N + rj]; }
    eq_y = 0u;
    eq_x = 0u;
#pragma unroll
    for (int q = 0; q < kQuads; ++q) {
        // `one` holds 1 but is a run-time value: the bits are set by multiply-adds, which
        // issue on the FMA pipe while the comparisons keep the integer ALU busy
        asm("{ .reg .pred e0, e1, e2, e3;\n\t"
            "setp.eq.s32 e0, %1, %5; setp.eq.s32 e1, %2, %5; setp.eq.s32 e2, %3, %5; setp.eq.s32 e3, %4, %5;\n\t"
            "@e0 mad.lo.u32 %0, %10, %6, %0; @e1 mad.lo.u32 %0, %10, %7, %0;\n\t"
            "@e2 mad.lo.u32 %0, %10, %8, %0; @e3 mad.lo.u32 %0, %10, %9, %0; }"
            : "+r"(eq_y)
            : "r"(vi[q].x), "r"(vi[q].y), "r"(vi[q].z), "r"(vi[q].w), "r"(y),
              "r"(1u << (4 * q)), "r"(2u << (4 * q)), "r"(4u << (4 * q)), "r"(8u << (4 * q)), "r"(one));
        asm("{ .reg .pred e0, e1, e2, e3;\n\t"
            "setp.eq.s32 e0, %1, %5; setp.eq.s32 e1, %2, %5; setp.eq.s32 e2, %3, %5; setp.eq.s32 e3, %4, %5;\n\t"
            "@e0 mad.lo.u32 %0, %10, %6, %0; @e1 mad.lo.u32 %0, %10, %7, %0;\n\t"
            "@e2 mad.lo.u32 %0, %10, %8, %0; @e3 mad.lo.u32 %0, %10, %9, %0; }"
            : "+r"(eq_x)
            : "r"(vj[q].x), "r"(vj[q].y), "r"(vj[q].z), "r"(vj[q].w), "r"(x),
              "r"(1u << (4 * q)), "r"(2u << (4 * q)), "r"(4u << (4 * q)), "r"(8u << (4 * q)), "r"(one));
    }
}

// One thread per pair, `gpb` groups per CTA.  The header (hot in L2: every CTA reads it)
// says how many steps the state has taken, which bounds every length; with that, all a
// pair needs -- its state, the two lengths, the two new actions AND the stored actions of
// both rollouts -- is requested in ONE round of independent loads instead of waiting for
// the lengths first (a second trip to DRAM per step made the kernel latency-bound).  The
// stored actions are read straight from the state: the pairs of a group share N rows, so
// all but the first touch of a row hit L1 (staging them in shared memory with asynchronous
// copies was measured slower).  The CTA synchronises twice, before the appends and before
// the per-group sums.
// kN: the group size when it is known at compile time (8, the paper's G: row offsets and
// the pair count fold into immediates), 0 for any other size.
template <int kN>
__global__ void __launch_bounds__(512, 3)
incr_step_kernel(IncrArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = kN ? kN : a.N, P = pairs_of(N);
    const int tid = threadIdx.x;
    const int g0 = blockIdx.x * a.gpb;
    const int ng = min(a.gpb, a.n_groups - g0);
    int32_t* s_dist = reinterpret_cast<int32_t*>(smem + a.off_dist);    // [gpb][P]
    double* s_term = reinterpret_cast<double*>(smem + a.off_term);      // [gpb][P]

    const uint4 hdr = *reinterpret_cast<const uint4*>(a.state);         // magic, n_groups, N, max_steps
    const uint32_t steps_taken = reinterpret_cast<const uint32_t*>(a.state)[4];
    int32_t* g_len = reinterpret_cast<int32_t*>(a.state + a.L.off_lens) + (size_t)g0 * N;
    int32_t* g_hist = reinterpret_cast<int32_t*>(a.state + a.L.off_hist) + (size_t)g0 * N * kHistPitch;
    uint4* g_pairs = reinterpret_cast<uint4*>(a.state + a.L.off_pairs) + (size_t)g0 * P;
    const int32_t* g_new = a.new_actions + (size_t)g0 * N;

    const bool bad = hdr.x != kMagic || hdr.y != (uint32_t)a.n_groups || hdr.z != (uint32_t)N;
    if (bad) {                                     // uniform over the grid: nothing is touched
        if (tid == 0 && a.status) atomicOr(a.status, SR_STATUS_BAD_STATE);
        return;
    }
    const int max_steps = (int)hdr.w;
    // quads of stored actions any rollout can hold by now (the same for the whole grid, or
    // one more where a CTA already sees this step's own count: either is an upper bound)
    const int nq = (min((uint32_t)max_steps, steps_taken) + 3u) >> 2;

    if (blockIdx.x == 0 && tid == 0 && steps_taken < 0x7FFFFFFFu)
        reinterpret_cast<uint32_t*>(a.state)[4] = steps_taken + 1u;
    const bool is_pair = tid < ng * P;
    uint4 st = make_uint4(0u, 0u, 0u, 0u);
    int ri = 0, rj = 0, m = 0, n = 0, grp = 0;
    int32_t x = SR_NO_ACTION, y = SR_NO_ACTION;
    if (is_pair) {
        grp = (int)(((uint32_t)tid * a.inv_P) >> 20);
        const int pr = kPairs.v[N][tid - grp * P];
        ri = pr & 0xFF;
        rj = pr >> 8;
        st = g_pairs[tid];
        const int gi = grp * N + ri, gj = grp * N + rj;
        m = g_len[gi];
        n = g_len[gj];
        x = __ldg(g_new + gi);
        y = __ldg(g_new + gj);
    }
    uint32_t eq_y = 0u, eq_x = 0u;                 // match masks of y in rollout ri, of x in rollout rj
    if (is_pair) {
        const int4* quads = reinterpret_cast<const int4*>(g_hist) + (size_t)grp * 8 * N;
        switch (nq) {
            case 0: break;
            case 1: match_masks<1>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 2: match_masks<2>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 3: match_masks<3>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 4: match_masks<4>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 5: match_masks<5>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 6: match_masks<6>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            case 7: match_masks<7>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
            default: match_masks<8>(quads, N, ri, rj, y, x, a.one, eq_y, eq_x); break;
        }
    }
    // appenders: thread e < ng*N owns rollout e of this CTA
    const bool is_roll = tid < ng * N;
    int my_len = 0;
    int32_t my_act = SR_NO_ACTION;
    if (is_roll) { my_len = g_len[tid]; my_act = __ldg(g_new + tid); }
    if (m >= max_steps) x = SR_NO_ACTION;          // rollout already full: the action is ignored
    if (n >= max_steps) y = SR_NO_ACTION;
    if (is_roll && my_act != SR_NO_ACTION && my_len >= max_steps) {
        my_act = SR_NO_ACTION;
        if (a.status) atomicOr(a.status, SR_STATUS_STEP_OVERFLOW);
    }

    const bool ai = x != SR_NO_ACTION, aj = y != SR_NO_ACTION;
    int hout = 1, vout = 1;
    uint32_t VP2 = st.x, VN2 = st.y, HP2 = st.z, HN2 = st.w;
    if (is_pair) {
        if (aj && m > 0) hout = column_step(eq_y, VP2, VN2, m);
        if (ai && n > 0) vout = column_step(eq_x, HP2, HN2, n);
    }
    __syncthreads();       // every thread has read the lengths (and the stored actions) before the appends
    if (is_roll && my_act != SR_NO_ACTION) {
        const int g = (int)(((uint32_t)tid * a.inv_N) >> 20), i = tid - g * N;
        g_hist[(((size_t)g * 8 + (my_len >> 2)) * N + i) * 4 + (my_len & 3)] = my_act;
        g_len[tid] = my_len + 1;
    }
    if (is_pair) {
        uint32_t VP = st.x, VN = st.y, HP = st.z, HN = st.w;
        const int c = n + __popc(VP) - __popc(VN);
        int d = c, mi = m, mj = n;
        if (ai && aj) {
            const int left = c + vout, up = c + hout;
            d = min(min(c + (x != y ? 1 : 0), up + 1), left + 1);
            const int vd = d - up, hd = d - left;
            VP = VP2 | (vd > 0 ? 1u << m : 0u);
            VN = VN2 | (vd < 0 ? 1u << m : 0u);
            HP = HP2 | (hd > 0 ? 1u << n : 0u);
            HN = HN2 | (hd < 0 ? 1u << n : 0u);
            mi = m + 1; mj = n + 1;
        } else if (aj) {
            d = c + hout;
            VP = VP2; VN = VN2;
            HP |= hout > 0 ? 1u << n : 0u;
            HN |= hout < 0 ? 1u << n : 0u;
            mj = n + 1;
        } else if (ai) {
            d = c + vout;
            HP = HP2; HN = HN2;
            VP |= vout > 0 ? 1u << m : 0u;
            VN |= vout < 0 ? 1u << m : 0u;
            mi = m + 1;
        }
        if (ai || aj) g_pairs[tid] = make_uint4(VP, VN, HP, HN);
        s_dist[tid] = d;
        s_term[tid] = a.norm_mode == SR_NORM_NONE ? (double)d : kQuot.v[d * 33 + max(mi, mj)];
        if (a.pair_dist) a.pair_dist[(size_t)g0 * P + tid] = d;
    }
    __syncthreads();
    if (tid < ng) {
        GateArgs out{};
        out.pair_sum = a.pair_sum; out.mean = a.mean; out.stop = a.stop; out.threshold = a.threshold;
        group_sum_and_gate(s_term + tid * P, s_dist + tid * P, P, out, (size_t)g0 + tid);
    }
}

}  // namespace

size_t incr_state_bytes(int32_t n_groups, int32_t N, int32_t max_steps) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N || max_steps < 1 || max_steps > SR_MAX_INCR_STEPS)
        return 0;
    return incr_layout(n_groups, N).total;
}

int launch_incr_init(void* state, size_t bytes, int32_t n_groups, int32_t N, int32_t max_steps,
                     cudaStream_t s) {
    const IncrLayout L = incr_layout(n_groups, N);
    if (bytes < L.total) return SR_ERR_STATE_SIZE;
    size_t work = (size_t)n_groups * pairs_of(N);
    int blocks = (int)((work + 255) / 256);
    if (blocks < 1) blocks = 1;
    if (blocks > 4096) blocks = 4096;
    incr_init_kernel<<<blocks, 256, 0, s>>>(static_cast<unsigned char*>(state), L, n_groups, N, max_steps);
    SR_LAUNCH_CHECK("incr_init_kernel");
    return SR_OK;
}

int launch_incr_step(void* state, size_t bytes, const int32_t* new_actions, int32_t n_groups,
                     int32_t N, double threshold, int32_t norm_mode, int32_t* pair_dist,
                     int32_t* pair_sum, double* mean, uint8_t* stop, int32_t* status,
                     cudaStream_t s) {
    IncrArgs a;
    a.L = incr_layout(n_groups, N);
    if (bytes < a.L.total) return SR_ERR_STATE_SIZE;
    if (n_groups == 0) return SR_OK;
    a.state = static_cast<unsigned char*>(state);
    a.new_actions = new_actions;
    a.n_groups = n_groups; a.N = N;
    a.threshold = threshold; a.norm_mode = norm_mode;
    a.pair_dist = pair_dist; a.pair_sum = pair_sum; a.mean = mean; a.stop = stop; a.status = status;
    const int P = pairs_of(N);
    int gpb = 256 / P;
    if (gpb < 1) gpb = 1;
    if (gpb > 32) gpb = 32;
    while (gpb > 1 && gpb * N > 256) --gpb;      // one appending thread per rollout
    a.gpb = gpb;
    a.one = 1u;
    a.inv_P = ((1u << 20) + (uint32_t)P - 1u) / (uint32_t)P;
    a.inv_N = ((1u << 20) + (uint32_t)N - 1u) / (uint32_t)N;
    int off = 0;
    auto take = [&](int b) { int o = off; off = (off + b + 15) & ~15; return o; };
    a.off_dist = take(gpb * P * 4);
    a.off_term = take(gpb * P * 8);
    int threads = (gpb * P + 31) & ~31;
    if (threads < gpb * N) threads = (gpb * N + 31) & ~31;
    if (threads < 64) threads = 64;
    const int blocks = (n_groups + gpb - 1) / gpb;
    if (N == 8) incr_step_kernel<8><<<blocks, threads, off, s>>>(a);
    else incr_step_kernel<0><<<blocks, threads, off, s>>>(a);
    SR_LAUNCH_CHECK("incr_step_kernel");
    return SR_OK;
}

}  // namespace sr
