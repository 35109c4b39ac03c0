// Single-word gate kernels: prefixes of at most 32 symbols (action-level gate,
// Section 3.2 of the paper: d_K at K <= T_max = 30).  One thread per pair runs the
// bit-parallel column recurrence on one 32-bit word of +1 / -1 vertical deltas; the
// distance is read off as n + popc(Pv) - popc(Mv), so no per-column score is kept.  The
// two kernels differ in where a column's match word comes from.
//
// K <= 16 (the paper's K = 10 and 15): gate_direct_kernel.  A thread keeps both prefixes
// of its pair in registers (int4 loads; the rows of a group are shared by its pairs, so
// all but the first touch hit L1) and builds the match word of a column by comparing the
// text symbol with every pattern symbol: 2 instructions per cell against the ~14 of a
// column, no tables, no atomics, no shared memory before the final sums -- at these
// lengths cheaper than naming the symbols first, and free of the latencies that kept the
// table kernel from filling the issue slots.
//
// K = 17..32: gate_single_kernel.  A group is handled by one warp (N <= 8) or one CTA:
//   1. every thread fetches one or two quads of symbols (int4 loads) and keeps them in
//      registers; each symbol claims a slot of the group's open-addressing table in
//      shared memory (64-bit slots {symbol, claimed}; all 2^32 IDs are legal) -- the slot
//      index is the symbol's name within the group from here on -- and notes, in a byte
//      map indexed by (rollout, slot), one position at which the rollout holds it;
//   2. the positions of a rollout holding the same symbol OR their bits into the match
//      mask peq[rollout][noted position];
//   3. the pair threads take a column's match word from
//      peq[pattern][map[pattern][slot of the text symbol]] (33rd mask = 0: absent);
//   4. one thread per group adds the normalised terms in fp64 in pair order, thresholds
//      (Eq. 2) and writes out, for all groups of a CTA side by side.
// Three synchronisations per group before that (warp-level for N <= 8).  All index
// arithmetic is shifts and adds.
#include "common.cuh"

namespace sr {
namespace {

constexpr int kTxtPitch = 36;          // 16-bit slot names per rollout: 32 + pad, rows 8-byte aligned
constexpr int kPeqPitch = 33;          // 32 masks by position + one all-zero mask for "absent"
constexpr uint32_t kAbsentOff = 32 * 4;   // map entries are BYTE offsets into a peq row
constexpr int kMaxItems = 2;           // quads of symbols a thread may own

struct SingleLayout {
    int hslots, hshift, hlog;          // slots of the group table (power of two), 32 - log2, log2
    int qshift;                        // log2 of the quads per rollout that are fetched (K <= 4 << qshift)
    int n_items;                       // N << qshift
    // byte offsets within a group's shared memory: the table and the masks (cleared to 0
    // together), the map (cleared to "absent"), slot names of the symbols, lengths
    int off_hash, off_peq, off_map, off_txt, off_len;
    int zero_words16, map_words16;     // sizes of the two clears in 16-byte units
    int group_bytes;
    int off_term, off_dist;            // per CTA, after the groups: [groups per CTA][P]
};

__device__ __forceinline__ void group_sync(bool warp_level) {
    if (warp_level) __syncwarp(); else __syncthreads();
}

// kWarp: one warp per group, blockDim.x / 32 groups per CTA; otherwise one group per CTA.
template <bool kWarp>
__global__ void __launch_bounds__(kWarp ? 256 : 512)
gate_single_kernel(GateArgs a, SingleLayout L) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = a.N, K = a.K, P = pairs_of(N);
    const int t = kWarp ? (threadIdx.x & 31) : threadIdx.x;               // thread within the group
    const int nthr = kWarp ? 32 : blockDim.x;
    const int gl = kWarp ? (threadIdx.x >> 5) : 0;                        // group within the CTA
    const int g = kWarp ? blockIdx.x * (blockDim.x >> 5) + gl : blockIdx.x;
    const bool live = g < a.n_groups;              // a warp without a group only keeps the barrier company
    unsigned char* base = smem + (size_t)gl * L.group_bytes;
    unsigned long long* s_hash = reinterpret_cast<unsigned long long*>(base + L.off_hash);  // [hslots]
    unsigned char* s_peq = base + L.off_peq;                                                // [N][33] words
    unsigned char* s_map = base + L.off_map;                                                // [N][hslots]
    uint16_t* s_txt = reinterpret_cast<uint16_t*>(base + L.off_txt);                        // [N][36]
    int32_t* s_len = reinterpret_cast<int32_t*>(base + L.off_len);                          // [N]
    double* s_term = reinterpret_cast<double*>(smem + L.off_term) + gl * P;                 // [P]
    int32_t* s_dist = reinterpret_cast<int32_t*>(smem + L.off_dist) + gl * P;               // [P]

    if (live) {
        // ---- symbols first (the longest latency), then the clears
        const int qmask = (1 << L.qshift) - 1;
        int4 sym[kMaxItems];
        int row_len[kMaxItems];
#pragma unroll
        for (int u = 0; u < kMaxItems; ++u) {
            const int item = t + u * nthr;
            sym[u] = make_int4(0, 0, 0, 0);
            row_len[u] = 0;
            if (item < L.n_items) {
                const int i = item >> L.qshift, q = item & qmask;
                const size_t row = (size_t)g * N + i;
                int len = a.lens ? __ldg(a.lens + row) : K;
                if (q == 0) {
                    if (len < 0 && a.status) atomicOr(a.status, SR_STATUS_NEG_LEN);
                    s_len[i] = min(max(len, 0), K);
                }
                len = min(max(len, 0), K);
                row_len[u] = len;
                if (4 * q < len) sym[u] = __ldg(reinterpret_cast<const int4*>(a.seqs + row * a.stride) + q);
            }
        }
        {
            uint4* z4 = reinterpret_cast<uint4*>(s_hash);
#pragma unroll 4
            for (int e = t; e < L.zero_words16; e += nthr) z4[e] = make_uint4(0u, 0u, 0u, 0u);
            uint4* m4 = reinterpret_cast<uint4*>(s_map);
            const uint32_t absent4 = kAbsentOff * 0x01010101u;
#pragma unroll 4
            for (int e = t; e < L.map_words16; e += nthr) m4[e] = make_uint4(absent4, absent4, absent4, absent4);
        }
        group_sync(kWarp);

        // ---- every symbol claims (or finds) its slot; the slot index names the symbol
        uint32_t slot[kMaxItems][4];
#pragma unroll
        for (int u = 0; u < kMaxItems; ++u) {
            const int item = t + u * nthr;
            const int i = item >> L.qshift, q = item & qmask;
            const int32_t s4[4] = {sym[u].x, sym[u].y, sym[u].z, sym[u].w};
            volatile unsigned char* map_i = s_map + ((size_t)i << L.hlog);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = 4 * q + k;
                slot[u][k] = 0u;
                if (r < row_len[u]) {
                    const int32_t s = s4[k];
                    uint32_t h = ((uint32_t)s * 0x9E3779B1u) >> L.hshift;
                    const unsigned long long mine = ((unsigned long long)(uint32_t)s << 32) | 1ull;
                    // at most half of the slots ever fill up, so a free or matching slot is
                    // always found; the trip count is bounded all the same
                    for (int probe = 0; probe < L.hslots; ++probe) {
                        unsigned long long v = s_hash[h];
                        if ((uint32_t)v == 0u) v = atomicCAS(&s_hash[h], 0ull, mine);
                        if ((uint32_t)v == 0u || (int32_t)(v >> 32) == s) break;
                        h = (h + 1u) & (uint32_t)(L.hslots - 1);
                    }
                    slot[u][k] = h;
                    // several positions of a rollout with the same symbol store to the same
                    // byte; whichever store lands last names the representative: any will do
                    map_i[h] = (unsigned char)(4 * r);
                }
            }
            if (4 * q < row_len[u])
                *reinterpret_cast<uint2*>(s_txt + i * kTxtPitch + 4 * q) =
                    make_uint2(slot[u][0] | (slot[u][1] << 16), slot[u][2] | (slot[u][3] << 16));
        }
        group_sync(kWarp);

        // ---- match masks: peq[i][representative position] collects the positions of the symbol
#pragma unroll
        for (int u = 0; u < kMaxItems; ++u) {
            const int item = t + u * nthr;
            const int i = item >> L.qshift, q = item & qmask;
            const unsigned char* map_i = s_map + ((size_t)i << L.hlog);
            unsigned char* peq_i = s_peq + i * (kPeqPitch * 4);
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int r = 4 * q + k;
                if (r < row_len[u])
                    atomicOr(reinterpret_cast<uint32_t*>(peq_i + map_i[slot[u][k]]), 1u << r);
            }
        }
        group_sync(kWarp);

        // ---- one thread per pair; the pattern (rows) is the longer prefix
        for (int p = t; p < P; p += nthr) {
            const int pr = kPairs.v[N][p];
            int pi = pr & 0xFF, pj = pr >> 8;
            const int mi = s_len[pi], mj = s_len[pj];
            int mp = mi, mt = mj;
            if (mj > mi) { const int x = pi; pi = pj; pj = x; mp = mj; mt = mi; }
            const unsigned char* map = s_map + ((size_t)pi << L.hlog);
            const unsigned char* peq = s_peq + pi * (kPeqPitch * 4);
            const uint16_t* txt = s_txt + pj * kTxtPitch;
            uint32_t Pv = 0xFFFFFFFFu, Mv = 0u, Ph, Mh;
            int c = 0;
            for (; c + 4 <= mt; c += 4) {          // four columns per trip: their look-ups overlap
                const uint2 w = *reinterpret_cast<const uint2*>(txt + c);
                const uint32_t e0 = *reinterpret_cast<const uint32_t*>(peq + map[w.x & 0xFFFFu]);
                const uint32_t e1 = *reinterpret_cast<const uint32_t*>(peq + map[w.x >> 16]);
                const uint32_t e2 = *reinterpret_cast<const uint32_t*>(peq + map[w.y & 0xFFFFu]);
                const uint32_t e3 = *reinterpret_cast<const uint32_t*>(peq + map[w.y >> 16]);
                word_column(e0, Pv, Mv, Ph, Mh);
                word_column(e1, Pv, Mv, Ph, Mh);
                word_column(e2, Pv, Mv, Ph, Mh);
                word_column(e3, Pv, Mv, Ph, Mh);
            }
            for (; c < mt; ++c)
                word_column(*reinterpret_cast<const uint32_t*>(peq + map[txt[c]]), Pv, Mv, Ph, Mh);
            const uint32_t msk = low_mask(mp);
            const int d = mt + __popc(Pv & msk) - __popc(Mv & msk);
            s_dist[p] = d;
            // one term of d_K (Section 3.2): distance / longer prefix, from the quotient table
            s_term[p] = a.norm_mode == SR_NORM_NONE ? (double)d : kQuot.v[d * 33 + mp];
            if (a.pair_dist) a.pair_dist[(size_t)g * P + p] = d;
        }
    }
    __syncthreads();

    // ---- d_K: ordered fp64 sum, strict threshold (Eq. 2): one thread per group of the CTA
    const int groups_here = kWarp ? (blockDim.x >> 5) : 1;
    if ((int)threadIdx.x < groups_here) {
        const size_t gg = kWarp ? (size_t)blockIdx.x * groups_here + threadIdx.x : (size_t)blockIdx.x;
        if (gg < (size_t)a.n_groups)
            group_sum_and_gate(reinterpret_cast<const double*>(smem + L.off_term) + threadIdx.x * P,
                               reinterpret_cast<const int32_t*>(smem + L.off_dist) + threadIdx.x * P, P, a, gg);
    }
}


// ---------------------------------------------------------------------------------
// K <= 16: prefixes in registers, match words by direct comparison.  Threads are packed
// pair after pair: a CTA of T threads serves floor(T / P) groups.
template <int KR>      // pattern rows / text columns held in registers: K <= KR, KR % 4 == 0
__global__ void __launch_bounds__(512)
gate_direct_kernel(GateArgs a, int groups_per_cta, uint32_t one) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = a.N, K = a.K, P = pairs_of(N);
    double* s_term = reinterpret_cast<double*>(smem);                               // [groups_per_cta * P]
    int32_t* s_dist = reinterpret_cast<int32_t*>(s_term + groups_per_cta * P);      // [groups_per_cta * P]
    const int tid = threadIdx.x;
    const int gl = tid / P, p = tid - gl * P;
    const size_t g = (size_t)blockIdx.x * groups_per_cta + gl;
    if (gl < groups_per_cta && g < (size_t)a.n_groups) {
        const int pr = kPairs.v[N][p];
        int pi = pr & 0xFF, pj = pr >> 8;
        int mi = a.lens ? __ldg(a.lens + g * N + pi) : K;
        int mj = a.lens ? __ldg(a.lens + g * N + pj) : K;
        if ((mi < 0 || mj < 0) && a.status) atomicOr(a.status, SR_STATUS_NEG_LEN);
        mi = min(max(mi, 0), K);
        mj = min(max(mj, 0), K);
        int mp = mi, mt = mj;                      // the pattern (rows) is the longer prefix
        if (mj > mi) { const int x = pi; pi = pj; pj = x; mp = mj; mt = mi; }
        const int4* prow = reinterpret_cast<const int4*>(a.seqs + (g * N + pi) * a.stride);
        const int4* trow = reinterpret_cast<const int4*>(a.seqs + (g * N + pj) * a.stride);
        int32_t pat[KR], txt[KR];
#pragma unroll
        for (int q = 0; q < KR / 4; ++q) {
            // whole quads inside the row (stride is a multiple of 4 and >= K); symbols past
            // a prefix's end are never looked at: columns stop at mt, and rows past mp only
            // disturb bits the final mask drops (carries and shifts move upwards only)
            int4 v = make_int4(0, 0, 0, 0), w = make_int4(0, 0, 0, 0);
            if (4 * q < mp) v = __ldg(prow + q);
            if (4 * q < mt) w = __ldg(trow + q);
            pat[4 * q] = v.x; pat[4 * q + 1] = v.y; pat[4 * q + 2] = v.z; pat[4 * q + 3] = v.w;
            txt[4 * q] = w.x; txt[4 * q + 1] = w.y; txt[4 * q + 2] = w.z; txt[4 * q + 3] = w.w;
        }
        uint32_t Pv = 0xFFFFFFFFu, Mv = 0u, Ph, Mh;
#pragma unroll
        for (int c = 0; c < KR; ++c) {
            if (c < mt) {
                uint32_t Eq = 0u;
#pragma unroll
                for (int r = 0; r < KR; ++r)
                    // `one` holds 1 but is a run-time value, so the bit is set by a multiply-add:
                    // it issues on the FMA pipe while the comparisons keep the integer ALU busy
                    asm("{ .reg .pred q; setp.eq.s32 q, %1, %2; @q mad.lo.u32 %0, %3, %4, %0; }"
                        : "+r"(Eq) : "r"(pat[r]), "r"(txt[c]), "r"(one), "r"(1u << r));
                word_column(Eq, Pv, Mv, Ph, Mh);
            }
        }
        const uint32_t msk = low_mask(mp);
        const int d = mt + __popc(Pv & msk) - __popc(Mv & msk);
        s_dist[tid] = d;
        // one term of d_K (Section 3.2): distance / longer prefix, from the quotient table
        s_term[tid] = a.norm_mode == SR_NORM_NONE ? (double)d : kQuot.v[d * 33 + mp];
        if (a.pair_dist) a.pair_dist[g * P + p] = d;
    }
    __syncthreads();
    // ---- d_K: ordered fp64 sum, strict threshold (Eq. 2): one thread per group of the CTA
    if (tid < groups_per_cta) {
        const size_t gg = (size_t)blockIdx.x * groups_per_cta + tid;
        if (gg < (size_t)a.n_groups) group_sum_and_gate(s_term + tid * P, s_dist + tid * P, P, a, gg);
    }
}

template <int KR>
int launch_gate_direct(const GateArgs& a, cudaStream_t s) {
    const int P = pairs_of(a.N);
    const int threads = P <= 256 ? 256 : 512;
    const int gpc = threads / P;
    const int smem = gpc * P * 12;
    const int blocks = (a.n_groups + gpc - 1) / gpc;
    gate_direct_kernel<KR><<<blocks, threads, smem, s>>>(a, gpc, 1u);
    SR_LAUNCH_CHECK("gate_direct_kernel");
    return SR_OK;
}

}  // namespace

int launch_gate_single(const GateArgs& a, cudaStream_t s) {
    if (a.n_groups == 0) return SR_OK;
    if (a.K <= 4) return launch_gate_direct<4>(a, s);
    if (a.K <= 8) return launch_gate_direct<8>(a, s);
    if (a.K <= 12) return launch_gate_direct<12>(a, s);
    if (a.K <= 16) return launch_gate_direct<16>(a, s);
    const int N = a.N, P = pairs_of(N);
    SingleLayout L;
    int h = 32;
    while (h < 2 * N * a.K) h <<= 1;
    L.hslots = h;
    L.hlog = 0;
    while ((1 << L.hlog) < h) ++L.hlog;
    L.hshift = 32 - L.hlog;
    L.qshift = 0;
    while ((4 << L.qshift) < a.K) ++L.qshift;
    L.n_items = N << L.qshift;
    int off = 0;
    auto take = [&](int bytes) { int o = off; off = (off + bytes + 15) & ~15; return o; };
    L.off_hash = take(L.hslots * 8);
    L.off_peq = take(N * kPeqPitch * 4);
    L.zero_words16 = off >> 4;                      // table and masks are adjacent: one clear
    L.off_map = take(L.hslots * N);
    L.map_words16 = (L.hslots * N) >> 4;            // hslots >= 32: a whole number of 16-byte units
    L.off_txt = take(N * kTxtPitch * 2);
    L.off_len = take(N * 4);
    L.group_bytes = off;
    const bool warp = N <= 8;
    int threads, groups_per_cta;
    if (warp) {
        // eight groups per CTA, fewer when shared memory would leave an SM under four CTAs
        groups_per_cta = 8;
        while (groups_per_cta > 2 && groups_per_cta * (L.group_bytes + P * 12) > 56 * 1024) groups_per_cta >>= 1;
        threads = groups_per_cta * 32;
    } else {
        groups_per_cta = 1;
        threads = (P + 31) & ~31;
        if (threads > 512) threads = 512;
        if (threads * kMaxItems < L.n_items) return SR_ERR_BAD_N;   // cannot happen for N <= 32
    }
    off = groups_per_cta * L.group_bytes;
    L.off_term = take(groups_per_cta * P * 8);
    L.off_dist = take(groups_per_cta * P * 4);
    const int smem = off;
    const int blocks = (a.n_groups + groups_per_cta - 1) / groups_per_cta;
    if (smem > 48 * 1024) {
        // per-device note of what each kernel was already allowed: the opt-in call is host
        // time on a path whose small calls are launch-bound
        static int granted[2][64] = {};
        int dev = 0;
        SR_CUDA_TRY(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64 || granted[warp][dev] < smem) {
            if (warp)
                SR_CUDA_TRY(cudaFuncSetAttribute(gate_single_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            else
                SR_CUDA_TRY(cudaFuncSetAttribute(gate_single_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            if (dev >= 0 && dev < 64) granted[warp][dev] = smem;
        }
    }
    if (warp) gate_single_kernel<true><<<blocks, threads, smem, s>>>(a, L);
    else gate_single_kernel<false><<<blocks, threads, smem, s>>>(a, L);
    SR_LAUNCH_CHECK("gate_single_kernel");
    return SR_OK;
}

}  // namespace sr
