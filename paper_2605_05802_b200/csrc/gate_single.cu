// Single-word gate kernel: prefixes of at most 32 symbols (action-level gate,
// Section 3.2 of the paper: d_K at K <= T_max = 30).
//
// One CTA handles `gpb` consecutive groups.  Per group it
//   1. stages the N prefixes once in shared memory (int4 loads),
//   2. renames the group's distinct IDs to dense local ids through a small
//      open-addressing table in shared memory,
//   3. builds the match masks Peq[i][id] (bit r set iff rollout i has symbol id at
//      position r),
//   4. runs one thread per pair through the bit-parallel column recurrence (one
//      32-bit word of +1 / -1 vertical deltas per pair; the distance is read off as
//      n + popc(Pv) - popc(Mv), so no per-column score is kept),
//   5. adds the normalised terms in fp64 in pair order, thresholds, and writes out.
#include "common.cuh"

namespace sr {
namespace {

struct SingleLayout {
    int gpb;        // groups per CTA
    int kpad;       // K rounded up to a multiple of 4 (<= 32)
    int hslots;     // hash slots per group (power of two)
    int hshift;     // 32 - log2(hslots)
    int dmax;       // upper bound of distinct symbols per group (N * K)
    // byte offsets into dynamic shared memory
    int off_len, off_sym, off_gid, off_owner, off_cnt, off_peq, off_dist, off_term, off_pairs;
    int total;
};

__global__ void __launch_bounds__(1024)
gate_single_kernel(GateArgs a, SingleLayout L) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = a.N, K = a.K, P = pairs_of(N);
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int g0 = blockIdx.x * L.gpb;
    const int ng = min(L.gpb, a.n_groups - g0);

    int32_t* s_len = reinterpret_cast<int32_t*>(smem + L.off_len);          // [gpb][N]
    int32_t* s_sym = reinterpret_cast<int32_t*>(smem + L.off_sym);          // [gpb][N][kpad]
    uint16_t* s_gid = reinterpret_cast<uint16_t*>(smem + L.off_gid);        // [gpb][N][kpad]
    uint32_t* s_owner = reinterpret_cast<uint32_t*>(smem + L.off_owner);    // [gpb][hslots]
    int32_t* s_cnt = reinterpret_cast<int32_t*>(smem + L.off_cnt);          // [gpb]
    uint32_t* s_peq = reinterpret_cast<uint32_t*>(smem + L.off_peq);        // [gpb][N][dmax]
    int32_t* s_dist = reinterpret_cast<int32_t*>(smem + L.off_dist);        // [gpb][P]
    double* s_term = reinterpret_cast<double*>(smem + L.off_term);          // [gpb][P]
    uint16_t* s_pairs = reinterpret_cast<uint16_t*>(smem + L.off_pairs);    // [P]  i | j << 8

    // ---- lengths, pair table, table clears
    bool neg = false;
    for (int e = tid; e < ng * N; e += nthr) {
        int len = a.lens ? a.lens[(size_t)g0 * N + e] : K;
        if (len < 0) { len = 0; neg = true; }
        s_len[e] = min(len, K);
    }
    if (neg && a.status) atomicOr(a.status, SR_STATUS_NEG_LEN);
    for (int p = tid; p < P; p += nthr) {
        int i, j;
        pair_from_index(p, N, i, j);
        s_pairs[p] = (uint16_t)(i | (j << 8));
    }
    for (int e = tid; e < ng * L.hslots; e += nthr) s_owner[e] = 0u;
    if (tid < ng) s_cnt[tid] = 0;

    // ---- stage the prefixes: one int4 per thread per trip, 16-byte aligned by contract
    const int q4 = (K + 3) >> 2, pitch4 = L.kpad >> 2;   // q4 == 0 when K == 0: nothing to stage
    for (int e = tid; e < ng * N * q4; e += nthr) {
        const int row = e / q4, q = e - row * q4;
        const int4 v = __ldg(reinterpret_cast<const int4*>(a.seqs + ((size_t)g0 * N + row) * a.stride) + q);
        reinterpret_cast<int4*>(s_sym)[row * pitch4 + q] = v;
    }
    __syncthreads();

    // ---- dense local ids: claim a slot per distinct symbol (slot identity = the
    // symbol of the claiming position), then number the claimed slots
    const int per_group = N * L.kpad;
    for (int e = tid; e < ng * per_group; e += nthr) {
        const int g = e / per_group, rem = e - g * per_group;
        const int i = rem / L.kpad, r = rem - i * L.kpad;
        if (r >= s_len[g * N + i]) continue;
        const int32_t sym = s_sym[e];
        uint32_t h = ((uint32_t)sym * 0x9E3779B1u) >> L.hshift;
        uint32_t* own = s_owner + g * L.hslots;
        // the table has at least twice as many slots as symbols, so a free or matching
        // slot is always found; the trip count is bounded all the same
        for (int probe = 0; probe < L.hslots; ++probe) {
            uint32_t o = own[h];
            if (o == 0u) o = atomicCAS(&own[h], 0u, (uint32_t)rem + 1u);
            if (o == 0u || s_sym[g * per_group + (int)o - 1] == sym) break;
            h = (h + 1u) & (uint32_t)(L.hslots - 1);
        }
        s_gid[e] = (uint16_t)h;
    }
    __syncthreads();
    for (int e = tid; e < ng * L.hslots; e += nthr) {
        if (s_owner[e] != 0u) {
            const int g = e / L.hslots;
            s_owner[e] = (uint32_t)atomicAdd(&s_cnt[g], 1);
        }
    }
    __syncthreads();
    for (int g = 0; g < ng; ++g) {
        const int cnt = s_cnt[g];
        uint32_t* peq = s_peq + (size_t)g * N * L.dmax;
        for (int e = tid; e < N * cnt; e += nthr) {
            const int i = e / cnt;
            peq[i * L.dmax + (e - i * cnt)] = 0u;
        }
    }
    __syncthreads();
    for (int e = tid; e < ng * per_group; e += nthr) {
        const int g = e / per_group, rem = e - g * per_group;
        const int i = rem / L.kpad, r = rem - i * L.kpad;
        if (r >= s_len[g * N + i]) continue;
        const uint32_t gid = s_owner[g * L.hslots + s_gid[e]];
        s_gid[e] = (uint16_t)gid;
        atomicOr(&s_peq[((size_t)g * N + i) * L.dmax + gid], 1u << r);
    }
    __syncthreads();

    // ---- one thread per pair
    if (tid < ng * P) {
        const int g = tid / P, p = tid - g * P;
        const int pr = s_pairs[p];
        int pi = pr & 0xFF, pj = pr >> 8;
        const int mi = s_len[g * N + pi], mj = s_len[g * N + pj];
        int mp = mi, mt = mj;                       // pattern = the longer prefix (rows)
        if (mj > mi) { const int t = pi; pi = pj; pj = t; mp = mj; mt = mi; }
        const uint32_t* peq = s_peq + ((size_t)g * N + pi) * L.dmax;
        const uint16_t* txt = s_gid + (size_t)g * per_group + pj * L.kpad;
        uint32_t Pv = 0xFFFFFFFFu, Mv = 0u;
        for (int c = 0; c < mt; ++c) {
            const uint32_t Eq = peq[txt[c]];
            const uint32_t Xv = Eq | Mv;
            const uint32_t Xh = (((Eq & Pv) + Pv) ^ Pv) | Eq;
            uint32_t Ph = Mv | ~(Xh | Pv);
            uint32_t Mh = Pv & Xh;
            Ph = (Ph << 1) | 1u;
            Mh = Mh << 1;
            Pv = Mh | ~(Xv | Ph);
            Mv = Ph & Xv;
        }
        const uint32_t msk = low_mask(mp);
        const int d = mt + __popc(Pv & msk) - __popc(Mv & msk);
        s_dist[tid] = d;
        s_term[tid] = pair_term(d, mi, mj, a.norm_mode);
        if (a.pair_dist) a.pair_dist[(size_t)g0 * P + tid] = d;
    }
    __syncthreads();

    // ---- d_K: ordered fp64 sum, strict threshold (Eq. 2)
    if (tid < ng) {
        double s = 0.0;
        int isum = 0;
        for (int p = 0; p < P; ++p) {
            s = __dadd_rn(s, s_term[tid * P + p]);
            isum += s_dist[tid * P + p];
        }
        const double dk = __ddiv_rn(s, (double)P);
        if (a.pair_sum) a.pair_sum[g0 + tid] = isum;
        if (a.mean) a.mean[g0 + tid] = dk;
        a.stop[g0 + tid] = dk < a.threshold ? 1 : 0;
    }
}

}  // namespace

int launch_gate_single(const GateArgs& a, cudaStream_t s) {
    if (a.n_groups == 0) return SR_OK;
    const int N = a.N, P = pairs_of(N);
    SingleLayout L;
    L.kpad = (a.K + 3) & ~3;
    if (L.kpad == 0) L.kpad = 4;
    L.dmax = N * a.K > 0 ? N * a.K : 1;
    int h = 32;
    while (h < 2 * N * L.kpad) h <<= 1;
    L.hslots = h;
    L.hshift = 32;
    while ((1 << (32 - L.hshift)) < h) --L.hshift;
    int gpb = 256 / P;
    if (gpb < 1) gpb = 1;
    if (gpb > 32) gpb = 32;
    int max_smem = 0, dev = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    SR_CUDA_TRY(cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
    while (true) {
        L.gpb = gpb;
        int off = 0;
        auto take = [&](int bytes) { int o = off; off = (off + bytes + 15) & ~15; return o; };
        L.off_len = take(gpb * N * 4);
        L.off_sym = take(gpb * N * L.kpad * 4);
        L.off_gid = take(gpb * N * L.kpad * 2);
        L.off_owner = take(gpb * L.hslots * 4);
        L.off_cnt = take(gpb * 4);
        L.off_peq = take(gpb * N * L.dmax * 4);
        L.off_dist = take(gpb * P * 4);
        L.off_term = take(gpb * P * 8);
        L.off_pairs = take(P * 2);
        L.total = off;
        // keep at least two CTAs per SM when the group count allows it
        if (L.total <= max_smem / 2 || gpb == 1) break;
        --gpb;
    }
    if (L.total > max_smem) return SR_ERR_BAD_N;
    int threads = (L.gpb * P + 31) & ~31;
    if (threads < 64) threads = 64;
    SR_CUDA_TRY(cudaFuncSetAttribute(gate_single_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     L.total));
    const int blocks = (a.n_groups + L.gpb - 1) / L.gpb;
    gate_single_kernel<<<blocks, threads, L.total, s>>>(a, L);
    SR_LAUNCH_CHECK("gate_single_kernel");
    return SR_OK;
}

}  // namespace sr
