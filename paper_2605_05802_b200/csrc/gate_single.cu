// Single-word gate kernel: prefixes of at most 32 symbols (action-level gate,
// Section 3.2 of the paper: d_K at K <= T_max = 30).
//
// One CTA handles `gpb` consecutive groups.  Per group it
//   1. stages the N prefixes once in shared memory (int4 loads, rows of 32 words),
//   2. renames the group's distinct IDs to dense local ids through a small
//      open-addressing table in shared memory,
//   3. builds, per rollout i, a byte map id -> a position of that symbol in rollout i
//      and the match masks peq[i][position] (bit r set iff rollout i has the same
//      symbol at r); the map costs one byte per (rollout, id) instead of one word,
//      which is what lets several CTAs share an SM,
//   4. runs one thread per pair through the bit-parallel column recurrence (one
//      32-bit word of +1 / -1 vertical deltas per pair; the distance is read off as
//      n + popc(Pv) - popc(Mv), so no per-column score is kept),
//   5. adds the normalised terms in fp64 in pair order, thresholds, and writes out.
// Index arithmetic uses shifts only (rows are 32 words), since integer division by a
// run-time value costs more than a whole column of the recurrence.
#include "common.cuh"

namespace sr {
namespace {

// d / L for 0 <= d, L <= 32 (0 when L == 0), correctly rounded: the compiler's
// constant evaluation of an IEEE division equals the device's __ddiv_rn.
struct QuotientTable {
    double v[33 * 33];
    constexpr QuotientTable() : v() {
        for (int d = 0; d <= 32; ++d)
            for (int l = 0; l <= 32; ++l) v[d * 33 + l] = l > 0 ? (double)d / (double)l : 0.0;
    }
};
__device__ const QuotientTable kQuot = QuotientTable();

// Row pitch (16-bit elements) of the local-id rows: 17 words, so that pair threads
// reading the same column of different rollouts hit different banks.
constexpr int kGidPitch = 34;
// Row pitch (words) of the per-rollout match masks: 32 masks indexed by a
// representative position of the symbol, plus one all-zero mask for "absent".
constexpr int kPeqPitch = 33;
constexpr uint32_t kAbsent = 32;

struct SingleLayout {
    int gpb;        // groups per CTA
    int hslots;     // hash slots per group (power of two)
    int hshift;     // 32 - log2(hslots)
    int mpitch;     // bytes per row of the id -> representative-position map (multiple of 4)
    // Byte offsets into dynamic shared memory.  `off_build` holds the staged symbols and
    // the hash table while the local ids are being assigned; once they are final the
    // same bytes are reused for the map and the match masks.
    int off_len, off_gid, off_cnt, off_dist, off_term, off_pairs, off_build;
    int build_bytes;                       // per group
    int sym_off, owner_off, sgid_off;      // within a group's build area (phase 1)
    int map_off, peq_off;                  // within a group's build area (phase 2)
    int total;
};

__global__ void __launch_bounds__(1024)
gate_single_kernel(GateArgs a, SingleLayout L) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = a.N, K = a.K, P = pairs_of(N);
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int g0 = blockIdx.x * L.gpb;
    const int ng = min(L.gpb, a.n_groups - g0);
    const int rows = ng * N;                       // staged prefixes, 32 words each
    const int per_group = N << 5;

    int32_t* s_len = reinterpret_cast<int32_t*>(smem + L.off_len);          // [gpb*N]
    uint16_t* s_gid = reinterpret_cast<uint16_t*>(smem + L.off_gid);        // [gpb*N][kGidPitch]
    int32_t* s_cnt = reinterpret_cast<int32_t*>(smem + L.off_cnt);          // [gpb]
    int32_t* s_dist = reinterpret_cast<int32_t*>(smem + L.off_dist);        // [gpb][P]
    double* s_term = reinterpret_cast<double*>(smem + L.off_term);          // [gpb][P]
    uint16_t* s_pairs = reinterpret_cast<uint16_t*>(smem + L.off_pairs);    // [P]  i | j << 8
    unsigned char* s_build = smem + L.off_build;                            // [gpb][build_bytes]
    auto sym_of = [&](int g) { return reinterpret_cast<int32_t*>(s_build + (size_t)g * L.build_bytes + L.sym_off); };
    auto owner_of = [&](int g) { return reinterpret_cast<uint32_t*>(s_build + (size_t)g * L.build_bytes + L.owner_off); };
    auto sgid_of = [&](int g) { return reinterpret_cast<uint16_t*>(s_build + (size_t)g * L.build_bytes + L.sgid_off); };
    auto map_of = [&](int g) { return s_build + (size_t)g * L.build_bytes + L.map_off; };
    auto peq_of = [&](int g) { return reinterpret_cast<uint32_t*>(s_build + (size_t)g * L.build_bytes + L.peq_off); };

    // ---- lengths, pair table, hash-table clear
    bool neg = false;
    for (int e = tid; e < rows; e += nthr) {
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
    for (int g = 0; g < ng; ++g) {
        uint32_t* own = owner_of(g);
        for (int e = tid; e < L.hslots; e += nthr) own[e] = 0u;
    }
    if (tid < ng) s_cnt[tid] = 0;

    // ---- stage the prefixes: 8 lanes per row, one int4 each (16-byte aligned by contract)
    const int q4 = (K + 3) >> 2;                   // 0 when K == 0: nothing to stage
    for (int e = tid; e < rows * 8; e += nthr) {
        const int row = e >> 3, q = e & 7;
        if (q < q4) {
            const int g = row / N, i = row - g * N;
            const int4 v = __ldg(reinterpret_cast<const int4*>(a.seqs + ((size_t)g0 * N + row) * a.stride) + q);
            reinterpret_cast<int4*>(sym_of(g))[i * 8 + q] = v;
        }
    }
    __syncthreads();

    // ---- dense local ids: claim a slot per distinct symbol (slot identity = the
    // symbol of the claiming position); the claimant draws the group's next free id
    for (int g = 0; g < ng; ++g) {
        uint32_t* own = owner_of(g);
        uint16_t* sgid = sgid_of(g);
        const int32_t* sym_g = sym_of(g);
        for (int e = tid; e < per_group; e += nthr) {
            if ((e & 31) >= s_len[g * N + (e >> 5)]) continue;
            const int32_t sym = sym_g[e];
            uint32_t h = ((uint32_t)sym * 0x9E3779B1u) >> L.hshift;
            // the table has at least twice as many slots as symbols, so a free or matching
            // slot is always found; the trip count is bounded all the same
            for (int probe = 0; probe < L.hslots; ++probe) {
                uint32_t o = own[h];
                if (o == 0u) o = atomicCAS(&own[h], 0u, (uint32_t)e + 1u);
                if (o == 0u) { sgid[h] = (uint16_t)atomicAdd(&s_cnt[g], 1); break; }
                if (sym_g[o - 1u] == sym) break;
                h = (h + 1u) & (uint32_t)(L.hslots - 1);
            }
            s_gid[(g * N + (e >> 5)) * kGidPitch + (e & 31)] = (uint16_t)h;
        }
    }
    __syncthreads();
    for (int g = 0; g < ng; ++g) {
        const uint16_t* sgid = sgid_of(g);
        for (int e = tid; e < per_group; e += nthr) {
            if ((e & 31) >= s_len[g * N + (e >> 5)]) continue;
            uint16_t* slot = s_gid + (g * N + (e >> 5)) * kGidPitch + (e & 31);
            *slot = sgid[*slot];
        }
    }
    __syncthreads();

    // ---- the staged symbols and the hash table are dead; their bytes now hold, per
    // rollout i, map[i][id] = a position of rollout i holding symbol id (kAbsent if none)
    // and peq[i][pos] = bit mask of all positions of rollout i with the symbol found at pos
    for (int g = 0; g < ng; ++g) {                 // 16-byte stores: map = "absent", masks = 0
        uint4* init = reinterpret_cast<uint4*>(map_of(g));
        const int map_q = L.peq_off >> 4, all_q = (L.peq_off + ((N * kPeqPitch * 4 + 15) & ~15)) >> 4;
        const uint32_t absent4 = kAbsent * 0x01010101u;
        for (int e = tid; e < all_q; e += nthr)
            init[e] = e < map_q ? make_uint4(absent4, absent4, absent4, absent4) : make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    for (int g = 0; g < ng; ++g) {
        volatile unsigned char* map = map_of(g);
        for (int e = tid; e < per_group; e += nthr) {
            const int i = e >> 5, r = e & 31;
            if (r >= s_len[g * N + i]) continue;
            // several positions with the same symbol store to the same byte; whichever store
            // lands last names the representative, and any of them is a valid one
            map[i * L.mpitch + s_gid[(g * N + i) * kGidPitch + r]] = (unsigned char)r;
        }
    }
    __syncthreads();
    for (int g = 0; g < ng; ++g) {
        const unsigned char* map = map_of(g);
        uint32_t* peq = peq_of(g);
        for (int e = tid; e < per_group; e += nthr) {
            const int i = e >> 5, r = e & 31;
            if (r >= s_len[g * N + i]) continue;
            const uint32_t rep = map[i * L.mpitch + s_gid[(g * N + i) * kGidPitch + r]];
            atomicOr(&peq[i * kPeqPitch + rep], 1u << r);
        }
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
        const unsigned char* map = map_of(g) + pi * L.mpitch;
        const uint32_t* peq = peq_of(g) + pi * kPeqPitch;
        const uint16_t* txt = s_gid + (g * N + pj) * kGidPitch;
        uint32_t Pv = 0xFFFFFFFFu, Mv = 0u;
        for (int c = 0; c < mt; ++c) {
            const uint32_t Eq = peq[map[txt[c]]];
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
        // one term of d_K (Section 3.2): distance / longer prefix, from the quotient table
        s_term[tid] = a.norm_mode == SR_NORM_NONE ? (double)d : kQuot.v[d * 33 + mp];
        if (a.pair_dist) a.pair_dist[(size_t)g0 * P + tid] = d;
    }
    __syncthreads();

    // ---- d_K: ordered fp64 sum, strict threshold (Eq. 2).  The loads are issued eight
    // at a time ahead of the (necessarily sequential) additions.
    if (tid < ng) {
        const double* term = s_term + tid * P;
        const int32_t* dist = s_dist + tid * P;
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
        if (a.pair_sum) a.pair_sum[g0 + tid] = isum;
        if (a.mean) a.mean[g0 + tid] = dk;
        a.stop[g0 + tid] = dk < a.threshold ? 1 : 0;
    }
}

// ---------------------------------------------------------------------------------
// Groups of at most 8 rollouts (28 pairs: the paper's G = 8) fit one warp: lane r owns
// position r of every prefix during the set-up and pair `lane` during the recurrence,
// so the whole group is processed with warp-level synchronisation only and the warps
// of a CTA never wait for one another.  Same steps and tables as the CTA-wide kernel.
struct WarpLayout {
    int hslots, hshift, mpitch, kshift;
    int warp_bytes;                               // shared memory per warp, multiple of 16
    int sym_off, owner_off, sgid_off;             // build area, phase 1
    int map_off, peq_off;                         // build area, phase 2 (same bytes)
    int gid_off, len_off, dist_off, term_off;
};

constexpr int kWarpsPerCta = 8;

__global__ void __launch_bounds__(kWarpsPerCta * 32)
gate_single_warp_kernel(GateArgs a, WarpLayout L) {
    extern __shared__ __align__(16) unsigned char smem[];
    const int N = a.N, K = a.K, P = pairs_of(N);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = blockIdx.x * kWarpsPerCta + warp;
    if (g >= a.n_groups) return;                   // whole warps leave; no CTA-wide barrier below
    unsigned char* base = smem + (size_t)warp * L.warp_bytes;
    int32_t* s_sym = reinterpret_cast<int32_t*>(base + L.sym_off);        // [N][32]
    uint32_t* s_owner = reinterpret_cast<uint32_t*>(base + L.owner_off);  // [hslots]
    uint16_t* s_sgid = reinterpret_cast<uint16_t*>(base + L.sgid_off);    // [hslots]
    unsigned char* s_map = base + L.map_off;                              // [N][mpitch]
    uint32_t* s_peq = reinterpret_cast<uint32_t*>(base + L.peq_off);      // [N][33]
    uint16_t* s_gid = reinterpret_cast<uint16_t*>(base + L.gid_off);      // [N][kGidPitch]
    int32_t* s_len = reinterpret_cast<int32_t*>(base + L.len_off);        // [8], [8] = id counter
    int32_t* s_dist = reinterpret_cast<int32_t*>(base + L.dist_off);      // [32]
    double* s_term = reinterpret_cast<double*>(base + L.term_off);        // [32]

    if (lane < N) {
        int len = a.lens ? a.lens[(size_t)g * N + lane] : K;
        if (len < 0) { len = 0; if (a.status) atomicOr(a.status, SR_STATUS_NEG_LEN); }
        s_len[lane] = min(len, K);
    }
    if (lane == 8) s_len[8] = 0;
    for (int e = lane; e < L.hslots; e += 32) s_owner[e] = 0u;
    __syncwarp();
    // Elements (rollout i, position r) are spread over the lanes with r < 2^ks, 2^ks the
    // power of two >= K: at the paper's K = 10 or 15 a warp covers two rollouts per trip.
    const int ks = L.kshift, kmask = (1 << ks) - 1, n_elem = N << ks;
    // ---- symbols (consecutive lanes read consecutive positions of a row)
    for (int e = lane; e < n_elem; e += 32) {
        const int i = e >> ks, r = e & kmask;
        if (r < s_len[i]) s_sym[i * 32 + r] = __ldg(a.seqs + ((size_t)g * N + i) * a.stride + r);
    }
    __syncwarp();
    // ---- dense local ids
    for (int e = lane; e < n_elem; e += 32) {
        const int i = e >> ks, r = e & kmask;
        if (r >= s_len[i]) continue;
        const int el = i * 32 + r;
        const int32_t sym = s_sym[el];
        uint32_t h = ((uint32_t)sym * 0x9E3779B1u) >> L.hshift;
        for (int probe = 0; probe < L.hslots; ++probe) {      // a free or matching slot always exists
            uint32_t o = s_owner[h];
            if (o == 0u) o = atomicCAS(&s_owner[h], 0u, (uint32_t)el + 1u);
            if (o == 0u) { s_sgid[h] = (uint16_t)atomicAdd(&s_len[8], 1); break; }
            if (s_sym[o - 1u] == sym) break;
            h = (h + 1u) & (uint32_t)(L.hslots - 1);
        }
        s_gid[i * kGidPitch + r] = (uint16_t)h;
    }
    __syncwarp();
    for (int e = lane; e < n_elem; e += 32) {
        const int i = e >> ks, r = e & kmask;
        if (r < s_len[i]) s_gid[i * kGidPitch + r] = s_sgid[s_gid[i * kGidPitch + r]];
    }
    __syncwarp();
    // ---- the symbols and the hash table are dead: their bytes become the map and the masks
    {
        uint4* init = reinterpret_cast<uint4*>(s_map);
        const int map_q = L.peq_off >> 4, all_q = (L.peq_off + ((N * kPeqPitch * 4 + 15) & ~15)) >> 4;
        const uint32_t absent4 = kAbsent * 0x01010101u;
        for (int e = lane; e < all_q; e += 32)
            init[e] = e < map_q ? make_uint4(absent4, absent4, absent4, absent4) : make_uint4(0u, 0u, 0u, 0u);
    }
    __syncwarp();
    for (int e = lane; e < n_elem; e += 32) {
        const int i = e >> ks, r = e & kmask;
        // several positions with the same symbol store to the same byte; any of them is a
        // valid representative
        if (r < s_len[i])
            reinterpret_cast<volatile unsigned char*>(s_map)[i * L.mpitch + s_gid[i * kGidPitch + r]] = (unsigned char)r;
    }
    __syncwarp();
    for (int e = lane; e < n_elem; e += 32) {
        const int i = e >> ks, r = e & kmask;
        if (r < s_len[i]) {
            const uint32_t rep = s_map[i * L.mpitch + s_gid[i * kGidPitch + r]];
            atomicOr(&s_peq[i * kPeqPitch + rep], 1u << r);
        }
    }
    __syncwarp();
    // ---- lane p runs pair p
    if (lane < P) {
        int pi, pj;
        pair_from_index(lane, N, pi, pj);
        const int mi = s_len[pi], mj = s_len[pj];
        int mp = mi, mt = mj;
        if (mj > mi) { const int t = pi; pi = pj; pj = t; mp = mj; mt = mi; }
        const unsigned char* map = s_map + pi * L.mpitch;
        const uint32_t* peq = s_peq + pi * kPeqPitch;
        const uint16_t* txt = s_gid + pj * kGidPitch;
        uint32_t Pv = 0xFFFFFFFFu, Mv = 0u;
        for (int c = 0; c < mt; ++c) {
            const uint32_t Eq = peq[map[txt[c]]];
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
        s_dist[lane] = d;
        s_term[lane] = a.norm_mode == SR_NORM_NONE ? (double)d : kQuot.v[d * 33 + mp];
        if (a.pair_dist) a.pair_dist[(size_t)g * P + lane] = d;
    }
    __syncwarp();
    if (lane == 0) {                              // ordered fp64 sum (Section 3.2), strict gate (Eq. 2)
        double s = 0.0;
        int isum = 0, p = 0;
        for (; p + 4 <= P; p += 4) {
            const double t0 = s_term[p], t1 = s_term[p + 1], t2 = s_term[p + 2], t3 = s_term[p + 3];
            isum += s_dist[p] + s_dist[p + 1] + s_dist[p + 2] + s_dist[p + 3];
            s = __dadd_rn(__dadd_rn(__dadd_rn(__dadd_rn(s, t0), t1), t2), t3);
        }
        for (; p < P; ++p) { s = __dadd_rn(s, s_term[p]); isum += s_dist[p]; }
        const double dk = __ddiv_rn(s, (double)P);
        if (a.pair_sum) a.pair_sum[g] = isum;
        if (a.mean) a.mean[g] = dk;
        a.stop[g] = dk < a.threshold ? 1 : 0;
    }
}

int launch_gate_single_warp(const GateArgs& a, cudaStream_t s) {
    const int N = a.N;
    WarpLayout L;
    int h = 32;
    while (h < 2 * N * a.K) h <<= 1;
    L.hslots = h;
    L.hshift = 32;
    while ((1 << (32 - L.hshift)) < h) --L.hshift;
    L.kshift = 0;
    while ((1 << L.kshift) < a.K) ++L.kshift;
    int mwords = (N * a.K + 3) >> 2;
    if ((mwords & 1) == 0) ++mwords;
    L.mpitch = mwords * 4;
    L.sym_off = 0;
    L.owner_off = N * 32 * 4;
    L.sgid_off = L.owner_off + L.hslots * 4;
    L.map_off = 0;
    L.peq_off = (N * L.mpitch + 15) & ~15;
    const int phase1 = L.sgid_off + L.hslots * 2;
    const int phase2 = L.peq_off + ((N * kPeqPitch * 4 + 15) & ~15);
    int off = ((phase1 > phase2 ? phase1 : phase2) + 15) & ~15;
    auto take = [&](int bytes) { int o = off; off = (off + bytes + 15) & ~15; return o; };
    L.gid_off = take(N * kGidPitch * 2);
    L.len_off = take(9 * 4);
    L.dist_off = take(32 * 4);
    L.term_off = take(32 * 8);
    L.warp_bytes = off;
    const int smem = L.warp_bytes * kWarpsPerCta;
    SR_CUDA_TRY(cudaFuncSetAttribute(gate_single_warp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const int blocks = (a.n_groups + kWarpsPerCta - 1) / kWarpsPerCta;
    gate_single_warp_kernel<<<blocks, kWarpsPerCta * 32, smem, s>>>(a, L);
    SR_LAUNCH_CHECK("gate_single_warp_kernel");
    return SR_OK;
}

}  // namespace

int launch_gate_single(const GateArgs& a, cudaStream_t s) {
    if (a.n_groups == 0) return SR_OK;
    if (a.N <= 8) return launch_gate_single_warp(a, s);
    const int N = a.N, P = pairs_of(N);
    SingleLayout L;
    int h = 32;
    while (h < 2 * N * a.K) h <<= 1;
    L.hslots = h;
    L.hshift = 32;
    while ((1 << (32 - L.hshift)) < h) --L.hshift;
    // map rows: one byte per distinct id (at most N*K), padded to an odd number of words
    // so that consecutive rows start in different banks
    int mwords = (N * a.K + 3) >> 2;
    if ((mwords & 1) == 0) ++mwords;
    L.mpitch = mwords * 4;
    L.sym_off = 0;
    L.owner_off = N * 32 * 4;
    L.map_off = 0;
    L.peq_off = (N * L.mpitch + 15) & ~15;
    L.sgid_off = L.owner_off + L.hslots * 4;
    const int phase1 = L.sgid_off + L.hslots * 2;
    const int phase2 = L.peq_off + ((N * kPeqPitch * 4 + 15) & ~15);
    L.build_bytes = ((phase1 > phase2 ? phase1 : phase2) + 15) & ~15;
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
        L.off_gid = take(gpb * N * kGidPitch * 2);
        L.off_cnt = take(gpb * 4);
        L.off_dist = take(gpb * P * 4);
        L.off_term = take(gpb * P * 8);
        L.off_pairs = take(P * 2);
        L.off_build = take(gpb * L.build_bytes);
        L.total = off;
        if (L.total <= max_smem / 4 || gpb == 1) break;   // leave room for several CTAs per SM
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
