// Multi-word gate: prefixes of 33..SR_MAX_K symbols (token-level gate; same
// d_K of Section 3.2 of the paper, applied to token IDs).
//
// The edit-distance matrix of a pair is cut into 32-row blocks of the pattern; a
// block keeps its +1 / -1 vertical deltas in two 32-bit words and is advanced one
// text column at a time by the bit-vector recurrence, with the horizontal delta
// leaving a block entering the block below.  The work is organised as a pipeline
// of four launches on the caller's stream, sharing a caller-provided workspace:
//
//   prep     one CTA per (group, pattern rollout): hashes the pattern's symbols
//            in shared memory, then translates every text paired with it into a
//            "loc" stream: for text column c the position of the column's symbol in
//            the pattern (0x7FFF: absent; bit 15 set: several occurrences, walk
//            the pattern's chain).  A block's match word is then just
//            1 << (loc - first_row_of_block), no table lookup.  Also bins the pairs
//            by (team shape, text length).
//   order    counting sort of the pairs by bin: longest warp tasks first, one team
//            shape and similar text lengths per bin; warp-task table.
//   dp       persistent warps pull tasks.  A task is a warp of 32/T teams; a team of
//            T lanes (T in {1, 2, 4, 8}; up to 32 in small batches) owns one pair, lane l
//            holding R <= 6 consecutive blocks (32*R rows) in registers.  Lanes are skewed by four columns; the
//            delta words of a lane's last block reach the next lane by warp shuffles.
//            All pairs of a task share (T, R) and have similar lengths, so the warp's
//            lanes stay busy.
//   finish   one thread per group: ordered fp64 sum of the normalised terms,
//            threshold, outputs.
//
// Band (decide mode).  There prep also counts, per pair, the positions at which the two
// prefixes differ (after the common prefix): that count plus the length difference is an
// UPPER bound of the distance (substitute the differing positions, insert or delete the
// rest), and the threshold caps how large a distance can still matter.  An optimal
// alignment of distance <= ub never leaves the diagonals d = row - column with
// |d| + |(m - n) - d| <= ub (Ukkonen's cut-off), so pairs whose bound is small run a
// banded task, served by CTAs of their own within the dp launch: the pattern's 32-row
// blocks are grouped in stripes of R blocks, stripe g lives on lane g mod T of a ring of
// T lanes and is advanced only over the columns where the band crosses it; a stripe the
// band enters starts from +1 vertical deltas below the stripe above it and a stripe whose
// upper neighbour the band has left takes +1 horizontal deltas from above -- both
// over-estimates of cells outside the band, which leave every cell on an optimal path
// exact.  The distance is read from a running score
// at the bottom of the last stripe.  A result within the bound is the exact distance; a
// result above it only says "more than the bound".  (Banding the exact mode from the
// mismatch count alone was built as well: 41 % fewer block-columns on the token-level
// batch, but with the banded task bodies next to the six full ones the dp kernel no
// longer fits the instruction caches and the launch got slower, not faster.)
//
// Which rollout of a pair is the pattern is fixed by a round-robin tournament on the
// indices, so that every pattern CTA of `prep` serves the same number of texts.
#include "common.cuh"

namespace sr {
namespace {

constexpr int kPrepThreads = 256;
constexpr int kMaxR = 8;            // blocks (32 rows each) per lane
constexpr int kNumClasses = 32;     // team shapes (T lanes x R blocks), see class_of
constexpr int kLenBuckets = 32;     // buckets of estimated task duration
constexpr int kNumBins = kNumClasses * kLenBuckets;
constexpr uint32_t kLocNone = 0x7FFFu;    // bit 15 clear, far above any row: shifts to 0
constexpr uint32_t kLocMulti = 0x8000u;
constexpr uint32_t kChainEnd = 0xFFFFu;
constexpr int kDpWarpsPerCta = 4;
constexpr uint32_t kBinMask = 0x3FFu;
constexpr int32_t kCappedFlag = 0x40000000;   // decide mode: the pair's distance exceeds its cap
constexpr int kStripShift = 12;
constexpr uint32_t kNeedsDp = 0x80000000u;
static_assert(kNumBins <= (int)kBinMask + 1, "bin index must fit its field");

struct PairDesc {          // 16 bytes
    uint32_t mn;           // m | n << 16
    uint32_t pat_row;      // g * N + pattern rollout
    uint32_t bin;          // bits 0..9 bin index; bits 12..21 stripped common prefix (symbols,
                           // a multiple of 4); bit 31 = pair needs the dp kernel
    uint32_t lower;        // bits 0..15 a lower bound of the pair's distance (decide mode),
                           // bits 16..31 an upper bound (mismatching positions + length
                           // difference; in decide mode also capped by what the threshold
                           // still allows): the band of the pair follows from it
};

struct Ctl {               // int32 control block in the workspace
    int32_t hist[kNumBins];
    int32_t start[kNumBins];
    int32_t fill[kNumBins];
    int32_t task_start[kNumBins + 1];          // first warp task of every bin
    int32_t task_counter;
    int32_t total_tasks;
    int32_t task_counter_band;                 // the banded tasks' own launch
};

struct MultiWs {
    size_t off_dist, off_desc, off_loc, off_next, off_order, off_ctl, off_flag, total;
    int pitch;             // uint16 elements per loc / chain row
    int min_tlog;          // small batches: teams of at least 2^min_tlog lanes
};

MultiWs multi_layout(int32_t n_groups, int32_t N, int32_t K) {
    MultiWs w;
    const size_t P = pairs_of(N);
    w.pitch = (K + 7) & ~7;
    w.min_tlog = 0;
    size_t off = 0;
    w.off_ctl = off;   off = align_up(off + sizeof(Ctl), 256);
    w.off_flag = off;  off = align_up(off + (size_t)n_groups, 256);
    w.off_dist = off;  off = align_up(off + (size_t)n_groups * P * 4, 256);
    w.off_desc = off;  off = align_up(off + (size_t)n_groups * P * sizeof(PairDesc), 256);
    w.off_order = off; off = align_up(off + (size_t)n_groups * P * 4, 256);
    w.off_next = off;  off = align_up(off + (size_t)n_groups * N * w.pitch * 2, 256);
    w.off_loc = off;   off = align_up(off + (size_t)n_groups * P * w.pitch * 2, 256);
    w.total = off;
    return w;
}

__host__ __device__ inline void team_shape(int m, int min_tlog, int& tlog, int& R) {
    // T lanes x R blocks per lane >= W blocks of the pattern, with little padding and
    // R large enough to amortise the per-column work that does not depend on R
    const int W = (m + 31) >> 5;            // <= 32
    if (W <= 6) { tlog = 0; R = W; }
    else if (W <= 12) { tlog = 1; R = (W + 1) >> 1; }
    else if (W <= 24) { tlog = 2; R = (W + 3) >> 2; }
    else { tlog = 3; R = (W + 7) >> 3; }
    // A batch with too few pairs to give every resident warp its tasks spreads a pair over
    // more lanes (up to the whole warp): shorter tasks, more of them.
    if (tlog < min_tlog) {
        int t = tlog;
        while (t < min_tlog && (1 << t) < W) ++t;
        tlog = t;
        R = (W + (1 << t) - 1) >> t;
    }
}

// Class of a team shape.  T = 1, 2, 4, 8 with R = 1..6 fill slots log2(T) * 8 + R - 1; the
// shapes of small batches, T = 16 with R = 1, 2 and T = 32 with R = 1, take slots 6, 7, 14;
// the banded shapes (ring of T = 4 or 8 lanes, stripes of R = 1..4 blocks) take slots 15, 22,
// 23, 30, 31.
__host__ __device__ inline int class_of(int tlog, int R) {
    if (tlog < 4) return tlog * 8 + (R - 1);
    return tlog == 4 ? 5 + R : 14;
}
__host__ __device__ inline bool is_band_class(int cls) {
    return cls == 15 || cls == 22 || cls == 23 || cls == 30 || cls == 31;
}
__host__ __device__ inline void shape_of_class(int cls, int& tlog, int& R) {
    if ((cls & 7) < 6) { tlog = cls >> 3; R = (cls & 7) + 1; }
    else if (cls == 6) { tlog = 4; R = 1; }
    else if (cls == 7) { tlog = 4; R = 2; }
    else if (cls == 14) { tlog = 5; R = 1; }
    else if (cls == 15) { tlog = 2; R = 1; }
    else if (cls == 22) { tlog = 3; R = 1; }
    else if (cls == 23) { tlog = 3; R = 2; }
    else if (cls == 30) { tlog = 3; R = 3; }
    else { tlog = 3; R = 4; }               // 31
}

// Bins order the pairs by the estimated running time of their warp task (text
// columns x instructions per column, longest first) and, within one duration
// bucket, by team shape: all pairs of a bin share the shape and have text lengths
// within a few percent, and warps that pull tasks in bin order start the longest
// tasks first, which keeps the finishing times of the warps close together.
__host__ __device__ inline int bin_of_cost(int cost, int cls) {
    const int max_cost = (SR_MAX_K + 32) * (14 * kMaxR + 20) + 1;
    int bucket = (int)(((long long)cost * kLenBuckets) / max_cost);
    bucket = bucket < 0 ? 0 : (bucket >= kLenBuckets ? kLenBuckets - 1 : bucket);
    return (kLenBuckets - 1 - bucket) * kNumClasses + cls;
}

// Diagonals d = row - column an optimal alignment of an m x n pair can visit when its
// distance is at most ub: |d| + |(m - n) - d| <= ub.  At least two diagonals wide, so that
// a stripe always starts while the stripe above it is still running.
__host__ __device__ inline void band_of(int m, int n, int ub, int& dlo, int& dhi) {
    const int D = m - n, aD = D < 0 ? -D : D;
    int e = (ub - aD) >> 1;
    if (e < 0) e = 0;
    dlo = (D < 0 ? D : 0) - e;
    dhi = (D > 0 ? D : 0) + e;
    if (dhi == dlo) ++dhi;
}

// Shape and bin of a pair of m rows x n columns (what is left after the common prefix)
// whose distance is at most ub.  The banded shapes serve bands of up to 32 R (T - 1)
// diagonals; one is taken when its estimated lane-time is clearly below that of the full
// shape (the estimates count instructions per quad of columns and lane).
__host__ __device__ inline int shape_and_bin(int m, int n, int ub, int min_tlog) {
    int tlog, R;
    team_shape(m, min_tlog, tlog, R);
    const int nq = (n + 3) >> 2;
    const int full_time = (nq + (1 << tlog) - 1) * (14 * R + 14);
    const int full_work = full_time << tlog;
    int dlo, dhi;
    band_of(m, n, ub, dlo, dhi);
    const int w = dhi - dlo;
    // banded tasks are few and run with the machine half empty, so their shapes favour a
    // short task (many lanes, few blocks per lane) over the last bit of lane efficiency
    int bcls = -1;
    if (w <= 96) bcls = 15; else if (w <= 224) bcls = 22; else if (w <= 448) bcls = 23;
    else if (w <= 672) bcls = 30; else if (w <= 896) bcls = 31;
    if (bcls >= 0) {
        int btl, bR;
        shape_of_class(bcls, btl, bR);
        const int G = (((m + 31) >> 5) + bR - 1) / bR;      // stripes
        const int band_time = (nq + G - 1) * (14 * bR + 20);
        if ((band_time << btl) * 8 < full_work * 7) return bin_of_cost(4 * band_time, bcls);
    }
    return bin_of_cost(4 * full_time, class_of(tlog, R));
}

__device__ __forceinline__ int clamp_len(const int32_t* lens, size_t idx, int K, bool& neg) {
    int len = lens ? lens[idx] : K;
    if (len < 0) { len = 0; neg = true; }
    return min(len, K);
}

// ------------------------------------------------------------------------ prep
// A slot of the pattern's hash table: symbol in the high word, position of the
// claiming occurrence + 1 in the low word (0 = empty slot), so that one 8-byte
// shared-memory load answers "empty, this symbol, or another symbol".
__device__ __forceinline__ unsigned long long make_slot(int32_t sym, uint32_t pos_plus_1) {
    return ((unsigned long long)(uint32_t)sym << 32) | pos_plus_1;
}

// Position (or chain head) of `sym` in the pattern hashed in shared memory, given the
// content `v` of its home slot `h` (read by the caller, so that the first probes of the
// four look-ups of a quad are in flight together).
__device__ __forceinline__ uint32_t pattern_lookup(int32_t sym, uint32_t h, unsigned long long v,
                                                   const unsigned long long* s_slot,
                                                   const uint32_t* s_next, int hslots) {
    for (int probe = 0; probe < hslots; ++probe) {     // an empty slot always exists
        const uint32_t o = (uint32_t)v;
        if (o == 0u) break;
        if ((int32_t)(v >> 32) == sym) {
            const uint32_t first = o - 1u;
            return s_next[first] == kChainEnd ? first : (kLocMulti | first);
        }
        h = (h + 1u) & (uint32_t)(hslots - 1);
        v = s_slot[h];
    }
    return kLocNone;
}

// kBounds: also count, per text, the columns whose symbol does not occur in the pattern
// at all.  Each of them costs at least one edit, and so does every unit of length
// difference: max(|m - n|, absent columns) is a lower bound of the pair's distance that
// falls out of the look-ups for free.
template <bool kBounds>
__global__ void __launch_bounds__(kPrepThreads, 6)
multi_prep_kernel(GateArgs a, unsigned char* ws, MultiWs W, int hslots_max, int32_t* dist_out, int g_base) {
    extern __shared__ __align__(16) unsigned char smem[];
    unsigned long long* s_slot = reinterpret_cast<unsigned long long*>(smem);    // [hslots_max]
    uint32_t* s_next = reinterpret_cast<uint32_t*>(s_slot + hslots_max);         // [pitch]
    __shared__ int s_txt[SR_MAX_N], s_len[SR_MAX_N], s_qstart[SR_MAX_N + 1], s_absent[SR_MAX_N];
    __shared__ int s_cp[SR_MAX_N], s_differ[SR_MAX_N];
    // (At K = 1024 the 36 KB of dynamic plus these 656 bytes of static shared memory sit just
    // under the size at which six CTAs share an SM: 512 bytes more were measured to cost one
    // CTA per SM and a fifth of the kernel's speed.  Smaller tables with more CTAs per SM are
    // slower too: the probe length matters more than the residency.  Six CTAs of 256 threads
    // leave 40 registers per thread, which the launch bounds grant: capped at 32 the kernel's
    // time jumped by 10 % on changes as small as one more parameter.)

    const int N = a.N, K = a.K, P = pairs_of(N);
    const int g = g_base + blockIdx.x / N, i = blockIdx.x % N;
    const int tid = threadIdx.x;
    const int M = (N & 1) ? N : N - 1;
    if (i >= M) return;                               // the last rollout of an even group is never a pattern
    bool neg = false;
    const int m = clamp_len(a.lens, (size_t)g * N + i, K, neg);
    // the table holds at least four times as many slots as the pattern has symbols:
    // short probe sequences matter more than shared memory here (lanes wait for the
    // longest probe of their warp)
    int hslots = 64;
    while (hslots < 4 * m) hslots <<= 1;
    const int hshift = __clz(hslots) + 1;             // 32 - log2(hslots)
    for (int q = tid; 4 * q < m; q += kPrepThreads)
        reinterpret_cast<uint4*>(s_next)[q] = make_uint4(kChainEnd, kChainEnd, kChainEnd, kChainEnd);
    for (int h = tid; h < hslots; h += kPrepThreads) s_slot[h] = 0ull;
    // The texts this pattern is paired with, one warp per text.  The warp also measures the
    // common prefix of pattern and text (128 positions per trip, stopping at the first
    // mismatch): rollouts of one group start from the same state and often agree on their
    // first symbols, and the edit distance of two sequences equals that of what is left
    // after a common prefix is removed, so those rows and columns are never looked up nor
    // run through the recurrence.
    const int32_t* pat = a.seqs + ((size_t)g * N + i) * a.stride;
    // Which rollout of a pair is the pattern follows a round-robin tournament: with M = N
    // for odd N and N - 1 otherwise, rollout i < M is the pattern against the `half` rollouts
    // after it (cyclically among the first M) and, for even N, against the last rollout,
    // which is a text for everyone.  Every pattern so serves floor(N / 2) texts.  In
    // ascending order the texts of pattern i are: the rollouts more than `half` places
    // before it, the `half` places after it, and the last rollout of an even group.
    const int half = (M - 1) / 2;
    const int n_before = max(0, i - half), n_after = min(i + half, M - 1) - i;
    const int ntxt = n_before + n_after + ((N & 1) ? 0 : 1);
    {
        const int lane = tid & 31;
        for (int t = tid >> 5; t < ntxt; t += kPrepThreads / 32) {
            const int j = t < n_before ? t : (t < n_before + n_after ? i + 1 + (t - n_before) : N - 1);
            bool neg_t = false;
            const int n = clamp_len(a.lens, (size_t)g * N + j, K, neg_t);
            const int32_t* txt = a.seqs + ((size_t)g * N + j) * a.stride;
            const int lo = min(m, n);
            int cp = lo;                              // first mismatch; min(m, n) = none found
            for (int base = 0; base < lo && cp == lo; base += 128) {
                bool ne[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int p = base + 32 * u + lane;
                    ne[u] = p < lo && __ldg(pat + p) != __ldg(txt + p);
                }
#pragma unroll
                for (int u = 3; u >= 0; --u) {
                    const unsigned b = __ballot_sync(0xFFFFFFFFu, ne[u]);
                    if (b) cp = base + 32 * u + __ffs(b) - 1;
                }
            }
            if (lane == 0) {
                s_txt[t] = j;
                s_len[t] = n;
                s_absent[t] = 0;
                s_differ[t] = 0;
                s_cp[t] = cp;
                if (neg_t && a.status) atomicOr(a.status, SR_STATUS_NEG_LEN);
            }
        }
    }
    __syncthreads();
    if (tid == 0) {
        int quads = 0;
        for (int t = 0; t < ntxt; ++t) {
            const int lo = min(m, s_len[t]);
            // the removed prefix is a multiple of four symbols (the match stream is read in
            // 8-byte quads); if one prefix is the start of the other nothing is left to do
            const int strip = s_cp[t] >= lo ? -1 : (s_cp[t] & ~3);
            s_cp[t] = strip;
            s_qstart[t] = quads;
            quads += strip < 0 ? 0 : (s_len[t] - strip + 3) >> 2;
        }
        s_qstart[ntxt] = quads;
    }
    // every position claims the slot of its symbol, or links itself behind the
    // position that claimed it (the claimant heads the symbol's occurrence chain)
    for (int p = tid; p < m; p += kPrepThreads) {
        const int32_t sym = __ldg(pat + p);
        uint32_t h = ((uint32_t)sym * 0x9E3779B1u) >> hshift;
        const unsigned long long mine = make_slot(sym, (uint32_t)p + 1u);
        for (int probe = 0; probe < hslots; ++probe) {
            unsigned long long v = s_slot[h];
            if ((uint32_t)v == 0u) v = atomicCAS(&s_slot[h], 0ull, mine);
            if ((uint32_t)v == 0u) break;
            if ((int32_t)(v >> 32) == sym) {
                s_next[p] = atomicExch(&s_next[(uint32_t)v - 1u], (uint32_t)p);
                break;
            }
            h = (h + 1u) & (uint32_t)(hslots - 1);
        }
    }
    __syncthreads();
    uint16_t* g_next = reinterpret_cast<uint16_t*>(ws + W.off_next) + ((size_t)g * N + i) * W.pitch;
    for (int p = tid; p < m; p += kPrepThreads) g_next[p] = (uint16_t)s_next[p];

    PairDesc* descs = reinterpret_cast<PairDesc*>(ws + W.off_desc);
    uint16_t* locs = reinterpret_cast<uint16_t*>(ws + W.off_loc);
    Ctl* ctl = reinterpret_cast<Ctl*>(ws + W.off_ctl);
    // match streams of all texts, four columns per thread and trip: one 16-byte load
    // of symbols, four independent look-ups, one 8-byte store
    const int total_quads = s_qstart[ntxt];
    for (int item = tid; item < total_quads; item += kPrepThreads) {
        int t = 0;
        while (item >= s_qstart[t + 1]) ++t;
        const int q = (s_cp[t] >> 2) + item - s_qstart[t];      // quad index within the text
        const int j = s_txt[t];
        const int lo = min(i, j), hi = max(i, j);
        const size_t idx = (size_t)g * P + pair_index(lo, hi, N);
        const int4 sym = __ldg(reinterpret_cast<const int4*>(a.seqs + ((size_t)g * N + j) * a.stride) + q);
        const uint32_t h0 = ((uint32_t)sym.x * 0x9E3779B1u) >> hshift, h1 = ((uint32_t)sym.y * 0x9E3779B1u) >> hshift;
        const uint32_t h2 = ((uint32_t)sym.z * 0x9E3779B1u) >> hshift, h3 = ((uint32_t)sym.w * 0x9E3779B1u) >> hshift;
        const unsigned long long v0 = s_slot[h0], v1 = s_slot[h1], v2 = s_slot[h2], v3 = s_slot[h3];
        const uint32_t l0 = pattern_lookup(sym.x, h0, v0, s_slot, s_next, hslots);
        const uint32_t l1 = pattern_lookup(sym.y, h1, v1, s_slot, s_next, hslots);
        const uint32_t l2 = pattern_lookup(sym.z, h2, v2, s_slot, s_next, hslots);
        const uint32_t l3 = pattern_lookup(sym.w, h3, v3, s_slot, s_next, hslots);
        reinterpret_cast<uint2*>(locs + idx * W.pitch)[q] = make_uint2(l0 | (l1 << 16), l2 | (l3 << 16));
        if (kBounds) {
            // positions below both lengths whose symbol is not the pattern's symbol at the same
            // place (a symbol with several occurrences may be counted although it matches: the
            // count only has to be an upper bound of the mismatches)
            const int both = min(m, s_len[t]) - 4 * q;       // columns of this quad below both lengths
            const uint32_t c0 = 4u * (uint32_t)q;
            const int differ = (both > 0 && l0 != c0) + (both > 1 && l1 != c0 + 1u) +
                               (both > 2 && l2 != c0 + 2u) + (both > 3 && l3 != c0 + 3u);
            if (differ) atomicAdd(&s_differ[t], differ);
            const int left = s_len[t] - 4 * q;           // columns of this quad that exist
            const int absent = (l0 == kLocNone) + (left > 1 && l1 == kLocNone) +
                               (left > 2 && l2 == kLocNone) + (left > 3 && l3 == kLocNone);
            if (absent) atomicAdd(&s_absent[t], absent);
        }
    }
    if (kBounds) __syncthreads();
    if (tid < ntxt) {                                 // descriptors, bins, trivial pairs
        const int j = s_txt[tid], n = s_len[tid], strip = s_cp[tid];
        const int lo = min(i, j), hi = max(i, j);
        const size_t idx = (size_t)g * P + pair_index(lo, hi, N);
        if (strip < 0) {                              // one prefix starts the other (or is empty)
            dist_out[idx] = abs(m - n);
            descs[idx] = PairDesc{(uint32_t)m | ((uint32_t)n << 16), (uint32_t)(g * N + i), 0u,
                                  (uint32_t)abs(m - n) | ((uint32_t)abs(m - n) << 16)};
        } else {
            // upper bound: substitute the differing positions, insert / delete the rest (only
            // the decide mode bands its pairs: 0xFFFF stands for "no bound")
            const int upper = kBounds ? s_differ[tid] + abs(m - n) : 0xFFFF;
            const int bin = shape_and_bin(m - strip, n - strip, upper, W.min_tlog);
            const int lower = kBounds ? max(abs(m - n), s_absent[tid]) : 0;
            descs[idx] = PairDesc{(uint32_t)m | ((uint32_t)n << 16), (uint32_t)(g * N + i),
                                  (uint32_t)bin | ((uint32_t)strip << kStripShift) | kNeedsDp,
                                  (uint32_t)lower | ((uint32_t)upper << 16)};
            if (kBounds) dist_out[idx] = lower;            // the bound kernel bins the pairs it keeps
            else atomicAdd(&ctl->hist[bin], 1);
        }
    }
    if (neg && tid == 0 && a.status) atomicOr(a.status, SR_STATUS_NEG_LEN);
}

// ----------------------------------------------------------------------- order
// Exclusive prefix sum over the kNumBins threads of a CTA (one value per thread).
__device__ __forceinline__ int block_exclusive_scan(int v, int* s_part /* [32] */) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) s_part[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = s_part[lane];
        int wi = w;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, wi, d);
            if (lane >= d) wi += up;
        }
        s_part[lane] = wi - w;
    }
    __syncthreads();
    const int r = incl - v + s_part[warp];
    __syncthreads();                       // s_part may be reused at once
    return r;
}

// Counting sort of the pairs by bin: longest warp tasks first, one team shape and similar
// text lengths per bin.  Every CTA turns the bin counts into bin starts by itself (a scan
// of kNumBins values costs less than a launch) and places kNumBins pairs; the first CTA
// also leaves the tables the dp kernel reads.  `fill` is zeroed by the caller's memset.
__global__ void __launch_bounds__(kNumBins)
multi_order_kernel(const PairDesc* descs, int32_t* order, Ctl* ctl, int n_pairs) {
    __shared__ int s_part[32];
    __shared__ int32_t s_start[kNumBins];
    const int t = threadIdx.x;
    const int own = ctl->hist[t];
    const int start = block_exclusive_scan(own, s_part);
    s_start[t] = start;
    if (blockIdx.x == 0) {
        // warp tasks per bin (32 / T pairs per task), exclusive prefix over the bins
        int tl, rr;
        shape_of_class(t % kNumClasses, tl, rr);
        const int tpw = 32 >> tl;
        const int own_tasks = (own + tpw - 1) / tpw;
        const int task_start = block_exclusive_scan(own_tasks, s_part);
        ctl->start[t] = start;
        ctl->task_start[t] = task_start;
        if (t == kNumBins - 1) {
            ctl->task_start[kNumBins] = task_start + own_tasks;
            ctl->total_tasks = task_start + own_tasks;
            ctl->task_counter = 0;
            ctl->task_counter_band = 0;
        }
    }
    __syncthreads();
    const int idx = blockIdx.x * kNumBins + t;
    if (idx >= n_pairs) return;
    const uint32_t b = descs[idx].bin;
    if (!(b & kNeedsDp)) return;
    const int bin = (int)(b & kBinMask);
    order[s_start[bin] + atomicAdd(&ctl->fill[bin], 1)] = idx;
}

// -------------------------------------------------------------------------- dp
__device__ __forceinline__ uint32_t shl_clamp(uint32_t v, uint32_t s) {
    uint32_t r;   // PTX shl clamps shift amounts above 31: the result is 0
    asm("shl.b32 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s));
    return r;
}

// One bit-vector column step over the R blocks a lane owns.  `loc` is the column's
// entry of the match stream, (inP, inM) the pre-shift horizontal delta words of the
// block above (only their top bits matter); returns this lane's last block's words in
// (inP, inM).
template <int R>
__device__ __forceinline__ void column_step(uint32_t loc, uint32_t rowbase, int m,
                                            const uint16_t* __restrict__ nxt,
                                            uint32_t (&Pv)[R], uint32_t (&Mv)[R],
                                            uint32_t& inP, uint32_t& inM, uint32_t two) {
    const uint32_t d0 = loc - rowbase;
    uint32_t Eq[R];
#pragma unroll
    for (int r = 0; r < R; ++r) Eq[r] = shl_clamp(1u, d0 - 32u * r);
    if (loc & kLocMulti) {          // several occurrences in the pattern: walk the chain
        uint32_t p = loc & 0x7FFFu;
        for (int hop = 0; hop < SR_MAX_K && p < (uint32_t)m; ++hop) {   // chain ends at 0xFFFF
            const uint32_t dd = p - rowbase;
#pragma unroll
            for (int r = 0; r < R; ++r) Eq[r] |= shl_clamp(1u, dd - 32u * r);
            p = __ldg(nxt + p);
        }
    }
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t pv = Pv[r], mv = Mv[r];
        const uint32_t hm = inM >> 31;
        const uint32_t Xv = Eq[r] | mv;
        const uint32_t Eh = Eq[r] | hm;
        const uint32_t Xh = (((Eh & pv) + pv) ^ pv) | Eh;
        const uint32_t Ph = mv | ~(Xh | pv);
        const uint32_t Mh = pv & Xh;
        const uint32_t Phs = __funnelshift_l(inP, Ph, 1);
        // `two` holds 2 but is a run-time value, so this shift-and-insert is a multiply-add:
        // it issues on the FMA pipe and leaves the integer ALU, the bottleneck, one
        // instruction lighter per block (measured: 8 % faster than a second funnel shift)
        const uint32_t Mhs = Mh * two + hm;              // (Mh << 1) | hm
        Pv[r] = Mhs | ~(Xv | Phs);
        Mv[r] = Phs & Xv;
        inP = Ph;
        inM = Mh;
    }
}

// A warp task: 32/T teams of T lanes, one pair per team, lane l of a team holding
// rows [32*R*l, 32*R*(l+1)) of the pattern.  Lanes are skewed by one QUAD of text
// columns: in iteration j lane l works on columns 4(j-l) .. 4(j-l)+3.  The four
// columns are unrolled, so (a) a lane fetches its four stream entries with one
// 8-byte load, one iteration ahead, (b) the delta words a lane needs from the lane
// above were produced a whole iteration earlier, so the shuffles never wait, and (c)
// the blocks of consecutive columns overlap in the pipeline.
// (Not inlined on purpose: as eight separate functions the instantiations are
// scheduled independently, which measured 8 % faster than one merged kernel body.)
template <int R>
__device__ __noinline__ void dp_task(int tlog, int pos, bool valid, const PairDesc* descs,
                                        const int32_t* order, const uint16_t* locs,
                                        const uint16_t* nexts, int pitch, int32_t* dist_out,
                                        uint32_t two) {
    const int lane = threadIdx.x & 31;
    const int T = 1 << tlog;
    const int lt = lane & (T - 1);
    // m_all: the whole pattern (bounds the occurrence chains); m, n: rows and columns left
    // after the common prefix of `strip` symbols, which neither side runs through
    int idx = 0, m_all = 0, m = 0, n = 0, strip = 0;
    const uint2* loc4 = reinterpret_cast<const uint2*>(locs);
    const uint16_t* nxt = nexts;
    if (valid) {
        idx = order[pos];
        const PairDesc d = descs[idx];
        strip = (int)((d.bin >> kStripShift) & 0x3FFu);
        m_all = (int)(d.mn & 0xFFFFu);
        m = m_all - strip;
        n = (int)(d.mn >> 16) - strip;
        // rows are 16-byte aligned and strip is a multiple of 4 entries: 8-byte loads
        loc4 = reinterpret_cast<const uint2*>(locs + (size_t)idx * pitch + strip);
        nxt = nexts + (size_t)d.pat_row * pitch;
    }
    const uint32_t rowbase = (uint32_t)(lt * R * 32);
    const uint32_t rowabs = rowbase + (uint32_t)strip;          // first pattern position of this lane
    const int nq = (n + 3) >> 2;                       // quads of text columns
    int iters = valid ? nq + T - 1 : 0;
    iters = __reduce_max_sync(0xFFFFFFFFu, iters);
    const bool top = lt == 0;

    uint32_t Pv[R], Mv[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { Pv[r] = 0xFFFFFFFFu; Mv[r] = 0u; }
    uint32_t outP[4] = {0u, 0u, 0u, 0u}, outM[4] = {0u, 0u, 0u, 0u};
    const uint2 none = make_uint2(kLocNone | (kLocNone << 16), kLocNone | (kLocNone << 16));
    uint2 q_next = (valid && top) ? __ldg(loc4) : none;

    for (int j = 0; j < iters; ++j) {
        const int qi = j - lt;
        const bool active = valid && qi >= 0 && qi < nq;
        const uint2 q = q_next;
        q_next = (valid && qi + 1 >= 0 && qi + 1 < nq) ? __ldg(loc4 + qi + 1) : none;
        // delta words leaving the lane above for this quad (it worked on it last iteration)
        uint32_t inP[4], inM[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            inP[u] = __shfl_up_sync(0xFFFFFFFFu, outP[u], 1);
            inM[u] = __shfl_up_sync(0xFFFFFFFFu, outM[u], 1);
            if (top) { inP[u] = 0x80000000u; inM[u] = 0u; }   // row 0: D[0][c] - D[0][c-1] = +1
        }
        if (active) {
            const int left = n - 4 * qi;               // columns of this quad that exist (>= 1)
            column_step<R>(q.x & 0xFFFFu, rowabs, m_all, nxt, Pv, Mv, inP[0], inM[0], two);
            if (left > 1) column_step<R>(q.x >> 16, rowabs, m_all, nxt, Pv, Mv, inP[1], inM[1], two);
            if (left > 2) column_step<R>(q.y & 0xFFFFu, rowabs, m_all, nxt, Pv, Mv, inP[2], inM[2], two);
            if (left > 3) column_step<R>(q.y >> 16, rowabs, m_all, nxt, Pv, Mv, inP[3], inM[3], two);
#pragma unroll
            for (int u = 0; u < 4; ++u) { outP[u] = inP[u]; outM[u] = inM[u]; }
        }
    }
    // D[m][n] = n + (sum of the vertical deltas of the last column over rows 1..m)
    int part = 0;
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const int rows = min(max(m - (int)(rowbase + 32 * r), 0), 32);
        const uint32_t msk = low_mask(rows);
        part += __popc(Pv[r] & msk) - __popc(Mv[r] & msk);
    }
    for (int off = 1; off < T; off <<= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, off);
    if (valid && top) dist_out[idx] = n + part;
}

// A banded warp task: 32/T teams, one pair per team, the team's T lanes a ring.  The
// pattern's blocks are grouped in stripes of R blocks; stripe g runs on lane g mod T over
// the quads of text columns in which the band crosses it, one iteration behind stripe
// g - 1, exactly like the lanes of the full task; when the band has left a stripe its lane
// takes the stripe T places further down, which starts from +1 vertical deltas below the
// stripe above; a stripe whose upper neighbour the band has left takes +1 horizontal
// deltas from above.  A lane keeps the score at the bottom row of its stripe (started from
// the stripe above plus the +1 deltas it is initialised with, then advanced by the
// horizontal delta that leaves the stripe in every column); the pair's distance is that
// score of the last stripe after the last column, less the vertical deltas of the rows
// beyond the pattern's end.  A result above the pair's bound is reported as bound + 1 with
// kCappedFlag.
template <int R>
__device__ __noinline__ void dp_task_band(int tlog, int pos, bool valid, const PairDesc* descs,
                                             const int32_t* order, const uint16_t* locs,
                                             const uint16_t* nexts, int pitch, int32_t* dist_out,
                                             uint32_t two) {
    const int lane = threadIdx.x & 31;
    const int T = 1 << tlog;
    const int lt = lane & (T - 1);
    const int src = (lane & ~(T - 1)) | ((lt - 1) & (T - 1));      // the lane of the stripe above
    int idx = 0, m_all = 0, m = 0, n = 0, strip = 0, ub = 0;
    const uint2* loc4 = reinterpret_cast<const uint2*>(locs);
    const uint16_t* nxt = nexts;
    if (valid) {
        idx = order[pos];
        const PairDesc d = descs[idx];
        strip = (int)((d.bin >> kStripShift) & 0x3FFu);
        m_all = (int)(d.mn & 0xFFFFu);
        m = m_all - strip;
        n = (int)(d.mn >> 16) - strip;
        ub = (int)(d.lower >> 16);
        loc4 = reinterpret_cast<const uint2*>(locs + (size_t)idx * pitch + strip);
        nxt = nexts + (size_t)d.pat_row * pitch;
    }
    int dlo, dhi;
    band_of(m, n, ub, dlo, dhi);
    const int nq = (n + 3) >> 2;                       // quads of text columns
    const int G = valid ? (((m + 31) >> 5) + R - 1) / R : 0;       // stripes
    int iters = valid ? nq + G - 1 : 0;
    iters = __reduce_max_sync(0xFFFFFFFFu, iters);
    // quads in which the band crosses stripe g: columns 32 R g - dhi .. 32 R (g + 1) - 1 - dlo
    auto first_quad = [&](int g) { const int c = 32 * R * g - dhi; return c <= 0 ? 0 : c >> 2; };
    auto last_quad = [&](int g) { return min((32 * R * (g + 1) - 1 - dlo) >> 2, nq - 1); };

    int g = lt;                                        // the stripe this lane holds
    int js = 0x7FFFFFFF, je = -1, above_end = -1;      // its iterations; last quad of the stripe above
    if (g < G) {
        js = first_quad(g) + g;
        je = last_quad(g) + g;
        above_end = g > 0 ? last_quad(g - 1) : -1;
    }
    uint32_t Pv[R], Mv[R];
#pragma unroll
    for (int r = 0; r < R; ++r) { Pv[r] = 0xFFFFFFFFu; Mv[r] = 0u; }
    uint32_t outP[4] = {0u, 0u, 0u, 0u}, outM[4] = {0u, 0u, 0u, 0u};
    uint32_t up = 0u, down = 0u;                       // +1 / -1 horizontal deltas seen at the stripe's bottom
    int base = 0, before = 0;                          // score = base + up - down; score before the last quad
    const uint2 none = make_uint2(kLocNone | (kLocNone << 16), kLocNone | (kLocNone << 16));
    uint2 q_next = none;

    for (int j = 0; j < iters; ++j) {
        // delta words and score of the stripe above, as its lane left them one iteration ago
        uint32_t inP[4], inM[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            inP[u] = __shfl_sync(0xFFFFFFFFu, outP[u], src);
            inM[u] = __shfl_sync(0xFFFFFFFFu, outM[u], src);
        }
        const int above_before = __shfl_sync(0xFFFFFFFFu, before, src);
        if (j > je && g < G) {                         // the band has left this stripe: take the next one
            g += T;
            if (g < G) {
                js = first_quad(g) + g;
                je = last_quad(g) + g;
                above_end = last_quad(g - 1);
#pragma unroll
                for (int r = 0; r < R; ++r) { Pv[r] = 0xFFFFFFFFu; Mv[r] = 0u; }
            } else {
                js = 0x7FFFFFFF;
                je = -1;
            }
        }
        if (j >= js && j <= je) {
            const int qi = j - g;
            uint2 q = q_next;
            if (j == js) {
                // first quad of the stripe: the rows start one apart below the stripe above
                // (or below the matrix's first column)
                q = __ldg(loc4 + qi);
                base = qi > 0 ? above_before + 32 * R : 32 * R * (g + 1);
                up = 0u;
                down = 0u;
            }
            if (g == 0 || qi > above_end) {            // nothing above: row 0, or the band left it
#pragma unroll
                for (int u = 0; u < 4; ++u) { inP[u] = 0x80000000u; inM[u] = 0u; }
            }
            before = base + (int)up - (int)down;
            const uint32_t rowabs = (uint32_t)(strip + 32 * R * g);
            const int left = n - 4 * qi;               // columns of this quad that exist (>= 1)
            column_step<R>(q.x & 0xFFFFu, rowabs, m_all, nxt, Pv, Mv, inP[0], inM[0], two);
            up = __umulhi(inP[0], two) + up;           // top bit of the word: the delta leaving the stripe
            down = __umulhi(inM[0], two) + down;
            if (left > 1) {
                column_step<R>(q.x >> 16, rowabs, m_all, nxt, Pv, Mv, inP[1], inM[1], two);
                up = __umulhi(inP[1], two) + up;
                down = __umulhi(inM[1], two) + down;
            }
            if (left > 2) {
                column_step<R>(q.y & 0xFFFFu, rowabs, m_all, nxt, Pv, Mv, inP[2], inM[2], two);
                up = __umulhi(inP[2], two) + up;
                down = __umulhi(inM[2], two) + down;
            }
            if (left > 3) {
                column_step<R>(q.y >> 16, rowabs, m_all, nxt, Pv, Mv, inP[3], inM[3], two);
                up = __umulhi(inP[3], two) + up;
                down = __umulhi(inM[3], two) + down;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) { outP[u] = inP[u]; outM[u] = inM[u]; }
            if (g == G - 1 && qi == nq - 1) {
                // the score at the stripe's bottom row, less the vertical deltas of the rows
                // past the pattern's end
                int d = base + (int)up - (int)down;
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    const int rows = min(max(m - 32 * (R * g + r), 0), 32);
                    const uint32_t past = ~low_mask(rows);
                    d -= __popc(Pv[r] & past) - __popc(Mv[r] & past);
                }
                dist_out[idx] = d > ub ? ((ub + 1) | kCappedFlag) : d;
            }
        }
        q_next = (j + 1 > js && j + 1 <= je) ? __ldg(loc4 + (j + 1 - g)) : none;
    }
}

// Persistent warps pull warp tasks, longest first, from the bins' task list.  kBoth: the
// batch has banded tasks as well (decide mode); CTAs with an odd index then serve those,
// from a task counter of their own, and the even CTAs the full tasks, so that the two
// kinds -- neither of which fills the machine -- run side by side.
template <bool kBoth>
__global__ void __launch_bounds__(kDpWarpsPerCta * 32)
multi_dp_kernel(unsigned char* ws, MultiWs W, int32_t* dist_out, uint32_t two) {
    const bool kBand = kBoth && (blockIdx.x & 1);
    Ctl* ctl = reinterpret_cast<Ctl*>(ws + W.off_ctl);
    const PairDesc* descs = reinterpret_cast<const PairDesc*>(ws + W.off_desc);
    const int32_t* order = reinterpret_cast<const int32_t*>(ws + W.off_order);
    const uint16_t* locs = reinterpret_cast<const uint16_t*>(ws + W.off_loc);
    const uint16_t* nexts = reinterpret_cast<const uint16_t*>(ws + W.off_next);
    const int lane = threadIdx.x & 31;
    const int total = ctl->total_tasks;
    int32_t* counter = kBand ? &ctl->task_counter_band : &ctl->task_counter;
    while (true) {
        int task = 0;
        if (lane == 0) task = atomicAdd(counter, 1);
        task = __shfl_sync(0xFFFFFFFFu, task, 0);
        if (task >= total) break;
        int k = 0, hi = kNumBins;                     // last bin whose first task is <= task
        while (hi - k > 1) {
            const int mid = (k + hi) >> 1;
            if (ctl->task_start[mid] <= task) k = mid; else hi = mid;
        }
        if (is_band_class(k % kNumClasses) != kBand) continue;
        int tlog, R;
        shape_of_class(k % kNumClasses, tlog, R);
        const int tpw = 32 >> tlog;
        const int pos = ctl->start[k] + (task - ctl->task_start[k]) * tpw + (lane >> tlog);
        const bool valid = pos < ctl->start[k] + ctl->fill[k];     // fill = pairs in the bin
        if (kBand) {
            switch (R) {
                case 1: dp_task_band<1>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 2: dp_task_band<2>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 3: dp_task_band<3>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                default: dp_task_band<4>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
            }
        } else {
            switch (R) {
                case 1: dp_task<1>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 2: dp_task<2>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 3: dp_task<3>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 4: dp_task<4>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                case 5: dp_task<5>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
                default: dp_task<6>(tlog, pos, valid, descs, order, locs, nexts, W.pitch, dist_out, two); break;
            }
        }
    }
}

// ----------------------------------------------------------------------- bound
// Decide mode.  Per group, d_K evaluated on the pairs' lower bounds, in the same order
// and arithmetic as the real thing: every term is <= the true term and rounded addition
// is monotone, so the result is <= the true d_K.  If it is already not below the
// threshold, the gate's answer is "continue" whatever the exact distances are: the
// group is finished here and its pairs never reach the bit-vector kernel.
// A group the bounds leave open still has a budget: with every other pair at its lower
// bound, pair p can only keep d_K below the threshold while its distance stays at or below
//     cap_p = L_p * (P * d_L - sum of the other pairs' bounded terms)
// (L_p the longer prefix, 1 for raw distances).  The pair's band is cut to that cap (plus a
// margin of two that swamps the rounding of this estimate); a pair whose banded result
// exceeds its cap is reported as "more than the cap", which is all Eq. 2 needs to know.
__global__ void __launch_bounds__(128)
multi_bound_kernel(GateArgs a, PairDesc* descs, Ctl* ctl, uint8_t* flag, uint8_t* exact, int min_tlog) {
    const int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= a.n_groups) return;
    const int N = a.N, P = pairs_of(N);
    PairDesc* d = descs + (size_t)g * P;
    double s = 0.0;
    int isum = 0;
    for (int p = 0; p < P; ++p) {
        const int m = (int)(d[p].mn & 0xFFFFu), n = (int)(d[p].mn >> 16);
        const int lb = (int)(d[p].lower & 0xFFFFu);
        isum += lb;
        s = __dadd_rn(s, pair_term(lb, m, n, a.norm_mode));      // max(m, n) is symmetric in the roles
    }
    const double dk = __ddiv_rn(s, (double)P);
    const bool open = dk < a.threshold;                  // the bound alone cannot decide
    flag[g] = open ? 1 : 0;
    if (exact) exact[g] = open ? 1 : 0;
    if (open) {
        const double budget = (double)P * a.threshold;
        for (int p = 0; p < P; ++p) {
            if (!(d[p].bin & kNeedsDp)) continue;
            const int m = (int)(d[p].mn & 0xFFFFu), n = (int)(d[p].mn >> 16);
            const int lb = (int)(d[p].lower & 0xFFFFu);
            int ub = (int)(d[p].lower >> 16);
            const double longer = a.norm_mode == SR_NORM_NONE ? 1.0 : (double)max(m, n);
            const double room = (budget - (s - pair_term(lb, m, n, a.norm_mode))) * longer;
            // room < 2^31 here: an open group has s < budget, so room <= (budget + term) * longer
            const int cap = max(lb, (int)fmin(room, 1.0e9)) + 2;
            ub = min(ub, cap);
            const int strip = (int)((d[p].bin >> kStripShift) & 0x3FFu);
            const int bin = shape_and_bin(m - strip, n - strip, ub, min_tlog);
            d[p].bin = (uint32_t)bin | ((uint32_t)strip << kStripShift) | kNeedsDp;
            d[p].lower = (uint32_t)lb | ((uint32_t)ub << 16);
            atomicAdd(&ctl->hist[bin], 1);
        }
    } else {
        for (int p = 0; p < P; ++p) d[p].bin &= ~kNeedsDp;
        if (a.pair_sum) a.pair_sum[g] = isum;
        if (a.mean) a.mean[g] = dk;
        a.stop[g] = 0;
    }
}

// ---------------------------------------------------------------------- finish
// One thread per pair turns its distance into a term of d_K (the loads and divisions of a
// group run side by side); one thread per group then adds the terms in pair order.
constexpr int kFinishThreads = 256;

__global__ void __launch_bounds__(kFinishThreads)
multi_finish_kernel(GateArgs a, int32_t* dist, const uint8_t* flag, uint8_t* exact, int gpb) {
    __shared__ double s_term[kFinishThreads];
    __shared__ int32_t s_dist[kFinishThreads];
    const int N = a.N, P = pairs_of(N);
    const int tid = threadIdx.x;
    const int g0 = blockIdx.x * gpb;
    const int ng = min(gpb, a.n_groups - g0);
    if (P <= kFinishThreads) {
        if (tid < ng * P) {
            const int g = tid / P, p = tid - g * P;
            int i, j;
            pair_from_index(p, N, i, j);
            bool neg = false;
            const int mi = clamp_len(a.lens, (size_t)(g0 + g) * N + i, a.K, neg);
            const int mj = clamp_len(a.lens, (size_t)(g0 + g) * N + j, a.K, neg);
            // decide mode marks a distance beyond its pair's cap: the value is then a lower bound
            const int raw = dist[(size_t)g0 * P + tid];
            const int d = raw & ~kCappedFlag;
            if (raw != d) dist[(size_t)g0 * P + tid] = d;
            s_dist[tid] = raw;
            s_term[tid] = pair_term(d, mi, mj, a.norm_mode);
        }
        __syncthreads();
        if (tid < ng) {
            const int g = g0 + tid;
            if (flag && flag[g] == 0) return;                // decided from the bounds
            double s = 0.0;
            int isum = 0, capped = 0;
            for (int p = 0; p < P; ++p) {
                s = __dadd_rn(s, s_term[tid * P + p]);
                isum += s_dist[tid * P + p] & ~kCappedFlag;
                capped |= s_dist[tid * P + p] & kCappedFlag;
            }
            const double dk = __ddiv_rn(s, (double)P);
            if (a.pair_sum) a.pair_sum[g] = isum;
            if (a.mean) a.mean[g] = dk;
            a.stop[g] = dk < a.threshold ? 1 : 0;
            if (capped && exact) exact[g] = 0;          // some distances are lower bounds
        }
        return;
    }
    // groups of more than 23 rollouts (more pairs than threads): one thread per group
    if (tid != 0) return;
    const int g = g0;
    if (flag && flag[g] == 0) return;
    bool neg = false;
    double s = 0.0;
    int isum = 0, p = 0, capped = 0;
    for (int i = 0; i < N; ++i) {
        const int mi = clamp_len(a.lens, (size_t)g * N + i, a.K, neg);
        for (int j = i + 1; j < N; ++j, ++p) {
            const int mj = clamp_len(a.lens, (size_t)g * N + j, a.K, neg);
            const int raw = dist[(size_t)g * P + p];
            const int d = raw & ~kCappedFlag;
            if (raw != d) dist[(size_t)g * P + p] = d;
            capped |= raw & kCappedFlag;
            isum += d;
            s = __dadd_rn(s, pair_term(d, mi, mj, a.norm_mode));
        }
    }
    const double dk = __ddiv_rn(s, (double)P);
    if (a.pair_sum) a.pair_sum[g] = isum;
    if (a.mean) a.mean[g] = dk;
    a.stop[g] = dk < a.threshold ? 1 : 0;
    if (capped && exact) exact[g] = 0;
}

}  // namespace

size_t gate_multi_workspace_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    (void)stride;
    return multi_layout(n_groups, N, K).total;
}

int launch_gate_multi(const GateArgs& a, void* ws_, size_t ws_bytes, cudaStream_t s,
                      const cudaEvent_t* ev, bool decide, uint8_t* exact, const GroupFeed* feed) {
    if (a.n_groups == 0) return SR_OK;
    MultiWs W = multi_layout(a.n_groups, a.N, a.K);
    if (ws_ == nullptr || ws_bytes < W.total || (reinterpret_cast<uintptr_t>(ws_) & 255) != 0)
        return SR_ERR_WORKSPACE;
    unsigned char* ws = static_cast<unsigned char*>(ws_);
    const int P = pairs_of(a.N);
    const long long n_pairs_ll = (long long)a.n_groups * P;
    if (n_pairs_ll > 0x7FFFFFFFLL) return SR_ERR_BAD_N;
    int dev = 0, sms = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    SR_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    // fewer than two pairs per resident warp (12 warps per SM): widen the teams until there
    // are about eight lanes' worth of pairs per warp (measured on token-level batches of 16 to
    // 256 groups: -40 % at 16 groups, -22 % at 64, nothing to gain from 128 on)
    const long long warps = 12LL * sms;
    if (n_pairs_ll < 2 * warps)
        while (W.min_tlog < 5 && (n_pairs_ll << W.min_tlog) < 8 * warps) ++W.min_tlog;
    // decide mode: what is left after the bounds is little work in a few long tasks, so the
    // launch lasts as long as its longest pair: spread every pair over as many lanes as it
    // has blocks (up to the whole warp), which shortens that pair fourfold
    if (decide) W.min_tlog = 5;
    const int n_pairs = (int)n_pairs_ll;
    int32_t* dist = a.pair_dist ? a.pair_dist : reinterpret_cast<int32_t*>(ws + W.off_dist);
    Ctl* ctl = reinterpret_cast<Ctl*>(ws + W.off_ctl);

    int hslots = 64;
    while (hslots < 4 * a.K) hslots <<= 1;
    const int prep_smem = hslots * 8 + W.pitch * 4;

    if (ev) SR_CUDA_TRY(cudaEventRecord(ev[0], s));
    // bin counts (filled by prep) and fill counters (used by the ordering kernel) start at zero
    static_assert(offsetof(Ctl, fill) + sizeof(Ctl::fill) == 3 * kNumBins * sizeof(int32_t), "hist, start, fill lead Ctl");
    SR_CUDA_TRY(cudaMemsetAsync(ctl, 0, 3 * kNumBins * sizeof(int32_t), s));
    uint8_t* flag = decide ? ws + W.off_flag : nullptr;
    // The match-stream pass works group by group, so when the groups arrive in pieces it runs
    // piece by piece: `feed->before` enqueues whatever makes groups [g0, g1) ready on `s`.
    const int pieces = feed ? feed->pieces : 1;
    for (int c = 0; c < pieces; ++c) {
        const int g0 = (int)((long long)a.n_groups * c / pieces);
        const int g1 = (int)((long long)a.n_groups * (c + 1) / pieces);
        if (g1 == g0) continue;
        if (feed) {
            const int rc = feed->before(feed->ctx, g0, g1, s);
            if (rc != SR_OK) return rc;
        }
        if (decide)
            multi_prep_kernel<true><<<(g1 - g0) * a.N, kPrepThreads, prep_smem, s>>>(a, ws, W, hslots, dist, g0);
        else
            multi_prep_kernel<false><<<(g1 - g0) * a.N, kPrepThreads, prep_smem, s>>>(a, ws, W, hslots, dist, g0);
        SR_LAUNCH_CHECK("multi_prep_kernel");
    }
    if (decide) {
        multi_bound_kernel<<<(a.n_groups + 127) / 128, 128, 0, s>>>(
            a, reinterpret_cast<PairDesc*>(ws + W.off_desc), ctl, flag, exact, W.min_tlog);
        SR_LAUNCH_CHECK("multi_bound_kernel");
    }
    if (ev) SR_CUDA_TRY(cudaEventRecord(ev[1], s));
    multi_order_kernel<<<(n_pairs + kNumBins - 1) / kNumBins, kNumBins, 0, s>>>(
        reinterpret_cast<const PairDesc*>(ws + W.off_desc),
        reinterpret_cast<int32_t*>(ws + W.off_order), ctl, n_pairs);
    SR_LAUNCH_CHECK("multi_order_kernel");
    if (ev) SR_CUDA_TRY(cudaEventRecord(ev[2], s));
    // persistent grid: a multiple of the SM count; warps pull tasks until none is left
    long long want = (n_pairs_ll + kDpWarpsPerCta - 1) / kDpWarpsPerCta;
    // 3 CTAs of 4 warps per SM (3 warps per scheduler): enough to keep the integer pipe
    // busy, few enough that most tasks are pulled dynamically, longest first (measured
    // best among 2..6 warps per scheduler)
    long long cap = (long long)sms * 3;
    int blocks = (int)(want < cap ? want : cap);
    if (blocks < 1) blocks = 1;
    if (decide) multi_dp_kernel<true><<<2 * blocks, kDpWarpsPerCta * 32, 0, s>>>(ws, W, dist, 2u);
    else multi_dp_kernel<false><<<blocks, kDpWarpsPerCta * 32, 0, s>>>(ws, W, dist, 2u);
    SR_LAUNCH_CHECK("multi_dp_kernel");
    if (ev) SR_CUDA_TRY(cudaEventRecord(ev[3], s));
    const int fin_gpb = P <= kFinishThreads ? kFinishThreads / P : 1;
    multi_finish_kernel<<<(a.n_groups + fin_gpb - 1) / fin_gpb, kFinishThreads, 0, s>>>(a, dist, flag, exact, fin_gpb);
    SR_LAUNCH_CHECK("multi_finish_kernel");
    if (ev) SR_CUDA_TRY(cudaEventRecord(ev[4], s));
    return SR_OK;
}

}  // namespace sr
