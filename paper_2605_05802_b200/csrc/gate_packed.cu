// sr_gate_host_packed: the gate on HOST input in packed (ragged) form.  Rollout prefixes
// of very different lengths (token-level gates) waste a third or more of a padded
// [rows][stride] array, and over a host link the copy, not the kernels, sets the time of
// a call; here only the symbols that exist cross the link.  On the device a small kernel
// spreads them into the padded rows the gate kernels read.
#include "common.cuh"

namespace sr {
namespace {

constexpr int kUnpackThreads = 256;

// One warp per row: row r of the chunk holds symbols [start[r], start[r + 1]) of `packed`
// (indices relative to packed[0] of the whole batch); the first min(len, stride) of them
// go to the row's padded slot, the full length to lens.
__global__ void __launch_bounds__(kUnpackThreads)
unpack_rows_kernel(const int32_t* __restrict__ packed, const long long* __restrict__ start,
                   int rows, int stride, int32_t* __restrict__ seqs, int32_t* __restrict__ lens) {
    const int row = blockIdx.x * (kUnpackThreads / 32) + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int lane = threadIdx.x & 31;
    const long long b = start[row], e = start[row + 1];
    const long long len = e - b;
    const int n = (int)(len < (long long)stride ? len : (long long)stride);
    const int32_t* src = packed + b;
    int32_t* dst = seqs + (size_t)row * stride;
    for (int t = lane; t < n; t += 32) dst[t] = __ldg(src + t);
    if (lane == 0) lens[row] = (int)(len < 0x7FFFFFFFLL ? len : 0x7FFFFFFFLL);
}

// What the pieces of a chunked transfer need on the kernels' stream: wait for the piece's
// copy, then spread its rows.
struct FeedCtx {
    const int32_t* d_packed;
    const long long* d_start;
    int32_t* d_seqs;
    int32_t* d_lens;
    int N, stride;
    cudaEvent_t* copied;      // one event per piece, recorded on the copy stream
    int pieces, n_groups;
};

int unpack_rows(const FeedCtx& f, int g0, int g1, cudaStream_t s) {
    const size_t row0 = (size_t)g0 * f.N;
    const int rows = (g1 - g0) * f.N;
    unpack_rows_kernel<<<(rows + kUnpackThreads / 32 - 1) / (kUnpackThreads / 32), kUnpackThreads, 0, s>>>(
        f.d_packed, f.d_start + row0, rows, f.stride, f.d_seqs + row0 * f.stride, f.d_lens + row0);
    SR_LAUNCH_CHECK("unpack_rows_kernel");
    return SR_OK;
}

int feed_piece(void* ctx, int g0, int g1, cudaStream_t s) {
    const FeedCtx& f = *static_cast<const FeedCtx*>(ctx);
    // the piece index follows from g0 the same way the pipeline cut the groups
    int c = 0;
    while (c + 1 < f.pieces && (int)((long long)f.n_groups * (c + 1) / f.pieces) <= g0) ++c;
    SR_CUDA_TRY(cudaStreamWaitEvent(s, f.copied[c], 0));
    return unpack_rows(f, g0, g1, s);
}

// Events of one call; destroyed when the call returns, whichever way (an event that is
// still pending is released by the driver once it has completed).
struct EventSet {
    cudaEvent_t ev[8];
    int n = 0;
    cudaError_t add() {
        const cudaError_t e = cudaEventCreateWithFlags(&ev[n], cudaEventDisableTiming);
        if (e == cudaSuccess) ++n;
        return e;
    }
    ~EventSet() { for (int k = 0; k < n; ++k) cudaEventDestroy(ev[k]); }
};

struct PackedArena {
    size_t off_packed, off_start, inner, total;     // `inner`: where the padded-input arena begins
};

PackedArena packed_arena(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    PackedArena p;
    size_t off = 0;
    p.off_packed = off; off = align_up(off + (size_t)n_groups * N * stride * 4, 256);
    p.off_start = off;  off = align_up(off + ((size_t)n_groups * N + 1) * 8, 256);
    p.inner = off;
    p.total = off + host_arena(n_groups, N, stride, K).total;
    return p;
}

}  // namespace
}  // namespace sr

using namespace sr;

extern "C" {

size_t sr_gate_host_packed_arena_bytes(int32_t n_groups, int32_t N, int32_t stride, int32_t K) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N || stride < 0 || (stride & 3) || K < 0 || K > stride ||
        K > SR_MAX_K)
        return 0;
    return packed_arena(n_groups, N, stride, K).total;
}

int sr_gate_host_packed(const int32_t* symbols, const int64_t* row_start, int32_t n_groups, int32_t N,
                        int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                        int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                        int32_t* status, void* arena, size_t arena_bytes, void* stream,
                        void* copy_stream) {
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (stride < 0 || (stride & 3) || K < 0 || K > stride || K > SR_MAX_K) return SR_ERR_BAD_K;
    if (norm_mode != SR_NORM_MAXLEN && norm_mode != SR_NORM_NONE) return SR_ERR_BAD_MODE;
    if (n_groups == 0) return SR_OK;
    if (row_start == nullptr || stop == nullptr) return SR_ERR_NULL;
    const size_t rows = (size_t)n_groups * N;
    // the offsets are host memory: checked here, before anything is enqueued
    if (row_start[0] != 0) return SR_ERR_BAD_OFFSETS;
    for (size_t r = 0; r < rows; ++r)
        if (row_start[r + 1] < row_start[r]) return SR_ERR_BAD_OFFSETS;
    const long long total = row_start[rows];
    if (total > 0 && symbols == nullptr) return SR_ERR_NULL;
    // a row longer than `stride` is legal (only its first K <= stride symbols matter), but the
    // packed staging area is sized for rows * stride symbols
    if ((unsigned long long)total > (unsigned long long)rows * (unsigned long long)stride)
        return SR_ERR_BAD_OFFSETS;
    const PackedArena pa = packed_arena(n_groups, N, stride, K);
    if (arena == nullptr || arena_bytes < pa.total || (reinterpret_cast<uintptr_t>(arena) & 255) != 0)
        return SR_ERR_WORKSPACE;
    unsigned char* d = static_cast<unsigned char*>(arena);
    unsigned char* di = d + pa.inner;
    const HostArena h = host_arena(n_groups, N, stride, K);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t P = pairs_of(N);
    int32_t* d_packed = reinterpret_cast<int32_t*>(d + pa.off_packed);
    long long* d_start = reinterpret_cast<long long*>(d + pa.off_start);
    int32_t* d_seqs = reinterpret_cast<int32_t*>(di + h.off_seqs);
    int32_t* d_lens = reinterpret_cast<int32_t*>(di + h.off_lens);
    GateArgs ga{d_seqs, d_lens, n_groups, N, stride, K, threshold, norm_mode,
                pair_dist ? reinterpret_cast<int32_t*>(di + h.off_dist) : nullptr,
                pair_sum ? reinterpret_cast<int32_t*>(di + h.off_sum) : nullptr,
                mean ? reinterpret_cast<double*>(di + h.off_mean) : nullptr,
                di + h.off_stop, status ? reinterpret_cast<int32_t*>(di + h.off_status) : nullptr};
    FeedCtx f{d_packed, d_start, d_seqs, d_lens, N, stride, nullptr, 1, n_groups};
    if (status) SR_CUDA_TRY(cudaMemcpyAsync(di + h.off_status, status, 4, cudaMemcpyHostToDevice, s));
    cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
    // With a copy stream and long prefixes the symbols go over in four pieces of whole groups
    // and the per-group pass of the gate (match streams) runs on each piece while the next one
    // is still on the link; the recurrence then runs ONCE over the whole batch.  Cutting the
    // whole gate into pieces was measured and lost: the kernels of a quarter of a token-level
    // batch take almost as long as those of the whole batch, because a few long pairs set the
    // time of the recurrence launch.
    if (cs != nullptr && cs != s && K > 32 && n_groups >= 64) {
        constexpr int kPieces = 4;
        EventSet events;                                  // [0] fork, [1 + c] piece c copied
        for (int k = 0; k < 1 + kPieces; ++k) SR_CUDA_TRY(events.add());
        // the copies must not overtake earlier work on `stream` that uses the arena
        SR_CUDA_TRY(cudaEventRecord(events.ev[0], s));
        SR_CUDA_TRY(cudaStreamWaitEvent(cs, events.ev[0], 0));
        SR_CUDA_TRY(cudaMemcpyAsync(d_start, row_start, (rows + 1) * 8, cudaMemcpyHostToDevice, cs));
        for (int c = 0; c < kPieces; ++c) {
            const size_t row0 = (size_t)((long long)n_groups * c / kPieces) * N;
            const size_t row1 = (size_t)((long long)n_groups * (c + 1) / kPieces) * N;
            const long long s0 = row_start[row0], s1 = row_start[row1];
            if (s1 > s0)
                SR_CUDA_TRY(cudaMemcpyAsync(d_packed + s0, symbols + s0, (size_t)(s1 - s0) * 4,
                                            cudaMemcpyHostToDevice, cs));
            SR_CUDA_TRY(cudaEventRecord(events.ev[1 + c], cs));
        }
        f.copied = events.ev + 1;
        f.pieces = kPieces;
        const GroupFeed feed{kPieces, feed_piece, &f};
        const int rc = launch_gate_multi(ga, di + h.off_ws, h.total - h.off_ws, s, nullptr, false, nullptr, &feed);
        if (rc != SR_OK) return rc;
    } else {
        SR_CUDA_TRY(cudaMemcpyAsync(d_start, row_start, (rows + 1) * 8, cudaMemcpyHostToDevice, s));
        if (total > 0)
            SR_CUDA_TRY(cudaMemcpyAsync(d_packed, symbols, (size_t)total * 4, cudaMemcpyHostToDevice, s));
        int rc = unpack_rows(f, 0, n_groups, s);
        if (rc != SR_OK) return rc;
        rc = sr_gate(ga.seqs, ga.lens, n_groups, N, stride, K, threshold, norm_mode, ga.pair_dist,
                     ga.pair_sum, ga.mean, ga.stop, ga.status, di + h.off_ws, h.total - h.off_ws, stream);
        if (rc != SR_OK) return rc;
    }
    if (pair_dist)
        SR_CUDA_TRY(cudaMemcpyAsync(pair_dist, di + h.off_dist, (size_t)n_groups * P * 4,
                                    cudaMemcpyDeviceToHost, s));
    if (pair_sum)
        SR_CUDA_TRY(cudaMemcpyAsync(pair_sum, di + h.off_sum, (size_t)n_groups * 4, cudaMemcpyDeviceToHost, s));
    if (mean)
        SR_CUDA_TRY(cudaMemcpyAsync(mean, di + h.off_mean, (size_t)n_groups * 8, cudaMemcpyDeviceToHost, s));
    SR_CUDA_TRY(cudaMemcpyAsync(stop, di + h.off_stop, (size_t)n_groups, cudaMemcpyDeviceToHost, s));
    if (status)
        SR_CUDA_TRY(cudaMemcpyAsync(status, di + h.off_status, 4, cudaMemcpyDeviceToHost, s));
    return SR_OK;
}

}  // extern "C"
