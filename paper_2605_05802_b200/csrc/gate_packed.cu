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
                        int32_t* status, void* arena, size_t arena_bytes, void* stream) {
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
    // The batch goes over in one piece.  Sending it in chunks whose kernels overlap the next
    // chunk's copy was measured and lost: the kernels of a quarter of a token-level batch take
    // almost as long as those of the whole batch (a few long pairs set the time of the
    // recurrence launch), far longer than the quarter's copy.
    if (status) SR_CUDA_TRY(cudaMemcpyAsync(di + h.off_status, status, 4, cudaMemcpyHostToDevice, s));
    SR_CUDA_TRY(cudaMemcpyAsync(d_start, row_start, (rows + 1) * 8, cudaMemcpyHostToDevice, s));
    if (total > 0)
        SR_CUDA_TRY(cudaMemcpyAsync(d_packed, symbols, (size_t)total * 4, cudaMemcpyHostToDevice, s));
    unpack_rows_kernel<<<(int)((rows + kUnpackThreads / 32 - 1) / (kUnpackThreads / 32)), kUnpackThreads, 0, s>>>(
        d_packed, d_start, (int)rows, stride, d_seqs, d_lens);
    SR_LAUNCH_CHECK("unpack_rows_kernel");
    const int rc = sr_gate(d_seqs, d_lens, n_groups, N, stride, K, threshold, norm_mode,
                           pair_dist ? reinterpret_cast<int32_t*>(di + h.off_dist) : nullptr,
                           pair_sum ? reinterpret_cast<int32_t*>(di + h.off_sum) : nullptr,
                           mean ? reinterpret_cast<double*>(di + h.off_mean) : nullptr,
                           di + h.off_stop, status ? reinterpret_cast<int32_t*>(di + h.off_status) : nullptr,
                           di + h.off_ws, h.total - h.off_ws, stream);
    if (rc != SR_OK) return rc;
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
