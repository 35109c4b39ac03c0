// Kept-group index list: the ascending indices of the groups that stay in the training
// batch after the gate (Appendix C.1: a cut group is skipped) and, optionally, after the
// zero-variance filter of the dynamic-sampling baseline (a group whose advantages are all
// zero adds nothing to the gradient, Section 2.1).
//
// Stream compaction in three launches, no waiting between blocks: every CTA counts the
// kept groups of its tile of 4096 groups; one CTA turns the tile counts into tile offsets;
// every CTA recomputes its tile's flags (they come from L2 the second time), scans them,
// collects its indices in shared memory and writes them out as one contiguous run.  The
// order is ascending by construction, whatever the scheduling.
#include "common.cuh"

namespace sr {
namespace {

constexpr int kTileThreads = 256;
constexpr int kPerThread = 16;                       // one 16-byte load of flags per thread
constexpr int kTile = kTileThreads * kPerThread;     // groups per CTA

// Bit k set iff group base + k is kept, for the 16 groups a thread owns.
template <bool kVec>
__device__ __forceinline__ uint32_t kept_bits(const uint8_t* __restrict__ stop,
                                              const uint8_t* __restrict__ zero_var, int base,
                                              int n_groups) {
    uint32_t drop = 0u;
    if (kVec && base + kPerThread <= n_groups) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (stop) v = __ldg(reinterpret_cast<const uint4*>(stop + base));
        if (zero_var) {
            const uint4 z = __ldg(reinterpret_cast<const uint4*>(zero_var + base));
            v.x |= z.x; v.y |= z.y; v.z |= z.z; v.w |= z.w;
        }
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            // a byte is "set" when any of its bits is: fold every byte onto its top bit
            uint32_t t = w[q];
            t |= t << 4; t |= t << 2; t |= t << 1;
            t &= 0x80808080u;
            // gather the four top bits (bytes 0..3) into bits 0..3: the multiplier puts
            // byte k's flag at bit 21 + k and no two partial products share a position
            drop |= ((((t >> 7) * 0x00204081u) >> 21) & 0xFu) << (4 * q);
        }
        return ~drop & 0xFFFFu;
    }
    uint32_t keep = 0u;
    for (int k = 0; k < kPerThread; ++k) {
        const int g = base + k;
        if (g >= n_groups) break;
        const bool d = (stop && stop[g] != 0) || (zero_var && zero_var[g] != 0);
        keep |= d ? 0u : 1u << k;
    }
    return keep;
}

template <bool kVec>
__global__ void __launch_bounds__(kTileThreads)
kept_count_kernel(const uint8_t* __restrict__ stop, const uint8_t* __restrict__ zero_var,
                  int n_groups, int32_t* __restrict__ tile_count) {
    __shared__ int s_warp[kTileThreads / 32];
    const int base = (blockIdx.x * kTileThreads + threadIdx.x) * kPerThread;
    int c = base < n_groups ? __popc(kept_bits<kVec>(stop, zero_var, base, n_groups)) : 0;
    c = __reduce_add_sync(0xFFFFFFFFu, c);
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = c;
    __syncthreads();
    if (threadIdx.x == 0) {
        int t = 0;
        for (int w = 0; w < kTileThreads / 32; ++w) t += s_warp[w];
        tile_count[blockIdx.x] = t;
    }
}

// Exclusive prefix sum of the tile counts, in place; the total goes to *count.  One CTA:
// a batch of 4 M groups has about a thousand tiles.
__global__ void __launch_bounds__(1024)
kept_offsets_kernel(int32_t* __restrict__ tile_count, int n_tiles, int32_t* __restrict__ count) {
    __shared__ int s_warp[32];
    __shared__ int s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (int t0 = 0; t0 < n_tiles; t0 += 1024) {
        const int t = t0 + threadIdx.x;
        const int v = t < n_tiles ? tile_count[t] : 0;
        int incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int w = s_warp[lane];
            int wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xFFFFFFFFu, wi, d);
                if (lane >= d) wi += up;
            }
            s_warp[lane] = wi - w;
        }
        __syncthreads();
        const int carry = s_carry;
        if (t < n_tiles) tile_count[t] = carry + s_warp[warp] + incl - v;
        __syncthreads();
        if (threadIdx.x == 1023) s_carry = carry + s_warp[warp] + incl;
        __syncthreads();
    }
    if (threadIdx.x == 0) *count = s_carry;
}

template <bool kVec>
__global__ void __launch_bounds__(kTileThreads)
kept_scatter_kernel(const uint8_t* __restrict__ stop, const uint8_t* __restrict__ zero_var,
                    int n_groups, const int32_t* __restrict__ tile_offset,
                    int32_t* __restrict__ index) {
    __shared__ int s_warp[kTileThreads / 32];
    __shared__ int32_t s_idx[kTile];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int base = (blockIdx.x * kTileThreads + threadIdx.x) * kPerThread;
    uint32_t keep = base < n_groups ? kept_bits<kVec>(stop, zero_var, base, n_groups) : 0u;
    const int c = __popc(keep);
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int before = incl - c, total = 0;
#pragma unroll
    for (int w = 0; w < kTileThreads / 32; ++w) {
        const int v = s_warp[w];
        if (w < warp) before += v;
        total += v;
    }
    while (keep) {                                   // ascending within the thread's 16 groups
        const int k = __ffs(keep) - 1;
        keep &= keep - 1u;
        s_idx[before++] = base + k;
    }
    __syncthreads();
    int32_t* out = index + tile_offset[blockIdx.x];
    for (int e = threadIdx.x; e < total; e += kTileThreads) out[e] = s_idx[e];
}

}  // namespace

size_t kept_groups_workspace_bytes(int32_t n_groups) {
    const size_t tiles = ((size_t)(n_groups > 0 ? n_groups : 0) + kTile - 1) / kTile;
    return align_up((tiles > 0 ? tiles : 1) * sizeof(int32_t), 256);
}

int launch_kept_groups(const uint8_t* stop, const uint8_t* zero_var, int32_t n_groups,
                       int32_t* index, int32_t* count, void* ws, cudaStream_t s) {
    if (n_groups == 0) {
        SR_CUDA_TRY(cudaMemsetAsync(count, 0, sizeof(int32_t), s));
        return SR_OK;
    }
    int32_t* tiles = static_cast<int32_t*>(ws);
    const int n_tiles = (n_groups + kTile - 1) / kTile;
    const bool vec = ((reinterpret_cast<uintptr_t>(stop) | reinterpret_cast<uintptr_t>(zero_var)) & 15) == 0;
    if (vec) kept_count_kernel<true><<<n_tiles, kTileThreads, 0, s>>>(stop, zero_var, n_groups, tiles);
    else kept_count_kernel<false><<<n_tiles, kTileThreads, 0, s>>>(stop, zero_var, n_groups, tiles);
    SR_LAUNCH_CHECK("kept_count_kernel");
    kept_offsets_kernel<<<1, 1024, 0, s>>>(tiles, n_tiles, count);
    SR_LAUNCH_CHECK("kept_offsets_kernel");
    if (vec) kept_scatter_kernel<true><<<n_tiles, kTileThreads, 0, s>>>(stop, zero_var, n_groups, tiles, index);
    else kept_scatter_kernel<false><<<n_tiles, kTileThreads, 0, s>>>(stop, zero_var, n_groups, tiles, index);
    SR_LAUNCH_CHECK("kept_scatter_kernel");
    return SR_OK;
}

}  // namespace sr
