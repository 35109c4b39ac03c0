// Register-only integer throughput probe (see include/sr_probe.h).  Each thread
// runs 8 independent dependency chains so that the integer pipe always has an
// instruction to issue; inline PTX keeps the compiler from folding the chains.
#include "common.cuh"
#include "sr_probe.h"

namespace sr {
namespace {

template <int VARIANT>
__global__ void __launch_bounds__(1024)
probe_int32_kernel(int iters, uint32_t* sink) {
    uint32_t x[8];
    const uint32_t t = blockIdx.x * blockDim.x + threadIdx.x;
#pragma unroll
    for (int k = 0; k < 8; ++k) x[k] = t * 2654435761u + (uint32_t)k * 40503u;
    uint32_t a = t | 1u, b = ~t;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 16; ++u) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const bool add = VARIANT == SR_PROBE_ADD || (VARIANT == SR_PROBE_MIX && (u % 5) == 4);
                if (add)
                    asm volatile("add.u32 %0, %0, %1;" : "+r"(x[k]) : "r"(a));
                else   // x = (x & a) ^ b as one three-input logic operation
                    asm volatile("lop3.b32 %0, %0, %1, %2, 0x6A;" : "+r"(x[k]) : "r"(a), "r"(b));
            }
        }
    }
    uint32_t acc = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) acc ^= x[k];
    sink[t] = acc;
}

}  // namespace
}  // namespace sr

extern "C" {

uint64_t sr_probe_int32_ops(int32_t iters, int32_t blocks, int32_t threads) {
    if (iters < 0 || blocks < 0 || threads < 0) return 0;
    return (uint64_t)iters * 16u * 8u * (uint64_t)blocks * (uint64_t)threads;
}

int sr_probe_int32(int32_t variant, int32_t iters, int32_t blocks, int32_t threads, uint32_t* sink,
                   void* stream) {
    if (sink == nullptr) return SR_ERR_NULL;
    if (iters < 1 || blocks < 1 || threads < 32 || threads > 1024 || (threads & 31)) return SR_ERR_BAD_N;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (variant) {
        case SR_PROBE_LOGIC: sr::probe_int32_kernel<SR_PROBE_LOGIC><<<blocks, threads, 0, s>>>(iters, sink); break;
        case SR_PROBE_ADD: sr::probe_int32_kernel<SR_PROBE_ADD><<<blocks, threads, 0, s>>>(iters, sink); break;
        case SR_PROBE_MIX: sr::probe_int32_kernel<SR_PROBE_MIX><<<blocks, threads, 0, s>>>(iters, sink); break;
        default: return SR_ERR_BAD_MODE;
    }
    SR_LAUNCH_CHECK("probe_int32_kernel");
    return SR_OK;
}

}  // extern "C"
