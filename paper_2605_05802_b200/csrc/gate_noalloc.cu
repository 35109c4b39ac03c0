// sr_gate_noalloc: the gate for callers that must not allocate device memory.
//
// A rollout worker that gates its groups usually lives inside a process whose GPU
// memory was handed out long before: the inference engine reserved its share at
// start-up, the trainer's allocator owns the rest, and a cudaMalloc from a helper
// library either fails or fragments somebody's pool (and synchronises the device
// at the worst moment, in the middle of a generation step).  For those callers the
// multi-word gate's scratch lives in the array below, which the CUDA runtime sets
// aside when the library is loaded on a GPU and releases at process exit.
#include <mutex>

#include "common.cuh"

namespace sr {
namespace {

// Scratch of the multi-word pipeline (control block, pair descriptors, match
// streams, ordering).  Held by every GPU that loads the library, until exit.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SR_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// In host code `g_noalloc_scratch` names a host-side shadow, not device memory; the
// device address has to be asked for, once per device, with that device current.
int scratch_address(void** out) {
    int dev = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SR_ERR_BAD_N;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        SR_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return SR_OK;
}

}  // namespace
}  // namespace sr

extern "C" int sr_gate_noalloc(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                               int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                               int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                               int32_t* status, void* stream) {
    using namespace sr;
    if (n_groups < 0 || N < 2 || N > SR_MAX_N) return SR_ERR_BAD_N;
    if (stride < 0 || K < 0 || K > stride || K > SR_MAX_K) return SR_ERR_BAD_K;
    if (K <= 32 || n_groups == 0)      // the single-word path needs no scratch at all
        return sr_gate(seqs, lens, n_groups, N, stride, K, threshold, norm_mode, pair_dist, pair_sum,
                       mean, stop, status, nullptr, 0, stream);
    const size_t need = sr_gate_workspace_bytes(n_groups, N, stride, K);
    if (need > (size_t)SR_NOALLOC_SCRATCH_BYTES) return SR_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != SR_OK) return rc;
    // the pipeline clears the part of the scratch that must start at zero (its bin
    // counters) at the head of every call; everything else is written before it is read
    return sr_gate(seqs, lens, n_groups, N, stride, K, threshold, norm_mode, pair_dist, pair_sum,
                   mean, stop, status, scratch, SR_NOALLOC_SCRATCH_BYTES, stream);
}

extern "C" size_t sr_gate_noalloc_limit_bytes(void) { return (size_t)SR_NOALLOC_SCRATCH_BYTES; }
