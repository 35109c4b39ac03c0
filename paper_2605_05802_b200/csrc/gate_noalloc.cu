// sr_gate_noalloc: the gate for callers that must not allocate device memory.
//
// A rollout worker that gates its groups usually lives inside a process whose GPU
// memory was handed out long before: the inference engine reserved its share at
// start-up, the trainer's allocator owns the rest, and a cudaMalloc from a helper
// library either fails or fragments somebody's pool (and synchronises the device
// at the worst moment, in the middle of a generation step).  For those callers the
// multi-word gate's scratch lives in the array below.  It is part of this file's device
// image: the CUDA runtime sets it aside on a GPU when that image is first loaded there --
// with the runtime's default lazy loading that is the first call below on that device --
// and releases it at process exit.
#include <mutex>

#include "common.cuh"

namespace sr {
namespace {

// Scratch of the multi-word pipeline (control block, pair descriptors, match
// streams, ordering).  Held, until exit, by every GPU on which the entry point has run.
static __device__ __align__(256) unsigned char g_noalloc_scratch[SR_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// In host code `g_noalloc_scratch` names a host-side shadow, not device memory; the
// device address has to be asked for, once per device, with that device current.  The
// answer is remembered per device index (devices beyond the table are simply asked every
// time); a cudaDeviceReset invalidates it, so a process that resets a device must not
// call this entry point on it afterwards.
int scratch_address(void** out) {
    int dev = 0;
    SR_CUDA_TRY(cudaGetDevice(&dev));
    const bool cached = dev >= 0 && dev < kMaxDevices;
    std::lock_guard<std::mutex> lock(g_mu);
    if (cached && g_scratch_addr[dev] != nullptr) {
        *out = g_scratch_addr[dev];
        return SR_OK;
    }
    void* p = nullptr;
    SR_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    if (cached) g_scratch_addr[dev] = p;
    *out = p;
    return SR_OK;
}

}  // namespace
}  // namespace sr

extern "C" int sr_gate_noalloc(const int32_t* seqs, const int32_t* lens, int32_t n_groups, int32_t N,
                               int32_t stride, int32_t K, double threshold, int32_t norm_mode,
                               int32_t* pair_dist, int32_t* pair_sum, double* mean, uint8_t* stop,
                               int32_t* status, void* stream) {
    using namespace sr;
    // every argument rule of sr_gate first, so that an invalid call reports its own error
    const int bad = check_gate_args(seqs, n_groups, N, stride, K, norm_mode, stop);
    if (bad != SR_OK) return bad;
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
