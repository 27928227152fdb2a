// ipkv_attend_runs_noalloc: split-K decode attention for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc where they call attention: an inference server that
// hands its whole memory budget to its own pool at start-up (a later driver allocation would either fail
// or break its accounting), code that runs inside a latency-critical loop where cudaMalloc's implicit
// device synchronisation is not acceptable, or a plug-in whose contract forbids allocating. For them the
// scratch that split-K attention needs (descriptor tables, one partial (O, LSE) per work item, a status
// word) lives in a fixed array inside the library's own device image instead of in caller memory.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/ipkv.h"

namespace {

constexpr size_t kStaticScratchBytes = size_t(16) << 20;   // 16 MiB, held by every GPU on which the entry point has run

// File-scope device array. In host code this name is only a stand-in for the symbol, not a device address:
// the address the kernels need comes from cudaGetSymbolAddress, once per device.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the array on the CURRENT device, resolved on first use on that device.  With CUDA's lazy module
// loading that first use is also what makes the driver materialise the array on the device, so it can fail on a device
// whose memory is already taken; the address is remembered per device ordinal and is stale after a cudaDeviceReset.
cudaError_t static_scratch_address(void** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t ipkv_noalloc_scratch_limit(void) { return kStaticScratchBytes; }

ipkv_status ipkv_attend_runs_noalloc(const ipkv_attn_shape* shape, int32_t n_rows,
                                     const ipkv_run* runs, const int32_t* row_run_start,
                                     const void* q_dev, int32_t kv_splits,
                                     float* o_part_dev, float* lse_part_dev, uint32_t* status_dev, void* stream) {
    if (!shape || n_rows <= 0 || !row_run_start) return IPKV_EINVAL;
    const int32_t n_runs = row_run_start[n_rows];
    if (n_runs < 0 || (n_runs > 0 && !runs)) return IPKV_EINVAL;
    int64_t total_tokens = 0;
    for (int32_t k = 0; k < n_runs; ++k) {
        if (runs[k].n_tokens < 0) return IPKV_EINVAL;
        total_tokens += runs[k].n_tokens;
    }
    size_t need = 0;
    ipkv_status rc = ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total_tokens, kv_splits, &need);
    if (rc != IPKV_OK) return rc;
    if (need > kStaticScratchBytes) return IPKV_ERANGE;     // larger than the built-in array: use ipkv_attend_runs
    void* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return IPKV_ECUDA;
    // Every call shares the array and finds the previous call's bytes in it. Nothing in it has to start at
    // zero: the tables and the partials are rewritten in full before they are read, and the status word kept
    // in the array (used only when status_dev is NULL) is never read back.
    rc = ipkv_attend_runs(shape, n_rows, runs, row_run_start, q_dev, kv_splits, scratch, kStaticScratchBytes,
                          o_part_dev, lse_part_dev, status_dev, stream);
    return rc == IPKV_ENOMEM ? IPKV_ERANGE : rc;            // "does not fit the array" is a range error of this call
}

}  // extern "C"
