// Launching a kernel so that it may overlap the tail of the kernel before it in the stream (programmatic dependent launch).
//
// A kernel launched this way may become resident as soon as every CTA of the previous kernel has called
// ptx::grid_launch_dependents() (or exited).  It must call ptx::grid_dependency_wait() before it touches anything
// the previous kernel reads or writes; the wait returns once that kernel has completed and its writes are visible.
// What comes before the wait (barrier initialisation, reading launch tables, filling shared memory) then overlaps
// the previous kernel's drain, and the launch latency is hidden.  After anything else than a kernel (a copy, an event
// of another stream) the launch is ordered as usual and the wait returns at once.
#pragma once
#include <cuda_runtime.h>

#include <cstdlib>

namespace ipkvi {

inline bool overlap_launches() {
    static const bool on = std::getenv("IPKV_NO_LAUNCH_OVERLAP") == nullptr;
    return on;
}

// `overlap` false launches plainly: for a kernel whose launch tables were written by the kernel right in front of it
// (it reads them before its wait).
template <typename... Params, typename... Args>
inline cudaError_t launch_ordered(bool overlap, void (*kernel)(Params...), int grid, int block, size_t smem, cudaStream_t s, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(unsigned(block));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = (overlap && overlap_launches()) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}

template <typename... Params, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(Params...), int grid, int block, size_t smem, cudaStream_t s, Args&&... args) {
    return launch_ordered(true, kernel, grid, block, smem, s, static_cast<Args&&>(args)...);
}

}  // namespace ipkvi
