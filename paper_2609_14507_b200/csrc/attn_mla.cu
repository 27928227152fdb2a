// Compressed-latent (MLA) variant of the GPU-side decode attention. Placeholder until the kernel lands.
#include "kernels.h"

namespace ipkvi {

cudaError_t launch_attend_mla(const AttnLaunch& a, cudaStream_t) {
    if (a.n_items <= 0) return cudaSuccess;
    return cudaErrorNotSupported;
}

}  // namespace ipkvi
