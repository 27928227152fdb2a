// Measurement aid: the rate at which the SMs can pull bytes out of HBM through the same copy ring the attention
// kernels use (bulk asynchronous copies into a shared-memory ring that complete on mbarriers), with no arithmetic at
// all.  It is the ceiling the attention kernels are compared with beside the copy bandwidth of the roofline: a copy
// moves every byte twice (read + write), a decode-attention kernel only reads.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/ipkv.h"
#include "kernels.h"
#include "ptx.cuh"

namespace ipkvi {
namespace {

constexpr int kProbeStages = 3;
constexpr int kProbeStageBytes = 32768;

__global__ void __launch_bounds__(32) read_ring_kernel(const char* src, int64_t tiles_per_cta, uint32_t* sink, uint32_t* status) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_full = s_base + kProbeStages * kProbeStageBytes;
    if (threadIdx.x != 0) return;
    for (int s = 0; s < kProbeStages; ++s) ptx::mbar_init(s_full + 8 * s, 1);
    ptx::mbar_fence_init();
    const uint64_t pol = ptx::l2_evict_first_policy();
    const char* base = src + int64_t(blockIdx.x) * tiles_per_cta * kProbeStageBytes;
    uint32_t acc = 0;
    bool ok = true;
    for (int64_t i = 0; i < tiles_per_cta + kProbeStages && ok; ++i) {
        if (i >= kProbeStages) {                       // tile i - kProbeStages has landed: touch it, free the stage
            const int64_t j = i - kProbeStages;
            const int st = int(j % kProbeStages);
            if (!ptx::mbar_wait(s_full + 8 * st, uint32_t(j / kProbeStages) & 1u)) { ok = false; break; }
            acc += *reinterpret_cast<volatile uint32_t*>(smem + st * kProbeStageBytes);
        }
        if (i < tiles_per_cta) {
            const int st = int(i % kProbeStages);
            ptx::mbar_expect_tx(s_full + 8 * st, kProbeStageBytes);
            ptx::bulk_g2s_hint(s_base + st * kProbeStageBytes, base + i * kProbeStageBytes, kProbeStageBytes, s_full + 8 * st, pol);
        }
    }
    if (!ok) atomicOr(status, kStatusNoTile);
    if (acc == 0x9e3779b9u) *sink = acc;               // keeps the loads alive
}


// Self-test of the bounded waits: one CTA; its producer thread announces a tile on a stage barrier (expect_tx) and
// then issues no copy for it; a consumer thread waits for that tile with a short limit.  The wait runs out, the
// consumer records kStatusNoTile and the kernel returns: nothing spins without a limit, nothing faults, no copy is in
// flight when the CTA leaves.
__global__ void __launch_bounds__(64) expire_wait_kernel(uint32_t* status, uint64_t limit_ns) {
    __shared__ __align__(8) uint64_t bar_storage;
    const uint32_t bar = ptx::smem_addr(&bar_storage);
    if (threadIdx.x == 0) {
        ptx::mbar_init(bar, 1);
        ptx::mbar_fence_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) ptx::mbar_expect_tx(bar, 16);          // a tile of 16 bytes that never comes
    if (threadIdx.x == 32 && !ptx::mbar_wait(bar, 0, limit_ns)) atomicOr(status, kStatusNoTile);
}

}  // namespace

cudaError_t launch_expire_wait(uint32_t* status, uint64_t limit_ns, cudaStream_t s) {
    expire_wait_kernel<<<1, 64, 0, s>>>(status, limit_ns);
    return cudaGetLastError();
}

}  // namespace ipkvi

using namespace ipkvi;

ipkv_status ipkv_probe_read_bandwidth(int32_t device, size_t bytes, int32_t reps, double* best_gbs, double* mean_gbs) {
    if (!best_gbs || !mean_gbs || reps <= 0 || bytes < (size_t(64) << 20)) return IPKV_EINVAL;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return IPKV_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) return IPKV_ECUDA;
    const int ctas = 148 * 2;
    const int64_t tiles_per_cta = int64_t(bytes / kProbeStageBytes / ctas);
    const size_t total = size_t(tiles_per_cta) * kProbeStageBytes * ctas;
    const int n_buf = 2;                                // alternate two buffers: nothing read is still in L2
    char* buf = nullptr;
    uint32_t* words = nullptr;
    cudaEvent_t a = nullptr, b = nullptr;
    ipkv_status rc = IPKV_OK;
    const int smem = kProbeStages * kProbeStageBytes + 64 + 1024;
    do {
        if (cudaMalloc(&buf, total * n_buf) != cudaSuccess) { rc = IPKV_ENOMEM; break; }
        if (cudaMalloc(&words, 8) != cudaSuccess) { rc = IPKV_ENOMEM; break; }
        if (cudaMemset(buf, 1, total * n_buf) != cudaSuccess || cudaMemset(words, 0, 8) != cudaSuccess) { rc = IPKV_ECUDA; break; }
        if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { rc = IPKV_ECUDA; break; }
        if (cudaFuncSetAttribute(read_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) { rc = IPKV_ECUDA; break; }
        double best = 0.0, sum = 0.0;
        for (int r = 0; r < reps + 3 && rc == IPKV_OK; ++r) {      // three untimed warm-up launches
            cudaEventRecord(a);
            read_ring_kernel<<<ctas, 32, smem>>>(buf + size_t(r % n_buf) * total, tiles_per_cta, words, words + 1);
            cudaEventRecord(b);
            if (cudaEventSynchronize(b) != cudaSuccess) { rc = IPKV_ECUDA; break; }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, a, b);
            if (r >= 3) { const double g = double(total) / (double(ms) * 1e-3) / 1e9; best = g > best ? g : best; sum += g; }
        }
        uint32_t st = 0;
        if (rc == IPKV_OK && cudaMemcpy(&st, words + 1, 4, cudaMemcpyDeviceToHost) != cudaSuccess) rc = IPKV_ECUDA;
        if (rc == IPKV_OK && st != 0) rc = IPKV_ETIMEOUT;
        *best_gbs = best; *mean_gbs = sum / reps;
    } while (false);
    if (a) cudaEventDestroy(a);
    if (b) cudaEventDestroy(b);
    if (words) cudaFree(words);
    if (buf) cudaFree(buf);
    if (prev >= 0) cudaSetDevice(prev);
    return rc;
}
