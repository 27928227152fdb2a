// Measurement aid: what one tcgen05.mma costs on this GPU when the instruction is small.
//
// The compressed-latent attention kernel has only 16 query heads per cached row, so a fifth-generation tensor-core
// formulation of it issues many small MMAs (N = 16 .. 64).  Whether that can work is a question of the fixed cost per
// instruction against its useful work, and this probe answers it in isolation: one CTA, one issuing thread, operands
// in shared memory in the canonical 128-byte-swizzled K-major layout, accumulators in tensor memory; n back-to-back
// tcgen05.mma of one shape (K = 16, bf16 in, fp32 out) followed by one commit.  Two clocks are read: when the last
// instruction has been issued, and when the commit's mbarrier has completed.  From n = 1, 8 and 36 the fixed part
// (launch-to-completion latency of one instruction) and the per-instruction throughput separate; issuing into one
// accumulator or rotating over four shows whether the accumulation chain matters.
//
// Every wait is bounded; the tensor memory is released before the kernel returns.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/ipkv.h"
#include "ptx.cuh"

namespace ipkvi {
namespace {

constexpr int kABytes = 128 * 128;        // A tile: up to 128 rows x 64 bf16 columns (one swizzle atom wide)
constexpr int kBBytes = 256 * 128;        // B tile: up to 256 rows x 64 bf16 columns
constexpr uint32_t kTmemCols = 512;

// Shared-memory matrix descriptor, K-major, 128-byte swizzle: start address, leading / stride byte offsets (>> 4).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return uint64_t((addr & 0x3FFFFu) >> 4) | (uint64_t(lbo >> 4) << 16) | (uint64_t(sbo >> 4) << 32) | (uint64_t(1) << 46) |
           (uint64_t(2) << 61);
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
        ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

template <int M, int N, int NMMA, int ROT>
__global__ void __launch_bounds__(128) umma_probe_kernel(long long* out, uint32_t* status) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_a = s_base, s_b = s_base + kABytes, s_bar = s_b + kBBytes, s_slot = s_bar + 16;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kABytes + kBBytes + 16);
    const int tid = threadIdx.x, warp = tid >> 5;
    // operands: small finite values (what they are does not matter for the timing)
    for (int i = tid; i < (kABytes + kBBytes) / 4; i += 128) reinterpret_cast<uint32_t*>(smem)[i] = 0x3c003c00u + uint32_t(i & 7);
    if (tid == 0) {
        ptx::mbar_init(s_bar, 1);
        ptx::mbar_fence_init();
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_slot), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;
    if (tid == 0) {
        constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t(N) >> 3) << 17) | ((uint32_t(M) >> 4) << 24);
        // descriptors are a base plus a constant: the four K = 16 slices of the 64-column atom are 32 bytes apart
        const uint64_t a0 = smem_desc(s_a, 16, 1024), b0 = smem_desc(s_b, 16, 1024);
        const long long t0 = clock64();
#pragma unroll
        for (int i = 0; i < NMMA; ++i)
            umma(tmem + uint32_t(i % ROT) * uint32_t(N), a0 + uint64_t((i & 3) * 2), b0 + uint64_t((i & 3) * 2), idesc, i >= ROT ? 1u : 0u);
        umma_commit(s_bar);
        const long long t1 = clock64();
        const bool done = ptx::mbar_wait(s_bar, 0);
        const long long t2 = clock64();
        out[0] = t1 - t0;
        out[1] = t2 - t0;
        if (!done) atomicOr(status, 1u);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

template <int M, int N, int NMMA, int ROT>
cudaError_t run_one(long long* out_dev, uint32_t* status_dev, int reps, ipkv_umma_timing* t) {
    const int smem = kABytes + kBBytes + 64 + 1024;
    cudaError_t e = cudaFuncSetAttribute(umma_probe_kernel<M, N, NMMA, ROT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    long long best_issue = 1ll << 60, best_total = 1ll << 60;
    for (int r = 0; r < reps + 1; ++r) {                      // the first launch is a warm-up
        umma_probe_kernel<M, N, NMMA, ROT><<<1, 128, smem>>>(out_dev, status_dev);
        long long h[2];
        e = cudaMemcpy(h, out_dev, sizeof h, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) return e;
        if (r > 0) { best_issue = h[0] < best_issue ? h[0] : best_issue; best_total = h[1] < best_total ? h[1] : best_total; }
    }
    t->m = M; t->n = N; t->n_mma = NMMA; t->accumulators = ROT;
    t->issue_cycles = best_issue; t->total_cycles = best_total;
    return cudaSuccess;
}

template <int M, int N>
cudaError_t run_shape(long long* out_dev, uint32_t* status_dev, int reps, ipkv_umma_timing* t, int* k, int cap) {
    cudaError_t e = cudaSuccess;
    auto next = [&]() -> ipkv_umma_timing* { return (*k < cap) ? &t[(*k)++] : nullptr; };
    ipkv_umma_timing* x;
    if ((x = next()) && (e = run_one<M, N, 1, 1>(out_dev, status_dev, reps, x)) != cudaSuccess) return e;
    if ((x = next()) && (e = run_one<M, N, 8, 1>(out_dev, status_dev, reps, x)) != cudaSuccess) return e;
    if ((x = next()) && (e = run_one<M, N, 36, 1>(out_dev, status_dev, reps, x)) != cudaSuccess) return e;
    if (N <= 128) {
        if ((x = next()) && (e = run_one<M, N, 36, (N <= 128 ? 4 : 1)>(out_dev, status_dev, reps, x)) != cudaSuccess) return e;
    }
    return e;
}

}  // namespace
}  // namespace ipkvi

using namespace ipkvi;

ipkv_status ipkv_probe_umma(int32_t device, int32_t reps, ipkv_umma_timing* out, int32_t cap, int32_t* n_out) {
    if (!out || !n_out || cap <= 0 || reps <= 0) return IPKV_EINVAL;
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return IPKV_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) return IPKV_ECUDA;
    long long* out_dev = nullptr;
    uint32_t* status_dev = nullptr;
    ipkv_status rc = IPKV_OK;
    int k = 0;
    do {
        if (cudaMalloc(&out_dev, 16) != cudaSuccess || cudaMalloc(&status_dev, 4) != cudaSuccess) { rc = IPKV_ENOMEM; break; }
        if (cudaMemset(status_dev, 0, 4) != cudaSuccess) { rc = IPKV_ECUDA; break; }
        cudaError_t e = run_shape<64, 16>(out_dev, status_dev, reps, out, &k, cap);
        if (e == cudaSuccess) e = run_shape<64, 64>(out_dev, status_dev, reps, out, &k, cap);
        if (e == cudaSuccess) e = run_shape<64, 256>(out_dev, status_dev, reps, out, &k, cap);
        if (e == cudaSuccess) e = run_shape<128, 16>(out_dev, status_dev, reps, out, &k, cap);
        if (e == cudaSuccess) e = run_shape<128, 64>(out_dev, status_dev, reps, out, &k, cap);
        if (e == cudaSuccess) e = run_shape<128, 256>(out_dev, status_dev, reps, out, &k, cap);
        if (e != cudaSuccess) { rc = IPKV_ECUDA; break; }
        uint32_t st = 0;
        if (cudaMemcpy(&st, status_dev, 4, cudaMemcpyDeviceToHost) != cudaSuccess) { rc = IPKV_ECUDA; break; }
        if (st != 0) rc = IPKV_ETIMEOUT;
    } while (false);
    *n_out = k;
    if (out_dev) cudaFree(out_dev);
    if (status_dev) cudaFree(status_dev);
    if (prev >= 0) cudaSetDevice(prev);
    return rc;
}
