// Exact log-sum-exp joins (Sec. 4.2 "merged via log-sum-exp rescaling", Sec. 5.1 "merge exactly"):
//   LSE = m + ln sum_i exp(LSE_i - m), m = max_i LSE_i;   O = sum_i exp(LSE_i - LSE) * O_i.
//   split_reduce_kernel  second pass of split-K attention: joins the item partials of every
//                        (row, query head), optionally folding in an earlier partial of the same row
//   merge_kernel         joins up to 8 row-aligned partials (GPU share, CPU share, ...)
// One warp per output row; lanes stride over the value columns with 16-byte accesses.
#include <cuda_bf16.h>

#include "kernels.h"

namespace ipkvi {

namespace {

constexpr int kWarpsPerBlock = 4;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
split_reduce_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                    const int32_t* __restrict__ row_item_start, const float* acc_o, const float* acc_lse,
                    float* out_o, float* out_lse, int n_rows, int Hq, int dv) {
    const int wid = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (wid >= n_rows * Hq) return;
    const int row = wid / Hq, h = wid - row * Hq;
    const int i0 = row_item_start[row], i1 = row_item_start[row + 1];
    float m = acc_lse ? acc_lse[wid] : -INFINITY;
    for (int i = i0 + lane; i < i1; i += 32) m = fmaxf(m, part_lse[int64_t(i) * Hq + h]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    float* oo = out_o + int64_t(wid) * dv;
    if (m == -INFINITY) {                       // nothing attended: (0, -inf)
        for (int c = lane * 4; c < dv; c += 128) *reinterpret_cast<float4*>(oo + c) = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane == 0) out_lse[wid] = -INFINITY;
        return;
    }
    float z = 0.f;
    for (int i = i0 + lane; i < i1; i += 32) z += __expf(part_lse[int64_t(i) * Hq + h] - m);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) z += __shfl_xor_sync(0xffffffffu, z, d);
    const float wa = acc_lse ? __expf(acc_lse[wid] - m) : 0.f;
    z += wa;
    const float inv = 1.f / z;
    for (int c = lane * 4; c < dv; c += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (acc_o && wa != 0.f) {
            const float4 v = *reinterpret_cast<const float4*>(acc_o + int64_t(wid) * dv + c);
            acc.x = wa * v.x; acc.y = wa * v.y; acc.z = wa * v.z; acc.w = wa * v.w;
        }
        for (int i = i0; i < i1; ++i) {
            const float w = __expf(part_lse[int64_t(i) * Hq + h] - m);
            const float4 v = *reinterpret_cast<const float4*>(part_o + (int64_t(i) * Hq + h) * dv + c);
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
        }
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        *reinterpret_cast<float4*>(oo + c) = acc;
    }
    __syncwarp();   // every lane has read acc_lse[wid] (it may alias out_lse) before it is overwritten
    if (lane == 0) out_lse[wid] = m + logf(z);
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) merge_kernel(const MergeLaunch a) {
    const int row = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (row >= a.n_rows) return;
    float li[kMaxMergeParts];
    float m = -INFINITY;
#pragma unroll
    for (int i = 0; i < kMaxMergeParts; ++i) {
        li[i] = (i < a.n_parts) ? a.lse[i][row] : -INFINITY;
        m = fmaxf(m, li[i]);
    }
    float z = 0.f;
    float w[kMaxMergeParts];
#pragma unroll
    for (int i = 0; i < kMaxMergeParts; ++i) {
        w[i] = (m == -INFINITY || li[i] == -INFINITY) ? 0.f : __expf(li[i] - m);
        z += w[i];
    }
    const float inv = (z > 0.f) ? 1.f / z : 0.f;
    for (int c = lane * 4; c < a.dim_v; c += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int i = 0; i < kMaxMergeParts; ++i) {
            if (i < a.n_parts && w[i] != 0.f) {
                const float4 v = *reinterpret_cast<const float4*>(a.o[i] + int64_t(row) * a.dim_v + c);
                acc.x += w[i] * v.x; acc.y += w[i] * v.y; acc.z += w[i] * v.z; acc.w += w[i] * v.w;
            }
        }
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        if (a.out_is_bf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(a.out_o) + int64_t(row) * a.dim_v + c) = pk;
        } else {
            *reinterpret_cast<float4*>(static_cast<float*>(a.out_o) + int64_t(row) * a.dim_v + c) = acc;
        }
    }
    if (lane == 0 && a.out_lse) a.out_lse[row] = (z > 0.f) ? m + logf(z) : -INFINITY;
}

}  // namespace

cudaError_t launch_split_reduce(const AttnLaunch& a, cudaStream_t s) {
    const int total = a.n_rows * a.n_q_heads;
    if (total <= 0) return cudaSuccess;
    const int grid = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    split_reduce_kernel<<<grid, kWarpsPerBlock * 32, 0, s>>>(a.part_o, a.part_lse, a.row_item_start, a.acc_o, a.acc_lse,
                                                            a.out_o, a.out_lse, a.n_rows, a.n_q_heads, a.dim_v);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeLaunch& m, cudaStream_t s) {
    if (m.n_rows <= 0) return cudaSuccess;
    const int grid = (m.n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
    merge_kernel<<<grid, kWarpsPerBlock * 32, 0, s>>>(m);
    return cudaGetLastError();
}

}  // namespace ipkvi
