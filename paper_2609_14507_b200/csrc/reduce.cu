// Exact log-sum-exp joins (Sec. 4.2 "merged via log-sum-exp rescaling", Sec. 5.1 "merge exactly"):
//   LSE = m + ln sum_i exp(LSE_i - m), m = max_i LSE_i;   O = sum_i exp(LSE_i - LSE) * O_i.
//   split_reduce_kernel  second pass of split-K attention: joins the item partials of every
//                        (row, query head), optionally folding in an earlier partial of the same row;
//                        one CTA per output row, threads split over (items, columns)
//   merge_kernel         joins up to 8 row-aligned partials (GPU share, CPU share, ...); one warp per row
#include <cuda_bf16.h>

#include "kernels.h"
#include "launch.cuh"
#include "ptx.cuh"

namespace ipkvi {

namespace {

constexpr int kWarpsPerBlock = 4;
constexpr int kPrefetch = 2;       // partial outputs per thread requested up front (of the own and of the extra partials)
constexpr int kLseCache = 512;     // LSE values kept in shared memory between the two passes

// One CTA per (row, query head, slab of up to 128 value columns). The partials to join are those of the spans of
// the head's group (parts_per_span consecutive entries per span), row `rin` of each. Threads are arranged as
// (entry slice, 4-column group): every thread sums the weighted partials of its slice for its four columns;
// the slices are then added through shared memory. CG = slab / 4 column groups, SL = 256 / CG slices: with at
// most 128 columns per CTA there are at least 8 slices, so a thread has few entries to fetch one after the other
// (a 512-column head handled by one CTA had two slices and ten dependent loads per thread).
struct ReduceParams {
    const float* part_o;
    const float* part_lse;
    const int32_t* rg_span_start;
    const float* acc_o;
    const float* acc_lse;
    float* out_o;
    float* out_lse;
    int Hq, dv, G, n_hg, n_gh, RG, NW;
    int CS, dvl;                  // column slabs per (row, head) and columns per slab
    const int32_t* extra_count;   // per (row, head group): extra partials written by CTAs that helped with its spans (null: none)
    const int32_t* extra_list;    // [n_rows * n_gh][kStealListCap] their indices; extra partial i is stored as if it were span n_spans + i
    int n_spans;
    int32_t* clear;               // scheduling words to zero for the next launch
    int clear_words;
};

// EXTRAS: the launch was dynamically balanced and may have extra partials (kept out of the plain instantiation, which
// then needs few enough registers for five CTAs per SM: launches with thousands of (row, head) pairs run in fewer waves).
// THREADS: 256, or 128 for launches with so many (row, head) pairs that 256-thread CTAs would need several waves (a
// ragged batch of 64 sequences x 32 heads: 2048 CTAs, at five per SM 2.8 waves, measured 10.4 us; with 128 threads ten
// fit an SM, 1.4 waves, 7.3 us; squeezing them to 32 registers so that 14 or 16 fit, one wave, spills, and was slower:
// 2.225 -> 2.269 ms per step).
template <bool EXTRAS, int THREADS>
__global__ void __launch_bounds__(THREADS, THREADS == 256 ? (EXTRAS ? 4 : 5) : 10) split_reduce_kernel(const ReduceParams p) {
    constexpr int kReduceThreads = THREADS;
    extern __shared__ float4 red[];                 // [SL][CG]
    __shared__ float s_warp[kReduceThreads / 32];
    __shared__ float s_w[kLseCache];               // LSE of the first entries
    __shared__ float s_zs[kReduceThreads / 16];    // weight sum of every entry slice (SL <= 16)
    __shared__ int s_extra[kStealListCap];         // extra partials that belong to this (row, head group)
    __shared__ int s_n_extra;
    const int wid = blockIdx.x / p.CS;               // row * Hq + h
    const int col0 = (blockIdx.x - wid * p.CS) * p.dvl;
    const int row = wid / p.Hq, h = wid - row * p.Hq;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = h / p.G, hin = h - g * p.G;
    const int gh = g * p.n_hg + hin / 16, rin = hin % 16;
    // the list of extra partials is requested together with the span range: one round of latency for both
    const int rg = row * p.n_gh + gh;
    const int sp0 = p.rg_span_start[rg], sp1 = p.rg_span_start[rg + 1];
    ptx::grid_dependency_wait();        // the attention kernel's partials and lists are complete from here on
    ptx::grid_launch_dependents();
    int list_entry = 0, list_count = 0;
    if (EXTRAS) {
        if (tid < kStealListCap) list_entry = p.extra_list[rg * kStealListCap + tid];
        if (tid == kStealListCap) list_count = min(p.extra_count[rg], kStealListCap);
    }
    const float la = p.acc_lse ? p.acc_lse[wid] : -INFINITY;
    for (int i = blockIdx.x * kReduceThreads + tid; i < p.clear_words; i += gridDim.x * kReduceThreads) p.clear[i] = 0;
    if (tid < kStealListCap) s_extra[tid] = list_entry;
    if (tid == kStealListCap) s_n_extra = list_count;
    __syncthreads();
    const int64_t e0 = int64_t(sp0) * p.NW;
    const int n_own = (sp1 - sp0) * p.NW;
    const int n_x = EXTRAS ? s_n_extra * p.NW : 0;  // entries of the extra partials
    const int n = n_own + n_x;
    const int dv = p.dv;
    // entry e of this (row, head group): the spans' own partials first, then the extra ones
    auto entry = [&](int e) -> int64_t {
        if (e < n_own) return e0 + e;
        const int k = (e - n_own) / p.NW;
        return int64_t(p.n_spans + s_extra[k]) * p.NW + (e - n_own - k * p.NW);
    };
    const float* lse_base = p.part_lse + rin;                      // entry e at lse_base[entry(e) * RG]
    const int CG = p.dvl >> 2, SL = kReduceThreads / CG;
    const int cg = tid % CG, sl = tid / CG;
    const float* po = p.part_o + int64_t(rin) * dv + col0 + cg * 4;
    const int64_t stride = int64_t(p.RG) * dv;

    // The partial outputs of this thread's first entries (own and extra) are requested before anything is known about
    // their weights, so that their latency overlaps the two passes over the LSE values (an entry that turns out to
    // be empty may hold anything: it is loaded but never used).
    constexpr int kPrefetchX = EXTRAS ? kPrefetch : 1;
    float4 pre[kPrefetch], prx[kPrefetchX];
#pragma unroll
    for (int j = 0; j < kPrefetch; ++j) {
        const int e = sl + j * SL;
        pre[j] = e < n_own ? *reinterpret_cast<const float4*>(po + (e0 + e) * stride) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < kPrefetchX; ++j) {
        const int x = sl + j * SL;
        prx[j] = x < n_x ? *reinterpret_cast<const float4*>(po + entry(n_own + x) * stride) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float4 fold = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p.acc_o && sl == 0) fold = *reinterpret_cast<const float4*>(p.acc_o + int64_t(wid) * dv + col0 + cg * 4);

    float m = la;
    for (int e = tid; e < n; e += kReduceThreads) {
        const float li = lse_base[entry(e) * p.RG];
        if (e < kLseCache) s_w[e] = li;
        m = fmaxf(m, li);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    if (lane == 0) s_warp[warp] = m;
    __syncthreads();
    {
        float mm = s_warp[0];
#pragma unroll
        for (int w = 1; w < kReduceThreads / 32; ++w) mm = fmaxf(mm, s_warp[w]);
        m = mm;
    }
    float* oo = p.out_o + int64_t(wid) * dv + col0;
    if (m == -INFINITY) {                           // nothing attended: (0, -inf)
        if (sl == 0) *reinterpret_cast<float4*>(oo + cg * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
        if (tid == 0 && col0 == 0) p.out_lse[wid] = -INFINITY;
        return;
    }
    // weight of entry e (0 for an empty one); the first kLseCache LSE values are in shared memory
    auto weight = [&](int e) -> float {
        const float li = e < kLseCache ? s_w[e] : lse_base[entry(e) * p.RG];
        return li == -INFINITY ? 0.f : __expf(li - m);
    };
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float z = 0.f;
    auto add = [&](float w, const float4& v) {
        if (w != 0.f) { acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w; z += w; }
    };
    // own entries, then extra ones; in each group the prefetched ones first, the rest loaded only if they count
#pragma unroll
    for (int j = 0; j < kPrefetch; ++j) {
        const int e = sl + j * SL;
        add(e < n_own ? weight(e) : 0.f, pre[j]);
    }
    for (int e = sl + kPrefetch * SL; e < n_own; e += SL) {
        const float w = weight(e);
        if (w != 0.f) add(w, *reinterpret_cast<const float4*>(po + (e0 + e) * stride));
    }
#pragma unroll
    for (int j = 0; j < kPrefetchX; ++j) {
        const int x = sl + j * SL;
        add(x < n_x ? weight(n_own + x) : 0.f, prx[j]);
    }
    for (int x = sl + kPrefetchX * SL; x < n_x; x += SL) {
        const float w = weight(n_own + x);
        if (w != 0.f) add(w, *reinterpret_cast<const float4*>(po + entry(n_own + x) * stride));
    }
    red[sl * CG + cg] = acc;
    // every thread of a slice holds the same weight sum z; column group 0 publishes it
    if (cg == 0) s_zs[sl] = z;
    __syncthreads();
    if (sl == 0) {
        float4 t = red[cg];
        for (int k = 1; k < SL; ++k) {
            const float4 u = red[k * CG + cg];
            t.x += u.x; t.y += u.y; t.z += u.z; t.w += u.w;
        }
        const float wa = (la == -INFINITY) ? 0.f : __expf(la - m);
        if (wa != 0.f) { t.x += wa * fold.x; t.y += wa * fold.y; t.z += wa * fold.z; t.w += wa * fold.w; }
        float zt = wa;
        for (int k = 0; k < SL; ++k) zt += s_zs[k];      // fixed order: results are reproducible bit for bit
        const float inv = 1.f / zt;
        t.x *= inv; t.y *= inv; t.z *= inv; t.w *= inv;
        *reinterpret_cast<float4*>(oo + cg * 4) = t;
        if (cg == 0 && col0 == 0) p.out_lse[wid] = m + logf(zt);
    }
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
    const PartGeom pg = part_geom(a.kind, a.n_q_heads, a.n_kv_heads);
    ReduceParams p;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.rg_span_start = a.rg_span_start;
    p.acc_o = a.acc_o; p.acc_lse = a.acc_lse; p.out_o = a.out_o; p.out_lse = a.out_lse;
    p.Hq = a.n_q_heads; p.dv = a.dim_v;
    p.G = a.kind == 1 ? a.n_q_heads : a.n_q_heads / a.n_kv_heads;
    p.n_hg = (p.G + 15) / 16;
    p.n_gh = pg.n_gh; p.RG = pg.rows_per_group; p.NW = a.parts_per_span;
    p.dvl = a.dim_v > 128 && a.dim_v % 128 == 0 ? 128 : a.dim_v;
    p.CS = a.dim_v / p.dvl;
    if (p.dvl % 4 != 0 || p.dvl / 4 > 128 || 128 % (p.dvl / 4) != 0) return cudaErrorInvalidValue;
    p.extra_count = a.steal_lists; p.extra_list = a.steal_lists ? a.steal_lists + a.n_rows * a.n_gh : nullptr; p.n_spans = a.n_spans;
    p.clear = a.steal_clear; p.clear_words = a.steal_clear ? a.steal_clear_words : 0;
    // one wave of 256-thread CTAs holds 148 x 5 of them; beyond that, and when a slab leaves at least two entry slices, halve the CTAs
    const bool narrow = int64_t(total) * p.CS > 148 * 5 && p.dvl <= 256;
    const int threads = narrow ? 128 : 256;
    const size_t smem = size_t(threads) * sizeof(float4);
    if (p.extra_count) {
        if (narrow) return launch_ordered(!a.plain_launch, split_reduce_kernel<true, 128>, total * p.CS, threads, smem, s, p);
        return launch_ordered(!a.plain_launch, split_reduce_kernel<true, 256>, total * p.CS, threads, smem, s, p);
    }
    if (narrow) return launch_ordered(!a.plain_launch, split_reduce_kernel<false, 128>, total * p.CS, threads, smem, s, p);
    return launch_ordered(!a.plain_launch, split_reduce_kernel<false, 256>, total * p.CS, threads, smem, s, p);
}

cudaError_t launch_merge(const MergeLaunch& m, cudaStream_t s) {
    if (m.n_rows <= 0) return cudaSuccess;
    const int grid = (m.n_rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
    merge_kernel<<<grid, kWarpsPerBlock * 32, 0, s>>>(m);
    return cudaGetLastError();
}

}  // namespace ipkvi

