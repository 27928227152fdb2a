// GPU-side decode attention over the GPU-resident share of each sequence (Sec. 5.1): for every
// (sequence, query head) the partial output and log-sum-exp over the D-window and the loaded part of
// the pinned region.  The paper names no GPU kernel; this one is written for sm_100a.
//
// Grouped-query variant, dim_qk = dim_v = D in {64, 128}.
//
// Work decomposition (split-K along the sequence): one CTA per (item, KV head[, group of 16 query
// heads]); an item is a range of 64-token tiles of one run of blocks.  The G query heads that share the
// KV head are packed into the M dimension of the tensor-core MMA, so one K/V read serves the group.
//
// Data path: a producer warp streams K and V tiles of the head (contiguous in the TILE block layout)
// into a ring of shared-memory stages with bulk asynchronous copies that complete on mbarriers; four
// consumer warps each own 16 tokens of every tile and keep a private online-softmax state
// (fp32 running max / sum, fp32 output accumulators in registers), so no CTA-wide synchronisation is
// needed per tile.  The four states are merged once at the end through shared memory and the
// normalised partial (O, natural-log LSE) of the item is written out.
//
// HBM traffic per KV token: bytes_per_token / n_kv_heads per CTA row, read exactly once.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace ipkvi {

namespace {

constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct GqaParams {
    const __nv_bfloat16* q;
    const char* bases[kMaxBases];
    const Seg* segs;
    const Item* items;
    float* part_o;
    float* part_lse;
    uint32_t* status;
    int Hq, Hkv, G, n_hg;
    int bt;
    int64_t head_bytes, block_bytes;
    float scale_log2;
};

template <int D, int STAGES>
struct SmemPlan {
    static constexpr int kPlane = D * 128;               // bytes of a 64-token K (or V) tile
    static constexpr int kStage = 2 * kPlane;
    static constexpr int kQPitch = D * 2 + 16;           // padded row pitch of the Q tile
    static constexpr int kStagesBytes = STAGES * kStage;
    static constexpr int kQOff = kStagesBytes;
    static constexpr int kBarOff = kQOff + 16 * kQPitch;
    static constexpr int kTotal = kBarOff + 2 * STAGES * 8;
    // cross-warp merge area, overlaid on the stage ring once the pipeline has drained
    static constexpr int kMergeO = 0;                                        // [warps][16][D] fp32
    static constexpr int kMergeM = kConsumerWarps * 16 * D * 4;              // [warps][16] fp32
    static constexpr int kMergeL = kMergeM + kConsumerWarps * 16 * 4;
    static_assert(kMergeL + kConsumerWarps * 16 * 4 <= kStagesBytes + 16 * kQPitch, "merge area must fit");
};

template <int D, int STAGES, bool DUP>
__global__ void __launch_bounds__(kThreads) attn_gqa_kernel(const GqaParams p) {
    using SP = SmemPlan<D, STAGES>;
    extern __shared__ unsigned char smem_dyn[];
    // align the ring to 1024 bytes so that the 128-byte chunk swizzle maps onto distinct banks
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_q = s_base + SP::kQOff;
    const uint32_t s_full = s_base + SP::kBarOff;
    const uint32_t s_empty = s_full + STAGES * 8;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const Item item = p.items[blockIdx.x];
    const Seg seg = p.segs[item.seg];
    const int g = blockIdx.y / p.n_hg, hg = blockIdx.y - g * p.n_hg;
    const int head0 = g * p.G + hg * 16;                       // first query head of this CTA
    const int n_heads = min(16, p.G - hg * 16);

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(s_full + 8 * s, 1);
            ptx::mbar_init(s_empty + 8 * s, kConsumerWarps);
        }
        ptx::mbar_fence_init();
    }
    // Q tile: 16 rows (query heads of the group, zero beyond n_heads) x D bf16
    for (int c = tid; c < 16 * (D / 8); c += kThreads) {
        const int r = c / (D / 8), ch = c - r * (D / 8);
        uint4 val = make_uint4(0, 0, 0, 0);
        const int hr = DUP ? (r & 7) : r;                  // DUP: rows 8..15 repeat rows 0..7
        if (hr < n_heads)
            val = *reinterpret_cast<const uint4*>(p.q + (int64_t(item.row) * p.Hq + head0 + hr) * D + ch * 8);
        *reinterpret_cast<uint4*>(smem + SP::kQOff + r * SP::kQPitch + ch * 16) = val;
    }
    if (p.bt < kTileTokens) {
        // tiles spanning several small blocks may leave rows unwritten at the end of a run: make them finite
        for (int c = tid; c < SP::kStagesBytes / 16; c += kThreads)
            reinterpret_cast<uint4*>(smem)[c] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    const char* seg_base = p.bases[seg.base_id] + seg.off;
    bool ok = true;

    if (warp == kConsumerWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            for (int i = 0; i < item.ntiles; ++i) {
                const int st = i % STAGES;
                if (i >= STAGES && !ptx::mbar_wait(s_empty + 8 * st, ((i / STAGES) - 1) & 1)) { ok = false; break; }
                const int64_t t0 = int64_t(item.tile0 + i) * kTileTokens;
                const uint32_t dst = s_base + st * SP::kStage;
                const uint32_t bar = s_full + 8 * st;
                if (p.bt >= kTileTokens) {
                    const int64_t blk = t0 / p.bt;
                    const int r0 = int(t0 - blk * p.bt);
                    const char* src = seg_base + blk * p.block_bytes + int64_t(g) * p.head_bytes;
                    ptx::mbar_expect_tx(bar, SP::kStage);
                    if (p.bt == kTileTokens) {
                        ptx::bulk_g2s(dst, src, SP::kStage, bar);          // K plane and V plane are adjacent
                    } else {
                        const int64_t kplane = int64_t(p.bt) * D * 2;
#pragma unroll
                        for (int pn = 0; pn < D / 64; ++pn) {
                            const char* s0 = src + int64_t(pn) * p.bt * 128 + int64_t(r0) * 128;
                            ptx::bulk_g2s(dst + pn * 8192, s0, 8192, bar);
                            ptx::bulk_g2s(dst + SP::kPlane + pn * 8192, s0 + kplane, 8192, bar);
                        }
                    }
                } else {
                    const int nsub = kTileTokens / p.bt;
                    const int64_t blk0 = t0 / p.bt;
                    int live = 0;
                    for (int j = 0; j < nsub; ++j) live += ((blk0 + j) * p.bt < seg.n_tokens);
                    const uint32_t sub_bytes = uint32_t(p.bt) * 128;
                    ptx::mbar_expect_tx(bar, uint32_t(live) * sub_bytes * 2 * (D / 64));
                    const int64_t kplane = int64_t(p.bt) * D * 2;
                    for (int j = 0; j < live; ++j) {
                        const char* src = seg_base + (blk0 + j) * p.block_bytes + int64_t(g) * p.head_bytes;
#pragma unroll
                        for (int pn = 0; pn < D / 64; ++pn) {
                            ptx::bulk_g2s(dst + pn * 8192 + j * sub_bytes, src + int64_t(pn) * sub_bytes, sub_bytes, bar);
                            ptx::bulk_g2s(dst + SP::kPlane + pn * 8192 + j * sub_bytes, src + kplane + int64_t(pn) * sub_bytes, sub_bytes, bar);
                        }
                    }
                }
            }
            // do not leave the CTA while copies of ours may still be in flight
            const int first_pending = item.ntiles > STAGES ? item.ntiles - STAGES : 0;
            for (int i = first_pending; i < item.ntiles; ++i)
                if (!ptx::mbar_wait(s_full + 8 * (i % STAGES), (i / STAGES) & 1)) ok = false;
            if (!ok) atomicOr(p.status, 1u);
        }
        __syncwarp();
        __syncthreads();   // matches the consumers' barrier before the merge
        __syncthreads();   // ... and the one after the merge area has been written
        return;
    }

    // ---------------- consumers ----------------
    // The softmax weights are split into a bf16 head and a bf16 remainder (p = p_hi + p_lo, about 16
    // significant bits) before the P.V product, so that the output error stays at fp32-accumulation level.
    //   DUP (at most 8 query heads in the CTA): query rows 8..15 duplicate rows 0..7; MMA rows 0..7 carry
    //   p_hi and rows 8..15 carry p_lo, so the remainder costs no extra tensor-core work.
    //   otherwise: two P.V products per tile.
    uint32_t qa[D / 16][4];
    {
        const int mi = lane >> 3, r = lane & 7;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            const int row = (mi & 1) * 8 + r, chunk = ks * 2 + (mi >> 1);
            ptx::ldmatrix_x4(s_q + row * SP::kQPitch + chunk * 16, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
        }
    }
    float o[D / 8][4];
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    const int mi = lane >> 3, r8 = lane & 7;
    // per-lane ldmatrix row offsets inside a stage (token index inside the tile is warp*16 + ...)
    const int tokK = warp * 16 + (mi >> 1) * 8 + r8;     // K: matrices 0,1 tokens 0-7; 2,3 tokens 8-15
    const int tokV = warp * 16 + (mi & 1) * 8 + r8;      // V: matrices 0,2 tokens 0-7; 1,3 tokens 8-15
    const int tcol = warp * 16 + 2 * (lane & 3);         // token of accumulator element 0 (n-tile 0)

    for (int i = 0; i < item.ntiles; ++i) {
        const int st = i % STAGES;
        if (!ptx::mbar_wait(s_full + 8 * st, (i / STAGES) & 1)) { ok = false; break; }
        const int64_t t0 = int64_t(item.tile0 + i) * kTileTokens;
        const int64_t left = int64_t(seg.n_tokens) - t0;
        const int n_valid = left < kTileTokens ? int(left) : kTileTokens;
        if (warp * 16 < n_valid) {
            const uint32_t kb = s_base + st * SP::kStage;
            const uint32_t vb = kb + SP::kPlane;
            float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const int chunk = ks * 2 + (mi & 1);
                uint32_t b0, b1, b2, b3;
                ptx::ldmatrix_x4(kb + (chunk >> 3) * 8192 + tokK * 128 + (((chunk & 7) ^ r8) << 4), b0, b1, b2, b3);
                ptx::mma_bf16(s[0], qa[ks], b0, b1);
                ptx::mma_bf16(s[1], qa[ks], b2, b3);
            }
            // scale, mask the ragged tail, online softmax in the log2 domain
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int j = 0; j < (DUP ? 2 : 4); ++j) {
                    const int t = tcol + nt * 8 + (j & 1);
                    s[nt][j] = (t < n_valid) ? s[nt][j] * p.scale_log2 : -INFINITY;
                }
            float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
            const float mn0 = fmaxf(m0, mx0);
            const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0;
            const float a0 = ptx::ex2(m0 - ms0);
            m0 = mn0;
            float a1 = a0, ms1 = ms0;
            if (!DUP) {
                float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                const float mn1 = fmaxf(m1, mx1);
                ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
                a1 = ptx::ex2(m1 - ms1);
                m1 = mn1;
            }
            float pr[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                pr[nt][0] = ptx::ex2(s[nt][0] - ms0);
                pr[nt][1] = ptx::ex2(s[nt][1] - ms0);
                if (!DUP) {
                    pr[nt][2] = ptx::ex2(s[nt][2] - ms1);
                    pr[nt][3] = ptx::ex2(s[nt][3] - ms1);
                }
            }
            l0 = l0 * a0 + (pr[0][0] + pr[0][1] + pr[1][0] + pr[1][1]);
            if (!DUP) l1 = l1 * a1 + (pr[0][2] + pr[0][3] + pr[1][2] + pr[1][3]);
            if (__any_sync(0xffffffffu, (a0 != 1.f) | (a1 != 1.f))) {
#pragma unroll
                for (int nt = 0; nt < D / 8; ++nt) { o[nt][0] *= a0; o[nt][1] *= a0; o[nt][2] *= a1; o[nt][3] *= a1; }
            }
            uint32_t pa[4], pb[4];
            if (DUP) {
                pa[0] = ptx::pack_bf16(pr[0][0], pr[0][1]);
                pa[2] = ptx::pack_bf16(pr[1][0], pr[1][1]);
                pa[1] = ptx::pack_bf16(pr[0][0] - ptx::bf16_lo(pa[0]), pr[0][1] - ptx::bf16_hi(pa[0]));
                pa[3] = ptx::pack_bf16(pr[1][0] - ptx::bf16_lo(pa[2]), pr[1][1] - ptx::bf16_hi(pa[2]));
            } else {
                pa[0] = ptx::pack_bf16(pr[0][0], pr[0][1]);
                pa[1] = ptx::pack_bf16(pr[0][2], pr[0][3]);
                pa[2] = ptx::pack_bf16(pr[1][0], pr[1][1]);
                pa[3] = ptx::pack_bf16(pr[1][2], pr[1][3]);
                pb[0] = ptx::pack_bf16(pr[0][0] - ptx::bf16_lo(pa[0]), pr[0][1] - ptx::bf16_hi(pa[0]));
                pb[1] = ptx::pack_bf16(pr[0][2] - ptx::bf16_lo(pa[1]), pr[0][3] - ptx::bf16_hi(pa[1]));
                pb[2] = ptx::pack_bf16(pr[1][0] - ptx::bf16_lo(pa[2]), pr[1][1] - ptx::bf16_hi(pa[2]));
                pb[3] = ptx::pack_bf16(pr[1][2] - ptx::bf16_lo(pa[3]), pr[1][3] - ptx::bf16_hi(pa[3]));
            }
#pragma unroll
            for (int jj = 0; jj < D / 16; ++jj) {
                const int chunk = 2 * jj + (mi >> 1);
                uint32_t b0, b1, b2, b3;
                ptx::ldmatrix_x4_trans(vb + (chunk >> 3) * 8192 + tokV * 128 + (((chunk & 7) ^ r8) << 4), b0, b1, b2, b3);
                ptx::mma_bf16(o[2 * jj], pa, b0, b1);
                ptx::mma_bf16(o[2 * jj + 1], pa, b2, b3);
                if (!DUP) {
                    ptx::mma_bf16(o[2 * jj], pb, b0, b1);
                    ptx::mma_bf16(o[2 * jj + 1], pb, b2, b3);
                }
            }
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(s_empty + 8 * st);
    }
    if (!ok && lane == 0) atomicOr(p.status, 1u);

    // row sums are per-thread partials so far: finish them across the quad
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    __syncthreads();   // every warp is done with the stage ring; the producer has seen all copies land
    float* mo = reinterpret_cast<float*>(smem + SP::kMergeO);
    float* mm = reinterpret_cast<float*>(smem + SP::kMergeM);
    float* ml = reinterpret_cast<float*>(smem + SP::kMergeL);
    {
        const int r0 = lane >> 2, c0 = 2 * (lane & 3);
        float* w = mo + warp * 16 * D;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            if (DUP) {
                *reinterpret_cast<float2*>(w + r0 * D + nt * 8 + c0) = make_float2(o[nt][0] + o[nt][2], o[nt][1] + o[nt][3]);
            } else {
                *reinterpret_cast<float2*>(w + r0 * D + nt * 8 + c0) = make_float2(o[nt][0], o[nt][1]);
                *reinterpret_cast<float2*>(w + (r0 + 8) * D + nt * 8 + c0) = make_float2(o[nt][2], o[nt][3]);
            }
        }
        if ((lane & 3) == 0) {
            mm[warp * 16 + r0] = m0; ml[warp * 16 + r0] = l0;
            if (!DUP) { mm[warp * 16 + r0 + 8] = m1; ml[warp * 16 + r0 + 8] = l1; }
        }
    }
    __syncthreads();
    for (int idx = tid; idx < n_heads * D; idx += kConsumerWarps * 32) {
        const int row = idx / D, col = idx - row * D;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, mm[w * 16 + row]);
        float acc = 0.f, L = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) {
                const float f = ptx::ex2(mm[w * 16 + row] - M);
                L += ml[w * 16 + row] * f;
                acc += mo[(w * 16 + row) * D + col] * f;
            }
            acc /= L;
        }
        const int64_t prow = int64_t(blockIdx.x) * p.Hq + head0 + row;
        p.part_o[prow * D + col] = acc;
        if (col == 0) p.part_lse[prow] = (M == -INFINITY) ? -INFINITY : (M + log2f(L)) * kLn2;
    }
}

template <int D, int STAGES, bool DUP>
cudaError_t launch_gqa(const AttnLaunch& a, cudaStream_t s) {
    using SP = SmemPlan<D, STAGES>;
    GqaParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    for (int i = 0; i < kMaxBases; ++i) p.bases[i] = a.bases[i];
    p.segs = a.segs; p.items = a.items;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.status = a.status;
    p.Hq = a.n_q_heads; p.Hkv = a.n_kv_heads; p.G = a.n_q_heads / a.n_kv_heads;
    p.n_hg = (p.G + 15) / 16;
    p.bt = a.bt;
    p.head_bytes = int64_t(a.bt) * (a.dim_qk + a.dim_v) * 2;
    p.block_bytes = p.head_bytes * a.n_kv_heads;
    p.scale_log2 = a.scale * kLog2e;
    const int smem = SP::kTotal + 1024;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(attn_gqa_kernel<D, STAGES, DUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    dim3 grid(a.n_items, a.n_kv_heads * p.n_hg);
    attn_gqa_kernel<D, STAGES, DUP><<<grid, kThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attend_gqa(const AttnLaunch& a, cudaStream_t s) {
    if (a.n_items <= 0) return cudaSuccess;
    const bool dup = a.n_q_heads / a.n_kv_heads <= 8;
    if (a.dim_qk == 128 && a.dim_v == 128) return dup ? launch_gqa<128, 3, true>(a, s) : launch_gqa<128, 3, false>(a, s);
    if (a.dim_qk == 64 && a.dim_v == 64) return dup ? launch_gqa<64, 4, true>(a, s) : launch_gqa<64, 4, false>(a, s);
    return cudaErrorInvalidValue;
}

}  // namespace ipkvi
