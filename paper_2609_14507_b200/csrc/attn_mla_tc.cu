// GPU-side decode attention over the GPU-resident share (Sec. 5.1), compressed-latent (MLA) variant on the
// fifth-generation tensor cores: tcgen05.mma issued by one thread, operands read from shared memory through
// matrix descriptors, accumulators in tensor memory (TMEM).
//
// Same work decomposition and data path as the mma.sync version (persistent split-K, one CTA per SM, the
// producer warp streams 64-token tiles of 73 728 bytes into a 2-stage ring with bulk asynchronous copies), but
// the two contractions no longer run in the warps' instruction streams:
//   S^T[64 tokens x 16 heads] = K_tile[64 x 576] . Q^T      36 MMAs (M=64, N=16, K=16), A = the tile as it lies
//                                                            (K-major, 128-byte swizzle = the TILE block layout),
//                                                            B = the query tile, re-laid in the same layout
//   O^T[512 x 16 heads]      += V^T[512 x 64] . P^T[64 x 16] 4 x 4 MMAs (M=128, N=16, K=16) for p_hi and again for
//                                                            p_lo; A = the first eight panels of the SAME tile read
//                                                            MN-major, B = the weights written by the softmax warps
// Roles: warps 0..3 softmax / rescale / epilogue (they own TMEM lane quadrants 0..3), warp 4 producer, warp 5
// MMA issuer.  The MMA warp issues the scores of tile i+1 before the output product of tile i, so the tensor
// core works on the next scores while the softmax warps handle the current ones.  The running maximum is only
// moved when a row's maximum grows by more than 2^8 (the weights stay below 2^8, exact in bf16 hi+lo), so the
// O accumulators in TMEM are rescaled rarely.
//
// Status: correct (same parity tests as the default kernel) but NOT the default. With only 16 heads the MMAs are
// skinny (N = 16): measured on B200 each score MMA costs about 160 cycles and each output MMA about 70, i.e. 4.1 us
// of tensor-core time per 64-token tile against a 1.7 us HBM budget (300 us per 0.725 GB launch against 122 us for
// the mma.sync kernel). It is selected with the environment variable IPKV_MLA_TC=1 and kept as the starting point
// for a formulation with wider MMAs.
#include <cuda_bf16.h>

#include "kernels.h"
#include "ptx.cuh"

namespace ipkvi {

namespace {

constexpr int kDqk = 576, kDv = 512;
constexpr int kPanels = kDqk / 64;
constexpr int kSoftmaxWarps = 4;
constexpr int kThreads = 6 * 32;
constexpr int kStages = 2;
constexpr int kStageBytes = kTileTokens * kDqk * 2;          // 73 728
constexpr int kQBytes = kPanels * 16 * 128;                  // query tile as a K-major B operand: [9][16 rows][128 B]
constexpr int kPBytes = 16 * 128;                            // weights as a K-major B operand: [16 rows][128 B]
constexpr int kSPitch = kTileTokens + 4;                     // floats
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;                     // log2 units

constexpr int kOffQ = kStages * kStageBytes;                 // 147 456 (1024-aligned)
constexpr int kOffP = kOffQ + kQBytes;                       // [2 buffers][hi, lo][kPBytes]
constexpr int kOffS = kOffP + 2 * 2 * kPBytes;               // transposed scores [16][kSPitch] fp32
constexpr int kOffAlpha = kOffS + 16 * kSPitch * 4;          // [16] alpha, [16] m, [16] l
constexpr int kOffBar = kOffAlpha + 3 * 16 * 4;
// barriers: full[2] empty[2] s_full[2] s_empty[2] p_full[2] p_empty[2] o_done q_ready
constexpr int kNumBars = 14;
constexpr int kOffTmem = kOffBar + kNumBars * 8;
constexpr int kSmemTotal = kOffTmem + 16;

constexpr uint32_t kTmemCols = 128;                          // S: 2 x 16 columns, O^T: 4 x 16 columns
constexpr uint32_t kColS = 0, kColO = 32;

constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((16u >> 3) << 17) | ((64u >> 4) << 24);
constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);

struct MlaTcParams {
    const __nv_bfloat16* q;
    const char* bases[kMaxBases];
    const Seg* segs;
    const Span* spans;
    const int32_t* cta_span_start;
    float* part_o;
    float* part_lse;
    uint32_t* status;
    int Hq;
    int bt;
    int64_t block_bytes;
    float scale_log2;
    int win_tail;        // valid tokens in the last tile of runs flagged kSegTailParam
};

// Shared-memory matrix descriptor, 128-byte swizzle. lbo / sbo in bytes.
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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void softmax_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kSoftmaxWarps * 32) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1) attn_mla_tc_kernel(const MlaTcParams p) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t bar0 = s_base + kOffBar;
    const uint32_t b_full = bar0, b_empty = bar0 + 16, b_sfull = bar0 + 32, b_sempty = bar0 + 48, b_pfull = bar0 + 64,
                   b_pempty = bar0 + 80, b_odone = bar0 + 96, b_qready = bar0 + 104;
    float* sS = reinterpret_cast<float*>(smem + kOffS);
    float* s_alpha = reinterpret_cast<float*>(smem + kOffAlpha);
    float* s_m = s_alpha + 16;
    float* s_l = s_alpha + 32;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + kOffTmem);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int span_begin = p.cta_span_start[blockIdx.x], span_end = p.cta_span_start[blockIdx.x + 1];

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(b_full + 8 * s, 1);
            ptx::mbar_init(b_empty + 8 * s, 1);
            ptx::mbar_init(b_sfull + 8 * s, 1);
            ptx::mbar_init(b_sempty + 8 * s, kSoftmaxWarps);
            ptx::mbar_init(b_pfull + 8 * s, kSoftmaxWarps);
            ptx::mbar_init(b_pempty + 8 * s, 1);
        }
        ptx::mbar_init(b_odone, 1);
        ptx::mbar_init(b_qready, kSoftmaxWarps);
        ptx::mbar_fence_init();
    }
    if (warp == 0) {   // one warp allocates the tensor memory for the CTA
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(s_base + kOffTmem), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (p.bt < kTileTokens) {
        for (int c = tid; c < kStages * kStageBytes / 16; c += kThreads) reinterpret_cast<uint4*>(smem)[c] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    bool ok = true;
    int it = 0;                      // tiles processed so far by this CTA

    if (warp == 4) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t pol = ptx::l2_evict_first_policy();
            for (int sn = span_begin; sn < span_end && ok; ++sn) {
                const Span span = p.spans[sn];
                Seg seg = p.segs[span.seg];
                if (seg.base_id & kSegTailParam) seg.n_tokens += p.win_tail - kTileTokens;
                const char* seg_base = p.bases[seg.base_id & kSegBaseMask] + seg.off;
                for (int i = 0; i < span.ntiles; ++i, ++it) {
                    const int st = it & 1;
                    if (it >= kStages && !ptx::mbar_wait(b_empty + 8 * st, ((it >> 1) - 1) & 1)) { ok = false; break; }
                    const int64_t t0 = int64_t(span.tile0 + i) * kTileTokens;
                    const uint32_t dst = s_base + st * kStageBytes;
                    const uint32_t bar = b_full + 8 * st;
                    if (p.bt >= kTileTokens) {
                        const int64_t blk = t0 / p.bt;
                        const int r0 = int(t0 - blk * p.bt);
                        const char* src = seg_base + blk * p.block_bytes;
                        ptx::mbar_expect_tx(bar, kStageBytes);
                        if (p.bt == kTileTokens) {
                            ptx::bulk_g2s_hint(dst, src, kStageBytes, bar, pol);
                        } else {
#pragma unroll
                            for (int pn = 0; pn < kPanels; ++pn)
                                ptx::bulk_g2s_hint(dst + pn * 8192, src + int64_t(pn) * p.bt * 128 + int64_t(r0) * 128, 8192, bar, pol);
                        }
                    } else {
                        const int nsub = kTileTokens / p.bt;
                        const int64_t blk0 = t0 / p.bt;
                        int live = 0;
                        for (int j = 0; j < nsub; ++j) live += ((blk0 + j) * p.bt < seg.n_tokens);
                        const uint32_t sub_bytes = uint32_t(p.bt) * 128;
                        ptx::mbar_expect_tx(bar, uint32_t(live) * sub_bytes * kPanels);
                        for (int j = 0; j < live; ++j) {
                            const char* src = seg_base + (blk0 + j) * p.block_bytes;
#pragma unroll
                            for (int pn = 0; pn < kPanels; ++pn)
                                ptx::bulk_g2s_hint(dst + pn * 8192 + j * sub_bytes, src + int64_t(pn) * sub_bytes, sub_bytes, bar, pol);
                        }
                    }
                }
            }
            const int first_pending = it > kStages ? it - kStages : 0;
            bool landed = true;
            for (int i = first_pending; i < it; ++i)
                if (!ptx::mbar_wait(b_full + 8 * (i & 1), (i >> 1) & 1)) landed = false;
            if (!ok) atomicOr(p.status, kStatusNoFreeStage);
            if (!landed) atomicOr(p.status, kStatusCopyNotLanded);
        }
    } else if (warp == 5) {
        // ---------------- MMA issuer (one thread) ----------------
        if (lane == 0) {
            auto issue_scores = [&](int tile_it) {
                const int st = tile_it & 1, sb = tile_it & 1;
                if (ok && !ptx::mbar_wait(b_full + 8 * st, (tile_it >> 1) & 1)) ok = false;
                if (tile_it >= 2 && ok && !ptx::mbar_wait(b_sempty + 8 * sb, ((tile_it >> 1) - 1) & 1)) ok = false;
                tc_fence_after();
                if (ok) {
                    const uint32_t kb = s_base + st * kStageBytes, qb = s_base + kOffQ;
#pragma unroll 4
                    for (int j = 0; j < 36; ++j) {
                        const uint64_t a = smem_desc(kb + (j >> 2) * 8192 + (j & 3) * 32, 16, 1024);
                        const uint64_t b = smem_desc(qb + (j >> 2) * 2048 + (j & 3) * 32, 16, 1024);
                        umma(tmem + kColS + sb * 16, a, b, kIdescS, j > 0);
                    }
                }
                umma_commit(b_sfull + 8 * sb);
            };
            int span_no = 0;
            for (int sn = span_begin; sn < span_end; ++sn, ++span_no) {
                const Span span = p.spans[sn];
                if (ok && !ptx::mbar_wait(b_qready, span_no & 1)) ok = false;      // the softmax warps laid out this span's queries
                issue_scores(it);
                for (int i = 0; i < span.ntiles; ++i, ++it) {
                    const int st = it & 1, pb = it & 1;
                    if (i + 1 < span.ntiles) issue_scores(it + 1);                 // next scores before this tile's output product
                    if (ok && !ptx::mbar_wait(b_pfull + 8 * pb, (it >> 1) & 1)) ok = false;
                    tc_fence_after();
                    if (ok) {
                        const uint32_t vb = s_base + st * kStageBytes;
#pragma unroll
                        for (int half = 0; half < 2; ++half) {                     // p_hi, then p_lo
                            const uint32_t pbuf = s_base + kOffP + (pb * 2 + half) * kPBytes;
#pragma unroll
                            for (int c = 0; c < 4; ++c)
#pragma unroll
                                for (int kk = 0; kk < 4; ++kk) {
                                    const uint64_t a = smem_desc(vb + (2 * c) * 8192 + kk * 2048, 8192, 1024);
                                    const uint64_t b = smem_desc(pbuf + kk * 32, 16, 1024);
                                    umma(tmem + kColO + c * 16, a, b, kIdescPV, (i > 0) | (half > 0) | (kk > 0));
                                }
                        }
                    }
                    umma_commit(b_empty + 8 * st);       // the stage may be refilled once these MMAs have read it
                    umma_commit(b_pempty + 8 * pb);
                    umma_commit(b_odone);
                }
            }
            if (!ok) atomicOr(p.status, kStatusNoTile);
        }
    } else {
        // ---------------- softmax / rescale / epilogue warps (TMEM lane quadrant = warp) ----------------
        const int srow = tid >> 3, cchunk = tid & 7, stok = cchunk * 8;     // softmax ownership: row, 8 tokens
        const uint32_t lane_base = uint32_t(32 * warp) << 16;
        int span_no = 0;
        for (int sn = span_begin; sn < span_end; ++sn, ++span_no) {
            const Span span = p.spans[sn];
            Seg seg = p.segs[span.seg];
            if (seg.base_id & kSegTailParam) seg.n_tokens += p.win_tail - kTileTokens;
            const int head0 = span.gh * 16;
            const int n_heads = min(16, p.Hq - head0);
            // query tile -> K-major swizzled operand [9 panels][16 rows][128 B]
            for (int c = tid; c < 16 * 72; c += kSoftmaxWarps * 32) {
                const int row = c / 72, ch = c - row * 72;
                uint4 val = make_uint4(0, 0, 0, 0);
                if (row < n_heads) val = __ldg(reinterpret_cast<const uint4*>(p.q + (int64_t(span.row) * p.Hq + head0 + row) * kDqk + ch * 8));
                *reinterpret_cast<uint4*>(smem + kOffQ + (ch >> 3) * 2048 + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) = val;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(b_qready);
            float m_ref = -INFINITY, l_run = 0.f;

            for (int i = 0; i < span.ntiles; ++i, ++it) {
                const int sb = it & 1, pb = it & 1;
                const int64_t t0 = int64_t(span.tile0 + i) * kTileTokens;
                const int64_t left = int64_t(seg.n_tokens) - t0;
                const int n_valid = left < kTileTokens ? int(left) : kTileTokens;
                // 1. scores of the tile: TMEM -> registers -> transposed into shared memory [head][token]
                if (ok && !ptx::mbar_wait(b_sfull + 8 * sb, (it >> 1) & 1)) ok = false;
                tc_fence_after();
                {
                    uint32_t r[16];
                    tmem_ld16(tmem + lane_base + kColS + sb * 16, r);     // lanes 0..15 of the quadrant hold tokens 16 warp + lane
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(b_sempty + 8 * sb);
                    if (lane < 16) {
#pragma unroll
                        for (int h = 0; h < 16; ++h) sS[h * kSPitch + 16 * warp + lane] = __uint_as_float(r[h]);
                    }
                }
                softmax_barrier();
                // 2. online softmax of row srow over its 8 tokens (8 threads per row)
                float sv[8];
                {
                    const float4 a0 = *reinterpret_cast<const float4*>(sS + srow * kSPitch + stok);
                    const float4 a1 = *reinterpret_cast<const float4*>(sS + srow * kSPitch + stok + 4);
                    sv[0] = a0.x; sv[1] = a0.y; sv[2] = a0.z; sv[3] = a0.w; sv[4] = a1.x; sv[5] = a1.y; sv[6] = a1.z; sv[7] = a1.w;
                }
                float mx = -INFINITY;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    sv[j] = (stok + j < n_valid) ? sv[j] * p.scale_log2 : -INFINITY;
                    mx = fmaxf(mx, sv[j]);
                }
#pragma unroll
                for (int d = 1; d < 8; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
                float alpha = 1.f;
                if (mx > m_ref + kRescaleThreshold || m_ref == -INFINITY) {       // move the reference maximum (rarely)
                    const float mn = fmaxf(m_ref, mx);
                    if (mn != -INFINITY) { alpha = ptx::ex2(m_ref - mn); m_ref = mn; }
                }
                const float ms = (m_ref == -INFINITY) ? 0.f : m_ref;
                uint32_t hi[4], lo[4];
                float psum = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float pa = ptx::ex2(sv[2 * j] - ms), pc = ptx::ex2(sv[2 * j + 1] - ms);
                    psum += pa + pc;
                    hi[j] = ptx::pack_bf16(pa, pc);
                    lo[j] = ptx::pack_bf16(pa - ptx::bf16_lo(hi[j]), pc - ptx::bf16_hi(hi[j]));
                }
                l_run = l_run * alpha + psum;
                if (it >= 2 && ok && !ptx::mbar_wait(b_pempty + 8 * pb, ((it >> 1) - 1) & 1)) ok = false;   // weights buffer drained
                {
                    unsigned char* ph = smem + kOffP + (pb * 2) * kPBytes + srow * 128 + ((cchunk ^ (srow & 7)) << 4);
                    *reinterpret_cast<uint4*>(ph) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                    *reinterpret_cast<uint4*>(ph + kPBytes) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                }
                if (cchunk == 0) s_alpha[srow] = alpha;
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                softmax_barrier();
                // 3. rescale the O^T accumulators in TMEM when some row moved its reference maximum
                if (i > 0) {
                    // Every phase of o_done is waited for, in order: a parity wait only tells the current phase from
                    // the previous one, so skipping a phase could let the end-of-span wait pass early.
                    if (ok && !ptx::mbar_wait(b_odone, (it - 1) & 1)) ok = false;         // the previous output product has landed
                    float al[16];
                    bool any = false;
#pragma unroll
                    for (int h = 0; h < 16; ++h) { al[h] = s_alpha[h]; any |= (al[h] != 1.f); }
                    if (any) {
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t r[16];
                            tmem_ld16(tmem + lane_base + kColO + c * 16, r);
#pragma unroll
                            for (int h = 0; h < 16; ++h) r[h] = __float_as_uint(__uint_as_float(r[h]) * al[h]);
                            tmem_st16(tmem + lane_base + kColO + c * 16, r);
                        }
                        tc_fence_before();
                    }
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(b_pfull + 8 * pb);
                softmax_barrier();          // s_alpha and sS are rewritten by the next tile
            }
            // ---- end of span: normalise O^T with the row sums and write the partial ----
#pragma unroll
            for (int d = 1; d < 8; d <<= 1) l_run += __shfl_xor_sync(0xffffffffu, l_run, d);
            if (cchunk == 0) { s_m[srow] = m_ref; s_l[srow] = l_run; }
            softmax_barrier();
            if (ok && !ptx::mbar_wait(b_odone, (it - 1) & 1)) ok = false;
            tc_fence_after();
            {
                float inv[16];
#pragma unroll
                for (int h = 0; h < 16; ++h) { const float L = s_l[h]; inv[h] = L > 0.f ? 1.f / L : 0.f; }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[16];
                    tmem_ld16(tmem + lane_base + kColO + c * 16, r);
                    float* dst = p.part_o + int64_t(sn) * 16 * kDv + c * 128 + 32 * warp + lane;
#pragma unroll
                    for (int h = 0; h < 16; ++h)
                        if (h < n_heads) dst[h * kDv] = __uint_as_float(r[h]) * inv[h];
                }
                tc_fence_before();
                if (tid < n_heads) {
                    const float M = s_m[tid], L = s_l[tid];
                    p.part_lse[int64_t(sn) * 16 + tid] = (M == -INFINITY) ? -INFINITY : (M + log2f(L)) * kLn2;
                }
            }
            softmax_barrier();
        }
        if (!ok && lane == 0) atomicOr(p.status, kStatusNoTile);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

cudaError_t launch_attend_mla_tc(const AttnLaunch& a, cudaStream_t s) {
    if (a.n_ctas <= 0 || a.n_spans <= 0) return cudaSuccess;
    if (a.dim_qk != kDqk || a.dim_v != kDv || a.n_kv_heads != 1) return cudaErrorInvalidValue;
    MlaTcParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    for (int i = 0; i < kMaxBases; ++i) p.bases[i] = a.bases[i];
    p.segs = a.segs; p.spans = a.spans; p.cta_span_start = a.cta_span_start;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.status = a.status;
    p.Hq = a.n_q_heads;
    p.bt = a.bt;
    p.block_bytes = int64_t(a.bt) * kDqk * 2;
    p.scale_log2 = a.scale * kLog2e;
    p.win_tail = a.win_tail;
    const int smem = kSmemTotal + 1024;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(attn_mla_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    attn_mla_tc_kernel<<<a.n_ctas, kThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace ipkvi
