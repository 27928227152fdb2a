// GPU-side decode attention over the GPU-resident share (Sec. 5.1), compressed-latent (MLA) variant:
// every head of a sequence attends the same cached row [latent 512 | rope 64] per token with an absorbed
// query of width 576, and the value is the row's first 512 columns (Sec. 6.1: the heads share one latent,
// each latent is read from memory once).  The paper's kernel for this case is a CPU kernel; this one is
// written for sm_100a.
//
// Persistent split-K (one CTA per SM, each with an equally long contiguous chunk of the launch's tiles, cut
// into spans where the (row, head group, run) changes): a producer warp streams 64-token tiles (73 728 contiguous
// bytes in the TILE block layout) into a 2-stage shared-memory ring with bulk asynchronous copies that
// complete on mbarriers; the tile is read twice from shared memory — as K (ldmatrix) and as V
// (ldmatrix.trans on the first eight 64-column panels) — and once from HBM.
//
// Eight consumer warps, three phases per tile:
//   1. scores: warp (ds, th) multiplies the 16 query rows with d-slice ds (144 of the 576 columns) of
//      token half th (32 tokens); the query fragments of its slice stay in registers for the whole CTA;
//      partial scores go to shared memory.
//   2. softmax: warp w owns query rows 2w, 2w+1: it sums the four d-slice partials, applies the scale,
//      masks the ragged tail and updates the running max / sum of its rows (fp32, log2 domain); the
//      weights are split p = p_hi + p_lo (two bf16) and written to shared memory with the rescale factor.
//   3. output: warp w owns value columns [64w, 64w+64) (one panel): O = O*alpha + (P_hi + P_lo) V with
//      fp32 accumulators in registers.  The stage goes back to the producer as soon as the tile's last bytes have
//      been read into registers, before the last p_lo products: what bounds this kernel is how long a stage is
//      held (a stage that is computed on is not being refilled), so everything that shortens the hold counts.
// HBM traffic per KV token: 1152 bytes, read exactly once per group of 16 heads.
#include <cuda_bf16.h>

#include <cstdlib>

#include "kernels.h"
#include "launch.cuh"
#include "ptx.cuh"

namespace ipkvi {

namespace {

constexpr int kDqk = 576, kDv = 512;
constexpr int kPanels = kDqk / 64;                 // 9
constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kStages = 2;
constexpr int kStageBytes = kTileTokens * kDqk * 2;          // 73 728
constexpr int kQPitch = kDqk * 2 + 16;                       // 1168
constexpr int kSPitch = kTileTokens + 8;                     // floats; rows 8 banks apart: the phase-1 float2 stores of 8 rows x 8 words spread over all 32 banks
constexpr int kPPitch = kTileTokens * 2 + 16;                // bytes (bf16 row of 64 tokens, padded)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

constexpr int kOffQ = kStages * kStageBytes;                 // 147 456
constexpr int kOffS = kOffQ + 16 * kQPitch;                  // partial scores [4][16][kSPitch] fp32
constexpr int kOffPhi = kOffS + 4 * 16 * kSPitch * 4;
constexpr int kOffPlo = kOffPhi + 16 * kPPitch;
constexpr int kOffAlpha = kOffPlo + 16 * kPPitch;            // [16] fp32 rescale factors, then [16] m, [16] l
constexpr int kOffBar = kOffAlpha + 3 * 16 * 4;
constexpr int kSmemTotal = kOffBar + 2 * kStages * 8;

struct MlaParams {
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
    int64_t base_bytes[kMaxBases];   // bounds-checked build: extent behind every base (0: not checked)
    int64_t part_rows;               // bounds-checked build: rows of partial storage
    int early;           // nonzero: the first copies of ring tiles (2: of window tiles too) need not wait for the previous kernel
};

__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1) attn_mla_kernel(const MlaParams p) {
    extern __shared__ unsigned char smem_dyn[];
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_q = s_base + kOffQ;
    const uint32_t s_phi = s_base + kOffPhi, s_plo = s_base + kOffPlo;
    const uint32_t s_full = s_base + kOffBar, s_empty = s_full + kStages * 8;
    float* sp = reinterpret_cast<float*>(smem + kOffS);
    float* s_alpha = reinterpret_cast<float*>(smem + kOffAlpha);
    float* s_m = s_alpha + 16;
    float* s_l = s_alpha + 32;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int span_begin = p.cta_span_start[blockIdx.x], span_end = p.cta_span_start[blockIdx.x + 1];

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(s_full + 8 * s, 1);
            ptx::mbar_init(s_empty + 8 * s, kConsumerWarps);
        }
        ptx::mbar_fence_init();
    }
    if (p.bt < kTileTokens) {
        for (int c = tid; c < kStages * kStageBytes / 16; c += kThreads) reinterpret_cast<uint4*>(smem)[c] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Everything above may run while the previous kernel of the stream drains (it may be the append that writes this
    // launch's newest token, or the reduce that still reads the partials' scratch).
    // With a host that vouches for the bytes (MlaParams::early) the producer fills the ring first and waits before its
    // first refill or its first window tile; it never signals the dependents itself, so that signal always follows a wait.
    const bool early = p.early != 0;
    if (!(early && warp == kConsumerWarps)) {
        ptx::grid_dependency_wait();
        ptx::grid_launch_dependents();
    }

    bool ok = true;
    int it = 0;                      // tiles streamed so far by this CTA: stage = it % kStages

    if (warp == kConsumerWarps) {
        // ---------------- producer: streams the whole chunk, never pausing at span boundaries ----------------
        if (lane == 0) {
            const uint64_t pol = ptx::l2_evict_first_policy();     // the KV stream is read once: first out of L2
            bool waited = !early;
            for (int sn = span_begin; sn < span_end && ok; ++sn) {
                const Span span = p.spans[sn];
                Seg seg = p.segs[span.seg];
                if (seg.base_id & kSegTailParam) seg.n_tokens += p.win_tail - kTileTokens;
                const char* seg_base = p.bases[seg.base_id & kSegBaseMask] + seg.off;
                const char* chk_lo = p.bases[seg.base_id & kSegBaseMask];       // bounds-checked build: the region the run must lie in
                const int64_t chk_n = p.base_bytes[seg.base_id & kSegBaseMask];
                auto CHK = [&](const char* a, uint32_t bytes) { return ptx::checked_src<kChecked>(a, bytes, chk_lo, chk_n, p.status, kStatusBadIndex); };
                for (int i = 0; i < span.ntiles; ++i, ++it) {
                    if (!waited && (it >= kStages || (p.early < 2 && (seg.base_id & kSegBaseMask) == kSegBaseWindow))) {
                        ptx::grid_dependency_wait();
                        waited = true;
                    }
                    // Everything that can be known before the stage is free is computed before the wait: the time between
                    // the consumers' release and the start of the copy is time in which the stage holds nothing.
                    const int st = it % kStages;
                    const int64_t t0 = int64_t(span.tile0 + i) * kTileTokens;
                    const uint32_t dst = s_base + st * kStageBytes;
                    const uint32_t bar = s_full + 8 * st;
                    const int64_t blk = t0 / p.bt;
                    const char* src = seg_base + blk * p.block_bytes;
                    const int64_t row_off = (t0 - blk * p.bt) * 128;
                    int live = 0;
                    if (p.bt < kTileTokens)
                        for (int j = 0; j < kTileTokens / p.bt; ++j) live += ((blk + j) * p.bt < seg.n_tokens);
                    if (it >= kStages && !ptx::mbar_wait(s_empty + 8 * st, ((it / kStages) - 1) & 1)) { ok = false; break; }
                    if (p.bt == kTileTokens) {
                        ptx::mbar_expect_tx(bar, kStageBytes);
                        ptx::bulk_g2s_hint(dst, CHK(src, kStageBytes), kStageBytes, bar, pol);
                    } else if (p.bt > kTileTokens) {
                        ptx::mbar_expect_tx(bar, kStageBytes);
#pragma unroll
                        for (int pn = 0; pn < kPanels; ++pn)
                            ptx::bulk_g2s_hint(dst + pn * 8192, CHK(src + int64_t(pn) * p.bt * 128 + row_off, 8192), 8192, bar, pol);
                    } else {
                        const uint32_t sub_bytes = uint32_t(p.bt) * 128;
                        ptx::mbar_expect_tx(bar, uint32_t(live) * sub_bytes * kPanels);
                        for (int j = 0; j < live; ++j) {
                            const char* sj = src + j * p.block_bytes;
#pragma unroll
                            for (int pn = 0; pn < kPanels; ++pn)
                                ptx::bulk_g2s_hint(dst + pn * 8192 + j * sub_bytes, CHK(sj + int64_t(pn) * sub_bytes, sub_bytes), sub_bytes, bar, pol);
                        }
                    }
                }
            }
            const int first_pending = it > kStages ? it - kStages : 0;
            bool landed = true;
            for (int i = first_pending; i < it; ++i)
                if (!ptx::mbar_wait(s_full + 8 * (i % kStages), (i / kStages) & 1)) landed = false;
            if (!ok) atomicOr(p.status, kStatusNoFreeStage);
            if (!landed) atomicOr(p.status, kStatusCopyNotLanded);
        }
        return;      // the consumers synchronise among themselves on a named barrier
    }

    // ---------------- consumers ----------------
    const int ds = warp & 3, th = warp >> 2;
    const int mi = lane >> 3, r8 = lane & 7;
    // phase-2 ownership: this lane works on query row `srow`, tokens [stok, stok + 4) of every tile
    const int srow = 2 * warp + (lane >> 4), stok = (lane & 15) * 4;

    for (int sn = span_begin; sn < span_end; ++sn) {
        const Span span = p.spans[sn];
        Seg seg = p.segs[span.seg];
        if (seg.base_id & kSegTailParam) seg.n_tokens += p.win_tail - kTileTokens;
        const int head0 = span.gh * 16;
        const int n_heads = min(16, p.Hq - head0);

        // query tile of the span's head group -> shared memory -> this warp's d-slice fragments
        for (int c = tid; c < 16 * (kDqk / 8); c += kConsumerWarps * 32) {
            const int r = c / (kDqk / 8), ch = c - r * (kDqk / 8);
            uint4 val = make_uint4(0, 0, 0, 0);
            if (r < n_heads) val = __ldg(reinterpret_cast<const uint4*>(p.q + (int64_t(span.row) * p.Hq + head0 + r) * kDqk + ch * 8));
            *reinterpret_cast<uint4*>(smem + kOffQ + r * kQPitch + ch * 16) = val;
        }
        consumer_barrier();
        uint32_t qa[9][4];
#pragma unroll
        for (int ks = 0; ks < 9; ++ks) {
            const int row = (mi & 1) * 8 + r8, chunk = ds * 18 + ks * 2 + (mi >> 1);
            ptx::ldmatrix_x4(s_q + row * kQPitch + chunk * 16, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
        }
        float o[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
        float m_run = -INFINITY, l_run = 0.f;

        for (int i = 0; i < span.ntiles; ++i, ++it) {
            const int st = it % kStages;
            if (ok && !ptx::mbar_wait(s_full + 8 * st, (it / kStages) & 1)) ok = false;   // after a timeout: no more waits, but keep the barriers below matched
            const int64_t t0 = int64_t(span.tile0 + i) * kTileTokens;
            const int64_t left = int64_t(seg.n_tokens) - t0;
            const int n_valid = left < kTileTokens ? int(left) : kTileTokens;
            const uint32_t kb = s_base + st * kStageBytes;

            // ---- phase 1: partial scores of d-slice ds for tokens [32 th, 32 th + 32) ----
            {
                float s[4][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) { s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f; }
#pragma unroll
                for (int ks = 0; ks < 9; ++ks) {
                    const int chunk = ds * 18 + ks * 2 + (mi & 1);
                    const uint32_t col = (chunk >> 3) * 8192 + (((chunk & 7) ^ r8) << 4);
#pragma unroll
                    for (int tg = 0; tg < 2; ++tg) {
                        const int tok = th * 32 + tg * 16 + (mi >> 1) * 8 + r8;
                        uint32_t b0, b1, b2, b3;
                        ptx::ldmatrix_x4(kb + col + tok * 128, b0, b1, b2, b3);
                        ptx::mma_bf16(s[2 * tg], qa[ks], b0, b1);
                        ptx::mma_bf16(s[2 * tg + 1], qa[ks], b2, b3);
                    }
                }
                float* dst = sp + ds * 16 * kSPitch;
                const int r0 = lane >> 2, c0 = th * 32 + 2 * (lane & 3);
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) {
                    *reinterpret_cast<float2*>(dst + r0 * kSPitch + c0 + nt * 8) = make_float2(s[nt][0], s[nt][1]);
                    *reinterpret_cast<float2*>(dst + (r0 + 8) * kSPitch + c0 + nt * 8) = make_float2(s[nt][2], s[nt][3]);
                }
            }
            consumer_barrier();

            // ---- phase 2: softmax bookkeeping for the rows this warp owns ----
            {
                float4 a = *reinterpret_cast<const float4*>(sp + srow * kSPitch + stok);
#pragma unroll
                for (int d = 1; d < 4; ++d) {
                    const float4 b = *reinterpret_cast<const float4*>(sp + (d * 16 + srow) * kSPitch + stok);
                    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                }
                float sv[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) sv[j] = (stok + j < n_valid) ? sv[j] * p.scale_log2 : -INFINITY;
                float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
#pragma unroll
                for (int d = 1; d < 16; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, d));
                const float mn = fmaxf(m_run, mx);
                const float ms = (mn == -INFINITY) ? 0.f : mn;
                const float alpha = ptx::ex2(m_run - ms);
                m_run = mn;
                float pr[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) pr[j] = ptx::ex2(sv[j] - ms);
                l_run = l_run * alpha + (pr[0] + pr[1] + pr[2] + pr[3]);
                const uint32_t h0 = ptx::pack_bf16(pr[0], pr[1]), h1 = ptx::pack_bf16(pr[2], pr[3]);
                const uint32_t l0 = ptx::pack_bf16(pr[0] - ptx::bf16_lo(h0), pr[1] - ptx::bf16_hi(h0));
                const uint32_t l1 = ptx::pack_bf16(pr[2] - ptx::bf16_lo(h1), pr[3] - ptx::bf16_hi(h1));
                *reinterpret_cast<uint2*>(smem + kOffPhi + srow * kPPitch + stok * 2) = make_uint2(h0, h1);
                *reinterpret_cast<uint2*>(smem + kOffPlo + srow * kPPitch + stok * 2) = make_uint2(l0, l1);
                if ((lane & 15) == 0) s_alpha[srow] = alpha;
            }
            consumer_barrier();

            // ---- phase 3: O[:, 64 warp .. 64 warp + 64) = O * alpha + (P_hi + P_lo) V ----
            {
                const int r0 = lane >> 2;
                const float a0 = s_alpha[r0], a1 = s_alpha[r0 + 8];
                if (__any_sync(0xffffffffu, (a0 != 1.f) | (a1 != 1.f))) {
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) { o[nt][0] *= a0; o[nt][1] *= a0; o[nt][2] *= a1; o[nt][3] *= a1; }
                }
                const uint32_t vb = kb + warp * 8192;
                auto load_p = [&](int kk, uint32_t (&ph)[4], uint32_t (&pl)[4]) {
                    const uint32_t poff = ((mi & 1) * 8 + r8) * kPPitch + (kk * 2 + (mi >> 1)) * 16;
                    ptx::ldmatrix_x4(s_phi + poff, ph[0], ph[1], ph[2], ph[3]);
                    ptx::ldmatrix_x4(s_plo + poff, pl[0], pl[1], pl[2], pl[3]);
                };
                auto load_v = [&](int kk, uint32_t (&vf)[4][4]) {
                    const int tok = kk * 16 + (mi & 1) * 8 + r8;
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj)
                        ptx::ldmatrix_x4_trans(vb + tok * 128 + (((2 * jj + (mi >> 1)) ^ r8) << 4), vf[jj][0], vf[jj][1], vf[jj][2], vf[jj][3]);
                };
                auto product = [&](const uint32_t (&pw)[4], const uint32_t (&vf)[4][4]) {
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        ptx::mma_bf16(o[2 * jj], pw, vf[jj][0], vf[jj][1]);
                        ptx::mma_bf16(o[2 * jj + 1], pw, vf[jj][2], vf[jj][3]);
                    }
                };
                // all value fragments of a 16-token step first, then the p_hi products, then the p_lo products: two MMAs on
                // the same accumulator are eight instructions apart
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
                    uint32_t ph[4], pl[4], vf[4][4];
                    load_p(kk, ph, pl);
                    load_v(kk, vf);
                    product(ph, vf);
                    product(pl, vf);
                }
                // The last two steps: both steps' value fragments are fetched first and their p_hi products issued (an MMA is
                // not issued before its operands are there, so after them the tile's last bytes have been read); the stage then
                // goes back to the producer while the p_lo products, half of these steps' MMAs, are still to come.
                {
                    uint32_t ph2[4], pl2[4], ph3[4], pl3[4], vf2[4][4], vf3[4][4];
                    load_p(2, ph2, pl2);
                    load_v(2, vf2);
                    load_p(3, ph3, pl3);
                    load_v(3, vf3);
                    product(ph2, vf2);
                    product(ph3, vf3);
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(s_empty + 8 * st);
                    product(pl2, vf2);
                    product(pl3, vf3);
                }
            }
        }

        // ---- end of span: the row owners publish m and l, every warp scales and writes its 64 columns ----
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) l_run += __shfl_xor_sync(0xffffffffu, l_run, d);
        if ((lane & 15) == 0) { s_m[srow] = m_run; s_l[srow] = l_run; }
        consumer_barrier();
        if (kChecked && (int64_t(sn) + 1) * 16 > p.part_rows) {             // the partial's rows must lie inside the scratch
            if (tid == 0) atomicOr(p.status, kStatusBadIndex);
        } else {
            const int r0 = lane >> 2, c0 = warp * 64 + 2 * (lane & 3);
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int row = r0 + half * 8;
                if (row < n_heads) {
                    const float L = s_l[row];
                    const float inv = (L > 0.f) ? 1.f / L : 0.f;
                    float* dst = p.part_o + (int64_t(sn) * 16 + row) * kDv + c0;
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt)
                        *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[nt][2 * half] * inv, o[nt][2 * half + 1] * inv);
                }
            }
            if (warp == 0 && lane < n_heads) {
                const float M = s_m[lane], L = s_l[lane];
                p.part_lse[int64_t(sn) * 16 + lane] = (M == -INFINITY) ? -INFINITY : (M + log2f(L)) * kLn2;
            }
        }
        consumer_barrier();      // s_m / s_l / the query tile are reused by the next span
    }
    if (!ok && lane == 0) atomicOr(p.status, kStatusNoTile);
}

}  // namespace

cudaError_t launch_attend_mla_tc(const AttnLaunch& a, cudaStream_t s);

cudaError_t launch_attend_mla(const AttnLaunch& a, cudaStream_t s) {
    if (a.n_ctas <= 0 || a.n_spans <= 0) return cudaSuccess;
    // opt-in tcgen05 / TMEM variant (attn_mla_tc.cu): correct, but slower than this kernel for 16-head groups
    static const bool use_tc = std::getenv("IPKV_MLA_TC") != nullptr;
    if (use_tc) return launch_attend_mla_tc(a, s);
    if (a.dim_qk != kDqk || a.dim_v != kDv || a.n_kv_heads != 1) return cudaErrorInvalidValue;
    MlaParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    for (int i = 0; i < kMaxBases; ++i) p.bases[i] = a.bases[i];
    p.segs = a.segs; p.spans = a.spans; p.cta_span_start = a.cta_span_start;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.status = a.status;
    p.Hq = a.n_q_heads;
    p.bt = a.bt;
    p.block_bytes = int64_t(a.bt) * kDqk * 2;
    p.scale_log2 = a.scale * kLog2e;
    p.early = a.early_tiles;
    p.win_tail = a.win_tail;
    for (int i = 0; i < kMaxBases; ++i) p.base_bytes[i] = a.base_bytes[i];
    p.part_rows = a.part_rows;
    const int smem = kSmemTotal + 1024;
    static bool configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(attn_mla_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    return launch_ordered(!a.plain_launch, attn_mla_kernel, a.n_ctas, kThreads, size_t(smem), s, p);
}

}  // namespace ipkvi
