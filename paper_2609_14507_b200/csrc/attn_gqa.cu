// GPU-side decode attention over the GPU-resident share of each sequence (Sec. 5.1): for every
// (sequence, query head) the partial output and log-sum-exp over the D-window and the loaded part of
// the pinned region.  The paper names no GPU kernel; this one is written for sm_100a.
//
// Grouped-query variant, dim_qk = dim_v = D in {64, 128}.
//
// Persistent split-K: the grid is one CTA per resident slot (148 SMs x 2).  The host planner gives every
// CTA one contiguous, equally long chunk of the launch's (64-token tile x KV head) units; inside a chunk
// a new span starts wherever the (row, KV head, run) changes.  A producer warp streams the K and V tiles
// of the whole chunk (contiguous 32 KB pieces in the TILE block layout) into a ring of shared-memory
// stages with bulk asynchronous copies that complete on mbarriers, without pausing at span boundaries.
// Four consumer warps each own 16 tokens of every tile and run a private flash-decoding stream: query
// fragments in registers (the G query heads that share the KV head are the M rows of the tensor-core MMA,
// so one K/V read serves the whole group), K fragments by ldmatrix, V fragments by ldmatrix.trans, fp32
// online softmax and fp32 output accumulators in registers.  Nothing synchronises the CTA per tile or per
// span: at the end of a span every warp writes its own normalised partial (O, natural-log LSE) and the
// LSE reduce joins the partials of all spans and warps of a (row, head).
//
// Dynamic balancing (default for the handle-based calls).  With equal chunks the CTAs do not finish together:
// some SMs are consistently served less of the memory bandwidth than others (end times spread over +-10 %),
// and a kernel is as slow as its last CTA.  So tiles are not handed out by position but claimed: every span has
// a counter that its owner advances in batches (an eighth of what is left per claim, the next claim issued
// before the current batch is copied), and a CTA whose own chunk is exhausted picks the chunk with the most
// unclaimed tiles per CTA already working on it, claims tiles from the span that chunk's owner would reach
// last, and accumulates them into an extra partial of its own (kStealSlots per CTA, entered in the list of the
// span's (row, head group), where the reduce finds it).  A partial is an exact softmax state over whatever set of tokens went into it, so
// any assignment of tiles to partials gives the same attention; only the fp32 summation order changes.  No CTA
// ever waits for another one.  The static schedule (null counters) visits the same tiles in plan order.
//
// HBM traffic per KV token: bytes_per_token, read exactly once.
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
    const Span* spans;
    const int32_t* cta_span_start;
    float* part_o;
    float* part_lse;
    uint32_t* status;
    int32_t* next;       // dynamic schedule: tiles claimed so far of every span [n_spans], of every CTA's chunk [n_ctas], and the
                         // number of CTAs that came to help with every chunk [n_ctas] (all zero at launch); null = static schedule
    const int32_t* cta_tiles;   // tiles in every CTA's chunk
    int32_t* lists;      // per (row, head group): the number of extra partials CTAs filled for it [n_rows * n_gh], then their indices
                         // [n_rows * n_gh][kStealListCap] (all zero at launch); null = no CTA helps another
    int n_spans, n_ctas, n_rows, n_gh;
    int Hq, G, n_hg, RG;
    int bt;
    int64_t head_bytes, block_bytes;
    float scale_log2;
};

template <int D, int STAGES>
struct SmemPlan {
    static constexpr int kPlane = D * 128;               // bytes of a 64-token K (or V) tile
    static constexpr int kStage = 2 * kPlane;
    static constexpr int kStagesBytes = STAGES * kStage;
    static constexpr int kBarOff = kStagesBytes;
    static constexpr int kMetaOff = kBarOff + 2 * STAGES * 8;     // one StageMeta (16 bytes) per stage
    static constexpr int kTotal = kMetaOff + STAGES * 16;
};

// What the producer tells the consumers about the tile in a stage.
struct StageMeta {
    int32_t slot;        // index of the partial this tile is accumulated into; kEndSlot = no more tiles
    int32_t n_valid;     // live tokens of the tile (64 except at the end of a run)
    int32_t q_row;       // row * Hq + first query head of the tile's head group
    int32_t n_heads;     // query heads in the group (at most 16)
};
constexpr int32_t kEndSlot = -1;
constexpr int kMinSteal = 3;        // a chunk is worth helping while at least this many of its tiles are unclaimed

template <int D, int STAGES, bool DUP>
__global__ void __launch_bounds__(kThreads) attn_gqa_kernel(const GqaParams p) {
    using SP = SmemPlan<D, STAGES>;
    extern __shared__ unsigned char smem_dyn[];
    // align the ring to 1024 bytes so that the 128-byte chunk swizzle maps onto distinct banks
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_full = s_base + SP::kBarOff;
    const uint32_t s_empty = s_full + STAGES * 8;
    volatile StageMeta* s_meta = reinterpret_cast<volatile StageMeta*>(smem + SP::kMetaOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int span_begin = p.cta_span_start[blockIdx.x], span_end = p.cta_span_start[blockIdx.x + 1];
    const bool dynamic = p.next != nullptr;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(s_full + 8 * s, 1);
            ptx::mbar_init(s_empty + 8 * s, kConsumerWarps);
        }
        ptx::mbar_fence_init();
    }
    if (p.bt < kTileTokens) {
        // tiles spanning several small blocks may leave rows unwritten at the end of a run: make them finite
        for (int c = tid; c < SP::kStagesBytes / 16; c += kThreads)
            reinterpret_cast<uint4*>(smem)[c] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    bool ok = true;
    int it = 0;                      // tiles streamed so far by this CTA: stage = it % STAGES

    if (warp == kConsumerWarps) {
        // ---------------- producer: lane 0 claims tiles and issues copies; the whole warp looks for work to take over ----------------
        {
            const uint64_t pol = ptx::l2_evict_first_policy();     // the KV stream is read once: first out of L2
            // stream tile `tile` of a span into the next stage, to be accumulated into partial `slot`
            auto issue = [&](const Span& span, const Seg& seg, const char* seg_base, int tile, int slot) -> bool {
                const int st = it % STAGES;
                if (it >= STAGES && !ptx::mbar_wait(s_empty + 8 * st, ((it / STAGES) - 1) & 1)) return false;
                const int64_t t0 = int64_t(tile) * kTileTokens;
                const int64_t left = int64_t(seg.n_tokens) - t0;
                const int g = span.gh / p.n_hg, hg = span.gh - g * p.n_hg;
                s_meta[st].slot = slot;
                s_meta[st].n_valid = left < kTileTokens ? int(left) : kTileTokens;
                s_meta[st].q_row = span.row * p.Hq + g * p.G + hg * 16;
                s_meta[st].n_heads = min(16, p.G - hg * 16);
                const uint32_t dst = s_base + st * SP::kStage;
                const uint32_t bar = s_full + 8 * st;
                if (p.bt >= kTileTokens) {
                    const int64_t blk = t0 / p.bt;
                    const int r0 = int(t0 - blk * p.bt);
                    const char* src = seg_base + blk * p.block_bytes;
                    ptx::mbar_expect_tx(bar, SP::kStage);
                    if (p.bt == kTileTokens) {
                        ptx::bulk_g2s_hint(dst, src, SP::kStage, bar, pol);   // K plane and V plane are adjacent
                    } else {
                        const int64_t kplane = int64_t(p.bt) * D * 2;
#pragma unroll
                        for (int pn = 0; pn < D / 64; ++pn) {
                            const char* s0 = src + int64_t(pn) * p.bt * 128 + int64_t(r0) * 128;
                            ptx::bulk_g2s_hint(dst + pn * 8192, s0, 8192, bar, pol);
                            ptx::bulk_g2s_hint(dst + SP::kPlane + pn * 8192, s0 + kplane, 8192, bar, pol);
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
                        const char* src = seg_base + (blk0 + j) * p.block_bytes;
#pragma unroll
                        for (int pn = 0; pn < D / 64; ++pn) {
                            ptx::bulk_g2s_hint(dst + pn * 8192 + j * sub_bytes, src + int64_t(pn) * sub_bytes, sub_bytes, bar, pol);
                            ptx::bulk_g2s_hint(dst + SP::kPlane + pn * 8192 + j * sub_bytes, src + kplane + int64_t(pn) * sub_bytes, sub_bytes, bar, pol);
                        }
                    }
                }
                ++it;
                return true;
            };
            // All unclaimed tiles of one span. Tiles are claimed in batches that shrink as the span runs out (an eighth
            // of what is left, 8 at most), so that little is locked in when other CTAs come to help, and the claim of
            // the next batch is under way while the copies of the current one are issued. Returns the number of
            // tiles streamed (-1 after a timeout).
            auto drain = [&](int sp, int chunk, int slot, bool helping) -> int {
                const Span span = p.spans[sp];
                const Seg seg = p.segs[span.seg];
                const char* seg_base = p.bases[seg.base_id] + seg.off + int64_t(span.gh / p.n_hg) * p.head_bytes;
                int n = 0;
                if (!dynamic) {
                    for (int t = 0; t < span.ntiles; ++t, ++n)
                        if (!issue(span, seg, seg_base, span.tile0 + t, slot)) return -1;
                    return n;
                }
                // the owner takes an eighth of what is left per claim, a helper a quarter
                const int shift = helping ? 2 : 3;
                auto batch = [shift](int left) { const int b = left >> shift; return b > 8 ? 8 : (b < 1 ? 1 : b); };
                int b = batch(span.ntiles - *reinterpret_cast<volatile int32_t*>(p.next + sp));
                int t0 = atomicAdd(p.next + sp, b);
                while (t0 < span.ntiles) {
                    const int first = t0, last = min(t0 + b, span.ntiles);
                    const int left = span.ntiles - last;           // as far as this CTA knows
                    b = batch(left);
                    t0 = left > 0 ? atomicAdd(p.next + sp, b) : span.ntiles;
                    atomicAdd(p.next + p.n_spans + chunk, last - first);     // what is left of the chunk, for CTAs looking for work
                    for (int t = first; t < last; ++t, ++n)
                        if (!issue(span, seg, seg_base, span.tile0 + t, slot)) return -1;
                }
                return n;
            };
            // own chunk first: the partial of a span lives at the span's index
            if (lane == 0)
                for (int sp = span_begin; sp < span_end && ok; ++sp) ok = drain(sp, int(blockIdx.x), sp, false) >= 0;
            // then help the CTAs that are behind (some SMs get less of the memory bandwidth than others): pick the chunk with
            // the most unclaimed tiles per CTA already working on it, take tiles from the span its owner will reach last,
            // and accumulate them into one of this CTA's extra partials
            if (dynamic && p.lists) {
                int32_t* claimed = p.next + p.n_spans;
                int32_t* helpers = claimed + p.n_ctas;
                int used = 0;
                for (int attempt = 0; used < kStealSlots && attempt < 3 * kStealSlots; ++attempt) {
                    if (!__shfl_sync(0xffffffffu, int(ok), 0)) break;
                    // the warp scans the chunks, kScan independent pairs of loads per lane and round
                    constexpr int kScan = 10;
                    int best = -1, best_score = 0;
                    for (int base = 0; base < p.n_ctas; base += 32 * kScan) {
                        int left[kScan], hl[kScan];
#pragma unroll
                        for (int k = 0; k < kScan; ++k) {
                            const int c = base + k * 32 + lane;
                            left[k] = c < p.n_ctas ? __ldg(p.cta_tiles + c) - __ldcg(claimed + c) : 0;
                            hl[k] = c < p.n_ctas ? __ldcg(helpers + c) : 0;
                        }
#pragma unroll
                        for (int k = 0; k < kScan; ++k) {
                            const int score = left[k] >= kMinSteal ? (left[k] << 6) / (1 + hl[k]) : 0;
                            if (score > best_score) { best_score = score; best = base + k * 32 + lane; }
                        }
                    }
                    // every lane now holds the best chunk of its share. Helpers that arrive together must not all pick
                    // the same one: take the candidate of a lane chosen by CTA and attempt, among the lanes whose
                    // candidate scores at least three quarters of the best
                    int top = best_score;
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) top = max(top, __shfl_xor_sync(0xffffffffu, top, d));
                    if (top <= 0) break;
                    const unsigned good = __ballot_sync(0xffffffffu, best_score > 0 && best_score >= top - (top >> 2));
                    const int rot = (int(blockIdx.x) * 7 + attempt * 13) & 31;
                    const unsigned turned = (good >> rot) | (rot ? good << (32 - rot) : 0u);
                    const int pick = (__ffs(turned) - 1 + rot) & 31;
                    const int victim = __shfl_sync(0xffffffffu, best, pick);
                    // lane 0: the last span of the victim's chunk that still has unclaimed tiles; one of this CTA's extra
                    // partials is entered in the list of the span's (row, head group) unless that list is full
                    const int mine = int(blockIdx.x) * kStealSlots + used;
                    int sp = -1;
                    if (lane == 0) {
                        atomicAdd(helpers + victim, 1);
                        sp = p.cta_span_start[victim + 1] - 1;
                        const int sp_first = p.cta_span_start[victim];
                        while (sp >= sp_first && __ldcg(p.next + sp) >= p.spans[sp].ntiles) --sp;
                        if (sp < sp_first) sp = -1;
                        if (sp >= 0) {
                            const int rg = p.spans[sp].row * p.n_gh + p.spans[sp].gh;
                            const int k = atomicAdd(p.lists + rg, 1);
                            if (k < kStealListCap) p.lists[p.n_rows * p.n_gh + rg * kStealListCap + k] = mine;
                            else sp = -1;
                        }
                    }
                    sp = __shfl_sync(0xffffffffu, sp, 0);
                    if (sp < 0) continue;
                    // the partial is listed from now on: empty until tiles arrive (the span may run out first)
                    for (int i = lane; i < kConsumerWarps * p.RG; i += 32)
                        p.part_lse[(int64_t(p.n_spans) + mine) * kConsumerWarps * p.RG + i] = -INFINITY;
                    __syncwarp();
                    ++used;
                    int n = 0;
                    if (lane == 0) {
                        n = drain(sp, victim, p.n_spans + mine, true);
                        if (n < 0) ok = false;
                    }
                }
            }
            if (lane == 0) {
                // tell the consumers that nothing follows
                if (ok) {
                    const int st = it % STAGES;
                    if (it >= STAGES && !ptx::mbar_wait(s_empty + 8 * st, ((it / STAGES) - 1) & 1)) ok = false;
                    if (ok) {
                        s_meta[st].slot = kEndSlot;
                        ptx::mbar_expect_tx(s_full + 8 * st, 0);
                        ++it;
                    }
                }
                // do not leave the CTA while copies of ours may still be in flight
                const int first_pending = it > STAGES ? it - STAGES : 0;
                for (int i = first_pending; i < it; ++i)
                    if (!ptx::mbar_wait(s_full + 8 * (i % STAGES), (i / STAGES) & 1)) ok = false;
                if (!ok) atomicOr(p.status, 1u);
            }
        }
        return;
    }

    // ---------------- consumers ----------------
    // The softmax weights are split into a bf16 head and a bf16 remainder (p = p_hi + p_lo, about 16
    // significant bits) before the P.V product, so that the output error stays at fp32-accumulation level.
    //   DUP (at most 8 query heads per KV head): query rows 8..15 duplicate rows 0..7; MMA rows 0..7 carry
    //   p_hi and rows 8..15 carry p_lo, so the remainder costs no extra tensor-core work.
    //   otherwise: two P.V products per tile.
    const int mi = lane >> 3, r8 = lane & 7;
    const int r0 = lane >> 2, c0 = 2 * (lane & 3);
    // per-lane ldmatrix row offsets inside a stage (token index inside the tile is warp*16 + ...)
    const int tokK = warp * 16 + (mi >> 1) * 8 + r8;     // K: matrices 0,1 tokens 0-7; 2,3 tokens 8-15
    const int tokV = warp * 16 + (mi & 1) * 8 + r8;      // V: matrices 0,2 tokens 0-7; 1,3 tokens 8-15
    const int tcol = warp * 16 + c0;                     // token of accumulator element 0 (n-tile 0)

    if (dynamic) {
        // a span of this CTA's chunk may be taken over completely by other CTAs: its partial then stays empty
        for (int sp = span_begin; sp < span_end; ++sp) {
            const int64_t prow = (int64_t(sp) * kConsumerWarps + warp) * p.RG;
            if ((lane & 3) == 0) {
                if (r0 < p.RG) p.part_lse[prow + r0] = -INFINITY;
                if (!DUP && r0 + 8 < p.RG) p.part_lse[prow + r0 + 8] = -INFINITY;
            }
        }
    }

    uint32_t qa[D / 16][4];
    float o[D / 8][4];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    int cur_slot = kEndSlot, n_heads = 0;

    // this warp's normalised partial of the tiles accumulated so far (rows = the group's query heads)
    auto flush = [&]() {
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        if (!DUP) {
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        }
        const int64_t prow = (int64_t(cur_slot) * kConsumerWarps + warp) * p.RG;
        if (r0 < n_heads) {
            const float inv = l0 > 0.f ? 1.f / l0 : 0.f;
            float* dst = p.part_o + (prow + r0) * D + c0;
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) {
                const float x = DUP ? o[nt][0] + o[nt][2] : o[nt][0], y = DUP ? o[nt][1] + o[nt][3] : o[nt][1];
                *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(x * inv, y * inv);
            }
            if ((lane & 3) == 0) p.part_lse[prow + r0] = (m0 == -INFINITY) ? -INFINITY : (m0 + log2f(l0)) * kLn2;
        }
        if (!DUP && r0 + 8 < n_heads) {
            const float inv = l1 > 0.f ? 1.f / l1 : 0.f;
            float* dst = p.part_o + (prow + r0 + 8) * D + c0;
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[nt][2] * inv, o[nt][3] * inv);
            if ((lane & 3) == 0) p.part_lse[prow + r0 + 8] = (m1 == -INFINITY) ? -INFINITY : (m1 + log2f(l1)) * kLn2;
        }
    };

    for (;; ++it) {
        const int st = it % STAGES;
        if (!ptx::mbar_wait(s_full + 8 * st, (it / STAGES) & 1)) { ok = false; break; }   // after a timeout: give up
        const int slot = s_meta[st].slot;
        if (slot != cur_slot) {
            if (cur_slot != kEndSlot) flush();
            if (slot == kEndSlot) break;
            cur_slot = slot;
            n_heads = s_meta[st].n_heads;
            // query fragments straight from global memory (a few KB per span, L2-resident)
            const __nv_bfloat16* qrow0 = p.q + (int64_t(s_meta[st].q_row) + r0) * D + c0;
            const bool v0 = r0 < n_heads, v1 = !DUP && (r0 + 8 < n_heads);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                const uint32_t x0 = v0 ? __ldg(reinterpret_cast<const uint32_t*>(qrow0 + ks * 16)) : 0u;
                const uint32_t x2 = v0 ? __ldg(reinterpret_cast<const uint32_t*>(qrow0 + ks * 16 + 8)) : 0u;
                qa[ks][0] = x0; qa[ks][2] = x2;
                if (DUP) { qa[ks][1] = x0; qa[ks][3] = x2; }
                else {
                    qa[ks][1] = v1 ? __ldg(reinterpret_cast<const uint32_t*>(qrow0 + 8 * D + ks * 16)) : 0u;
                    qa[ks][3] = v1 ? __ldg(reinterpret_cast<const uint32_t*>(qrow0 + 8 * D + ks * 16 + 8)) : 0u;
                }
            }
#pragma unroll
            for (int nt = 0; nt < D / 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
            m0 = m1 = -INFINITY; l0 = l1 = 0.f;
        }
        const int n_valid = s_meta[st].n_valid;
        {
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
    }
    if (!ok && lane == 0) atomicOr(p.status, 1u);
}

template <int D, int STAGES, bool DUP>
cudaError_t launch_gqa(const AttnLaunch& a, cudaStream_t s) {
    using SP = SmemPlan<D, STAGES>;
    GqaParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    for (int i = 0; i < kMaxBases; ++i) p.bases[i] = a.bases[i];
    p.segs = a.segs; p.spans = a.spans; p.cta_span_start = a.cta_span_start;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.status = a.status;
    p.next = a.steal_next; p.lists = a.steal_lists; p.n_spans = a.n_spans; p.n_ctas = a.n_ctas; p.cta_tiles = a.cta_tiles;
    p.n_rows = a.n_rows; p.n_gh = a.n_gh;
    p.Hq = a.n_q_heads; p.G = a.n_q_heads / a.n_kv_heads;
    p.n_hg = (p.G + 15) / 16;
    p.RG = part_geom(0, a.n_q_heads, a.n_kv_heads).rows_per_group;
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
    attn_gqa_kernel<D, STAGES, DUP><<<a.n_ctas, kThreads, smem, s>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attend_gqa(const AttnLaunch& a, cudaStream_t s) {
    if (a.n_ctas <= 0 || a.n_spans <= 0) return cudaSuccess;
    const bool dup = a.n_q_heads / a.n_kv_heads <= 8;
    if (a.dim_qk == 128 && a.dim_v == 128) return dup ? launch_gqa<128, 3, true>(a, s) : launch_gqa<128, 3, false>(a, s);
    if (a.dim_qk == 64 && a.dim_v == 64) return dup ? launch_gqa<64, 4, true>(a, s) : launch_gqa<64, 4, false>(a, s);
    return cudaErrorInvalidValue;
}

}  // namespace ipkvi
