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
// online softmax and fp32 output accumulators in registers.  Nothing synchronises the CTA per tile.  At the
// end of a span the four warps either write a normalised partial (O, natural-log LSE) each, or, in launches
// whose spans are long (the host decides, plan.hpp), join their states through shared memory into one; the
// LSE reduce joins the partials of all spans of a (row, head).
//
// Tiles are handed to the CTAs either in plan order or, by default for launches that are long enough, by the dynamic
// balancing of schedule.cuh (CTAs that finish early take over tiles of the ones that are behind).
//
// The kernel is launched so that it may become resident while the previous kernel of the stream drains (launch.cuh):
// everything up to the first use of the queries, the scheduling words or the partials' scratch runs before the wait
// for that kernel, and when the host knows the K/V bytes to be settled the producer even fills the copy ring first.
//
// HBM traffic per KV token: bytes_per_token, read exactly once.
#include <cuda_bf16.h>

#include "kernels.h"
#include "launch.cuh"
#include "ptx.cuh"
#include "schedule.cuh"

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
    const __nv_bfloat16* append_k;   // fused append: new K / V rows [n_rows][n_kv_heads][D], or null
    const __nv_bfloat16* append_v;
    int32_t* next;       // dynamic schedule: tiles claimed so far of every span [n_spans], of every CTA's chunk [n_ctas], and the
                         // number of CTAs that came to help with every chunk [n_ctas] (all zero at launch); null = static schedule
    const int32_t* cta_tiles;   // tiles in every CTA's chunk
    int32_t* lists;      // per (row, head group): the number of extra partials CTAs filled for it [n_rows * n_gh], then their indices
                         // [n_rows * n_gh][kStealListCap] (all zero at launch); null = no CTA helps another
    int n_spans, n_ctas, n_rows, n_gh;
    int early;          // nonzero: the producer may issue its first copies of ring tiles (2: of window tiles too) before the
                        // previous kernel of the stream has completed
    int Hq, G, n_hg, RG;
    int NW;             // partials per span: 1 = the consumer warps join their states at the end of a span, 4 = each writes its own
    int bt;
    int64_t head_bytes, block_bytes;
    float scale_log2;
    int win_tail;       // valid tokens in the last tile of runs flagged kSegTailParam
    int64_t base_bytes[kMaxBases];   // bounds-checked build: extent behind every base (0: not checked)
    int64_t part_rows;               // bounds-checked build: rows of partial storage
};

template <int D, int STAGES, int ROWS>
struct SmemPlan {
    static constexpr int kPlane = D * 128;               // bytes of a 64-token K (or V) tile
    static constexpr int kStage = 2 * kPlane;
    static constexpr int kStagesBytes = STAGES * kStage;
    static constexpr int kBarOff = kStagesBytes;
    static constexpr int kMetaOff = kBarOff + 2 * STAGES * 8;     // one StageMeta (32 bytes) per stage
    // joining the four consumer warps' states at the end of a partial: a give-up flag, every warp's (max, sum) per
    // query row, and one buffer of output rows (padded: rows 0..3 on distinct banks)
    static constexpr int kFlagOff = kMetaOff + STAGES * 32;
    static constexpr int kMlOff = kFlagOff + 16;
    static constexpr int kRowPitch = D + 8;              // floats
    static constexpr int kObufOff = kMlOff + 2 * kConsumerWarps * 16 * 4;
    static constexpr int kTotal = kObufOff + ROWS * kRowPitch * 4;
};

template <int D, int STAGES, bool DUP>
__global__ void __launch_bounds__(kThreads, 2) attn_gqa_kernel(const GqaParams p) {
    using SP = SmemPlan<D, STAGES, DUP ? 8 : 16>;
    extern __shared__ unsigned char smem_dyn[];
    // align the ring to 1024 bytes so that the 128-byte chunk swizzle maps onto distinct banks
    unsigned char* smem = smem_dyn + ((1024u - (ptx::smem_addr(smem_dyn) & 1023u)) & 1023u);
    const uint32_t s_base = ptx::smem_addr(smem);
    const uint32_t s_full = s_base + SP::kBarOff;
    const uint32_t s_empty = s_full + STAGES * 8;
    volatile StageMeta* s_meta = reinterpret_cast<volatile StageMeta*>(smem + SP::kMetaOff);
    volatile int* s_gave_up = reinterpret_cast<volatile int*>(smem + SP::kFlagOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int span_begin = p.cta_span_start[blockIdx.x], span_end = p.cta_span_start[blockIdx.x + 1];
    const bool dynamic = p.next != nullptr;

    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            ptx::mbar_init(s_full + 8 * s, 1);
            ptx::mbar_init(s_empty + 8 * s, kConsumerWarps);
        }
        *s_gave_up = 0;
        ptx::mbar_fence_init();
    }
    if (p.bt < kTileTokens) {
        // tiles spanning several small blocks may leave rows unwritten at the end of a run: make them finite
        for (int c = tid; c < SP::kStagesBytes / 16; c += kThreads)
            reinterpret_cast<uint4*>(smem)[c] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // Everything above may run while the previous kernel of the stream drains; the queries, the scheduling words and the
    // partials' scratch belong to it until it has completed.
    // With a host that vouches for the K/V bytes (GqaParams::early) the producer does not wait here: it fills the ring
    // first, so the copies' latency overlaps the previous kernel's drain as well, and waits before its first refill
    // (fixed schedule) or before its first claim (balanced schedule: the scheduling words may still be being cleared by
    // that kernel, so the first tiles of every chunk are its owner's without a claim).
    const bool early = p.early != 0;
    if (!(early && warp == kConsumerWarps)) {
        ptx::grid_dependency_wait();
        ptx::grid_launch_dependents();      // only ever after a wait has returned: the next kernel's start then implies the previous one's end
    }

    bool ok = true;
    int it = 0;                      // tiles streamed so far by this CTA: stage = it % STAGES

    if (warp == kConsumerWarps) {
        // ---------------- producer: lane 0 claims tiles and issues copies; the whole warp looks for work to take over ----------------
        {
            const uint64_t pol = ptx::l2_evict_first_policy();     // the KV stream is read once: first out of L2
            // stream tile `tile` of a span into the next stage, to be accumulated into partial `slot`
            int cached_sp = -1;
            Seg seg{};
            const char* seg_base = nullptr;
            const char* chk_lo = nullptr;       // bounds-checked build: the region the current run must lie in
            int64_t chk_n = 0;
            auto CHK = [&](const char* src, uint32_t bytes) { return ptx::checked_src<kChecked>(src, bytes, chk_lo, chk_n, p.status, kStatusBadIndex); };
            bool waited = !early;
            auto issue = [&](int sp, const Span& span, int tile, int slot) -> bool {
                if (!waited && it >= STAGES) { ptx::grid_dependency_wait(); waited = true; }
                if (sp != cached_sp) {                             // first tile of a span: where its run lives
                    seg = p.segs[span.seg];
                    if (seg.base_id & kSegTailParam) seg.n_tokens += p.win_tail - kTileTokens;
                    seg_base = p.bases[seg.base_id & kSegBaseMask] + seg.off + int64_t(span.gh / p.n_hg) * p.head_bytes;
                    chk_lo = p.bases[seg.base_id & kSegBaseMask]; chk_n = p.base_bytes[seg.base_id & kSegBaseMask];
                    cached_sp = sp;
                }
                // a tile of the D-window may have been written by the kernel in front of this one (an append kernel)
                if (!waited && p.early < 2 && (seg.base_id & kSegBaseMask) == kSegBaseWindow) { ptx::grid_dependency_wait(); waited = true; }
                const int st = it % STAGES;
                if (it >= STAGES && !ptx::mbar_wait(s_empty + 8 * st, ((it / STAGES) - 1) & 1)) return false;
                const int64_t t0 = int64_t(tile) * kTileTokens;
                const int64_t left = int64_t(seg.n_tokens) - t0;
                const int g = span.gh / p.n_hg, hg = span.gh - g * p.n_hg;
                s_meta[st].slot = slot;
                s_meta[st].n_valid = left < kTileTokens ? int(left) : kTileTokens;
                s_meta[st].q_row = span.row * p.Hq + g * p.G + hg * 16;
                s_meta[st].n_heads = min(16, p.G - hg * 16);
                int patch_tok = -1;
                if ((seg.base_id & kSegAppended) && tile == (seg.n_tokens - 1) / kTileTokens) {
                    // the run's last token comes with the launch (block_tokens >= 64 here: one block holds the tile)
                    patch_tok = (seg.n_tokens - 1) % kTileTokens;
                    const int64_t blk = t0 / p.bt;
                    const uint64_t g_row = reinterpret_cast<uint64_t>(seg_base + blk * p.block_bytes + (t0 - blk * p.bt + patch_tok) * 128);
                    s_meta[st].kv_row = span.row * (p.Hq / p.G) + g;
                    s_meta[st].g_lo = uint32_t(g_row);
                    s_meta[st].g_hi = uint32_t(g_row >> 32);
                    if (kChecked && chk_n > 0) {           // the new rows' K and V chunks must land inside the window region
                        const char* row_lo = reinterpret_cast<const char*>(g_row);
                        const char* row_hi = row_lo + int64_t(D / 64 - 1) * p.bt * 128 + 128 + int64_t(p.bt) * D * 2;
                        if (row_lo < chk_lo || row_hi > chk_lo + chk_n) { atomicOr(p.status, kStatusBadIndex); patch_tok = -1; }
                    }
                }
                s_meta[st].patch_tok = patch_tok;
                const uint32_t dst = s_base + st * SP::kStage;
                const uint32_t bar = s_full + 8 * st;
                if (p.bt >= kTileTokens) {
                    const int64_t blk = t0 / p.bt;
                    const int r0 = int(t0 - blk * p.bt);
                    const char* src = seg_base + blk * p.block_bytes;
                    ptx::mbar_expect_tx(bar, SP::kStage);
                    if (p.bt == kTileTokens) {
                        ptx::bulk_g2s_hint(dst, CHK(src, SP::kStage), SP::kStage, bar, pol);   // K plane and V plane are adjacent
                    } else {
                        const int64_t kplane = int64_t(p.bt) * D * 2;
#pragma unroll
                        for (int pn = 0; pn < D / 64; ++pn) {
                            const char* s0 = src + int64_t(pn) * p.bt * 128 + int64_t(r0) * 128;
                            ptx::bulk_g2s_hint(dst + pn * 8192, CHK(s0, 8192), 8192, bar, pol);
                            ptx::bulk_g2s_hint(dst + SP::kPlane + pn * 8192, CHK(s0 + kplane, 8192), 8192, bar, pol);
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
                            ptx::bulk_g2s_hint(dst + pn * 8192 + j * sub_bytes, CHK(src + int64_t(pn) * sub_bytes, sub_bytes), sub_bytes, bar, pol);
                            ptx::bulk_g2s_hint(dst + SP::kPlane + pn * 8192 + j * sub_bytes, CHK(src + kplane + int64_t(pn) * sub_bytes, sub_bytes), sub_bytes, bar, pol);
                        }
                    }
                }
                ++it;
                return true;
            };
            SchedParams sched;
            sched.spans = p.spans; sched.cta_span_start = p.cta_span_start; sched.cta_tiles = p.cta_tiles;
            sched.next = p.next; sched.lists = p.lists; sched.part_lse = p.part_lse;
            sched.n_spans = p.n_spans; sched.n_ctas = p.n_ctas; sched.n_rows = p.n_rows; sched.n_gh = p.n_gh;
            sched.lse_per_partial = p.NW * p.RG;
            sched.head_tiles = (early && dynamic) ? STAGES : 0;
            ok = produce_tiles(sched, lane, issue, [&]() { if (!waited) { ptx::grid_dependency_wait(); waited = true; } });
            if (lane == 0) {
                if (!ok) atomicOr(p.status, kStatusNoFreeStage);
                // tell the consumers that nothing follows
                if (ok) {
                    const int st = it % STAGES;
                    if (it >= STAGES && !ptx::mbar_wait(s_empty + 8 * st, ((it / STAGES) - 1) & 1)) { ok = false; atomicOr(p.status, kStatusNoFreeStage); }
                    if (ok) {
                        s_meta[st].slot = kEndSlot;
                        ptx::mbar_expect_tx(s_full + 8 * st, 0);
                        ++it;
                    }
                }
                // do not leave the CTA while copies of ours may still be in flight
                const int first_pending = it > STAGES ? it - STAGES : 0;
                for (int i = first_pending; i < it; ++i)
                    if (!ptx::mbar_wait(s_full + 8 * (i % STAGES), (i / STAGES) & 1)) atomicOr(p.status, kStatusCopyNotLanded);
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
        for (int i = (span_begin * p.NW + warp); i < span_end * p.NW; i += kConsumerWarps) {
            const int64_t prow = int64_t(i) * p.RG;
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

    // A barrier among the four consumer warps (they run privately otherwise).  It is a hardware barrier, which has no
    // limit of its own; what bounds it is the order of events.  The four warps wait for the same tiles.  A warp comes here
    // only after a tile has arrived that the others wait for as well, each with a limit that started no earlier than this
    // warp's: they get the tile too and follow.  A warp that gave up did so before that tile arrived, and said so in shared
    // memory before it left: whoever comes here afterwards sees the flag and leaves as well instead of waiting.
    auto consumer_sync = [&]() -> bool {
        __syncwarp();
        if (*s_gave_up) return false;
        asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
        return true;
    };

    // The partial of the tiles accumulated so far.  Either every warp writes its own (p.NW == 4), or the four warps' private
    // states (each over its 16 tokens of every tile) are joined into one normalised (O, LSE) per query head (Sec. 5.1's
    // identity, in the log2 domain), so that the split reduce reads one partial per span: warp w scales its accumulators by
    // exp2(m_w - M) / L; warp 0 stores its rows into the buffer, warps 1 and 2 add theirs in turn, warp 3 adds its own to
    // the buffer's and writes the result out.
    auto flush = [&]() -> bool {
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        if (!DUP) {
            l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
            l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        }
        if (p.NW != 1) {
            // every warp writes its own normalised partial: nothing is exchanged, the reduce reads four entries per span
            const int64_t prow = (int64_t(cur_slot) * kConsumerWarps + warp) * p.RG;
            if (kChecked && (prow < 0 || prow + p.RG > p.part_rows)) {    // the partial's rows must lie inside the scratch
                if (lane == 0) atomicOr(p.status, kStatusBadIndex);
                return true;
            }
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
            return true;
        }
        const uint32_t s_m = s_base + SP::kMlOff, s_l = s_m + kConsumerWarps * 16 * 4;
        if ((lane & 3) == 0) {
            ptx::sts_f(s_m + (warp * 16 + r0) * 4, m0); ptx::sts_f(s_l + (warp * 16 + r0) * 4, l0);
            if (!DUP) { ptx::sts_f(s_m + (warp * 16 + r0 + 8) * 4, m1); ptx::sts_f(s_l + (warp * 16 + r0 + 8) * 4, l1); }
        }
        if (!consumer_sync()) return false;
        float mw0[kConsumerWarps], lw0[kConsumerWarps], mw1[kConsumerWarps], lw1[kConsumerWarps];
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            mw0[w] = ptx::lds_f(s_m + (w * 16 + r0) * 4); lw0[w] = ptx::lds_f(s_l + (w * 16 + r0) * 4);
            if (!DUP) { mw1[w] = ptx::lds_f(s_m + (w * 16 + r0 + 8) * 4); lw1[w] = ptx::lds_f(s_l + (w * 16 + r0 + 8) * 4); }
        }
        float M0 = -INFINITY, M1 = -INFINITY, L0 = 0.f, L1 = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            M0 = fmaxf(M0, mw0[w]);
            if (!DUP) M1 = fmaxf(M1, mw1[w]);
        }
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
            if (mw0[w] != -INFINITY) L0 += ptx::ex2(mw0[w] - M0) * lw0[w];
            if (!DUP && mw1[w] != -INFINITY) L1 += ptx::ex2(mw1[w] - M1) * lw1[w];
        }
        const float f0 = (m0 != -INFINITY && L0 > 0.f) ? ptx::ex2(m0 - M0) / L0 : 0.f;
        const float f1 = (!DUP && m1 != -INFINITY && L1 > 0.f) ? ptx::ex2(m1 - M1) / L1 : 0.f;
        const uint32_t buf0 = s_base + SP::kObufOff + (r0 * SP::kRowPitch + c0) * 4;
        const uint32_t buf1 = buf0 + 8 * SP::kRowPitch * 4;
        const int64_t prow = int64_t(cur_slot) * p.RG;
        const bool rows_ok = !(kChecked && (prow < 0 || prow + p.RG > p.part_rows));   // the partial's rows must lie inside the scratch
        if (!rows_ok && warp == kConsumerWarps - 1 && lane == 0) atomicOr(p.status, kStatusBadIndex);
        const bool v0 = r0 < n_heads, v1 = !DUP && (r0 + 8 < n_heads);
        // this warp's scaled rows (in place: the accumulators are started afresh after a flush)
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) {
            o[nt][0] = (DUP ? o[nt][0] + o[nt][2] : o[nt][0]) * f0;
            o[nt][1] = (DUP ? o[nt][1] + o[nt][3] : o[nt][1]) * f0;
            if (!DUP) { o[nt][2] *= f1; o[nt][3] *= f1; }
        }
#pragma unroll 1
        for (int turn = 0; turn < kConsumerWarps; ++turn) {
            if (warp == turn) {
                if (turn > 0) {                    // the rows so far: all loads first, then the sums
                    float2 b0[D / 8], b1[D / 8];
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt) {
                        b0[nt] = ptx::lds_f2(buf0 + nt * 32);
                        if (!DUP) b1[nt] = ptx::lds_f2(buf1 + nt * 32);
                    }
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt) {
                        o[nt][0] += b0[nt].x; o[nt][1] += b0[nt].y;
                        if (!DUP) { o[nt][2] += b1[nt].x; o[nt][3] += b1[nt].y; }
                    }
                }
                if (turn + 1 < kConsumerWarps) {
#pragma unroll
                    for (int nt = 0; nt < D / 8; ++nt) {
                        ptx::sts_f2(buf0 + nt * 32, o[nt][0], o[nt][1]);
                        if (!DUP) ptx::sts_f2(buf1 + nt * 32, o[nt][2], o[nt][3]);
                    }
                } else if (rows_ok) {
                    if (v0) {
                        float* dst = p.part_o + (prow + r0) * D + c0;
#pragma unroll
                        for (int nt = 0; nt < D / 8; ++nt) *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[nt][0], o[nt][1]);
                        if ((lane & 3) == 0) p.part_lse[prow + r0] = (M0 == -INFINITY) ? -INFINITY : (M0 + log2f(L0)) * kLn2;
                    }
                    if (v1) {
                        float* dst = p.part_o + (prow + r0 + 8) * D + c0;
#pragma unroll
                        for (int nt = 0; nt < D / 8; ++nt) *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[nt][2], o[nt][3]);
                        if ((lane & 3) == 0) p.part_lse[prow + r0 + 8] = (M1 == -INFINITY) ? -INFINITY : (M1 + log2f(L1)) * kLn2;
                    }
                }
            }
            if (turn + 1 < kConsumerWarps && !consumer_sync()) return false;
        }
        return true;
    };

    // start a partial: query fragments of its head group straight from global memory (a few KB, L2-resident), then an empty
    // state.  The two are separate because the fragments of the partial before are dead once its last scores are taken: at a
    // change of partial the next one's loads are issued before the flush, so that their latency passes under it.
    auto load_queries = [&](int q_row, int nh) {
        const __nv_bfloat16* qrow0 = p.q + (int64_t(q_row) + r0) * D + c0;
        const bool v0 = r0 < nh, v1 = !DUP && (r0 + 8 < nh);
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
    };
    auto empty_state = [&](int nh) {
        n_heads = nh;
#pragma unroll
        for (int nt = 0; nt < D / 8; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
        m0 = m1 = -INFINITY; l0 = l1 = 0.f;
    };
    // The first tiles are almost always those of the CTA's own first span: its query fragments are fetched while the
    // first copies are in flight. (If another partial comes first, this one is written out empty, which is what it is.)
    if (span_begin < span_end) {
        const Span first = p.spans[span_begin];
        const int g = first.gh / p.n_hg, hg = first.gh - g * p.n_hg;
        cur_slot = span_begin;
        load_queries(first.row * p.Hq + g * p.G + hg * 16, min(16, p.G - hg * 16));
        empty_state(min(16, p.G - hg * 16));
    }

    for (;; ++it) {
        const int st = it % STAGES;
        if (!ptx::mbar_wait(s_full + 8 * st, (it / STAGES) & 1)) { ok = false; *s_gave_up = 1; break; }   // after a timeout: give up
        const int slot = s_meta[st].slot;
        if (slot != cur_slot) {
            const int nh_next = s_meta[st].n_heads;
            if (slot != kEndSlot) load_queries(s_meta[st].q_row, nh_next);
            if (cur_slot != kEndSlot && !flush()) { ok = false; break; }
            if (slot == kEndSlot) break;
            cur_slot = slot;
            empty_state(nh_next);
        }
        const int n_valid = s_meta[st].n_valid;
        {
            const int ptok = s_meta[st].patch_tok;
            if (ptok >= 0 && (ptok >> 4) == warp) {
                // fused append: this warp owns the new token's slice of the tile; lanes 0-15 bring its K row, 16-31 its V row
                const int chunk = lane & 15;
                const bool is_v = lane >= 16;
                if (chunk < D / 8) {
                    const __nv_bfloat16* src = (is_v ? p.append_v : p.append_k) + int64_t(s_meta[st].kv_row) * D + chunk * 8;
                    const uint4 val = __ldg(reinterpret_cast<const uint4*>(src));
                    const uint32_t swz = uint32_t((chunk & 7) ^ (ptok & 7)) << 4;
                    const uint32_t s_off = uint32_t(is_v ? SP::kPlane : 0) + (chunk >> 3) * 8192 + ptok * 128 + swz;
                    *reinterpret_cast<uint4*>(smem + st * SP::kStage + s_off) = val;
                    char* g_row = reinterpret_cast<char*>(uint64_t(s_meta[st].g_lo) | (uint64_t(s_meta[st].g_hi) << 32));
                    *reinterpret_cast<uint4*>(g_row + int64_t(chunk >> 3) * p.bt * 128 + swz + (is_v ? int64_t(p.bt) * D * 2 : 0)) = val;
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // before the stage goes back to the copy engine
                __syncwarp();
            }
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
    if (!ok) {
        *s_gave_up = 1;
        if (lane == 0) atomicOr(p.status, kStatusNoTile);
        return;
    }
}

template <int D, int STAGES, bool DUP>
cudaError_t launch_gqa(const AttnLaunch& a, cudaStream_t s) {
    using SP = SmemPlan<D, STAGES, DUP ? 8 : 16>;
    GqaParams p;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    for (int i = 0; i < kMaxBases; ++i) p.bases[i] = a.bases[i];
    p.segs = a.segs; p.spans = a.spans; p.cta_span_start = a.cta_span_start;
    p.part_o = a.part_o; p.part_lse = a.part_lse; p.status = a.status;
    p.append_k = static_cast<const __nv_bfloat16*>(a.append_k); p.append_v = static_cast<const __nv_bfloat16*>(a.append_v);
    p.next = a.steal_next; p.lists = a.steal_lists; p.n_spans = a.n_spans; p.n_ctas = a.n_ctas; p.cta_tiles = a.cta_tiles;
    p.n_rows = a.n_rows; p.n_gh = a.n_gh;
    p.early = a.early_tiles;
    p.win_tail = a.win_tail;
    for (int i = 0; i < kMaxBases; ++i) p.base_bytes[i] = a.base_bytes[i];
    p.part_rows = a.part_rows;
    p.Hq = a.n_q_heads; p.G = a.n_q_heads / a.n_kv_heads;
    p.n_hg = (p.G + 15) / 16;
    p.RG = part_geom(0, a.n_q_heads, a.n_kv_heads).rows_per_group;
    p.NW = a.parts_per_span == 1 ? 1 : kConsumerWarps;
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
    return launch_ordered(!a.plain_launch, attn_gqa_kernel<D, STAGES, DUP>, a.n_ctas, kThreads, size_t(smem), s, p);
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
