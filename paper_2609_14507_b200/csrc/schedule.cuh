// Tile scheduling shared by the persistent attention kernels: the order in which the producer warp of a CTA streams
// tiles, static (plan order) or dynamically balanced.
//
// Dynamic balancing.  With equal chunks the CTAs of a launch do not finish together: some SMs are consistently served
// less of the memory bandwidth than others (end times spread over +-10 % for the grouped-query kernel), and a kernel is
// as slow as its last CTA.  So tiles are not handed out by position but claimed: every span has a counter that its
// owner advances in batches (an eighth of what is left per claim, the next claim issued before the current batch is
// copied), and a CTA whose own chunk is exhausted picks the chunk with the most unclaimed tiles per CTA already working
// on it, claims tiles from the span that chunk's owner would reach last, and accumulates them into an extra partial
// of its own (kStealSlots per CTA, entered in the list of the span's (row, head group), where the reduce finds it).  A
// partial is an exact softmax state over whatever set of tokens went into it, so any assignment of tiles to partials
// gives the same attention; only the fp32 summation order changes.  No CTA ever waits for another one.
//
// Head tiles.  When the launch may start its copies before the previous kernel of the stream has completed (see
// launch.cuh), the scheduling words cannot be touched yet: that kernel may still be clearing them.  The first
// head_tiles tiles of every chunk then belong to the chunk's owner without a claim, the counter of the chunk's first
// span counts the tiles after them, and a producer streams its head tiles, waits, and claims only afterwards.
#pragma once
#include <cstdint>

#include "kernels.h"

namespace ipkvi {

// What the producer tells the consumers about the tile in a stage.
struct StageMeta {
    int32_t slot;        // index of the partial this tile is accumulated into; kEndSlot = no more tiles
    int32_t n_valid;     // live tokens of the tile (64 except at the end of a run)
    int32_t q_row;       // row * Hq + first query head of the tile's head group
    int32_t n_heads;     // query heads in the group (at most 16)
    int32_t patch_tok;   // fused append: token of this tile whose K/V rows come with the launch, -1 = none
    int32_t kv_row;      // ... their index (row * n_kv_heads + kv head) in the launch's new K/V rows
    uint32_t g_lo, g_hi; // ... and the global address of the token's K row in panel 0 of its block
};
constexpr int32_t kEndSlot = -1;
constexpr int kMinSteal = 3;        // a chunk is worth helping while at least this many of its tiles are unclaimed

struct SchedParams {
    const Span* spans;
    const int32_t* cta_span_start;
    const int32_t* cta_tiles;   // tiles in every CTA's chunk
    int32_t* next;              // dynamic schedule: tiles claimed so far of every span [n_spans], of every CTA's chunk [n_ctas], and
                                // the number of CTAs that came to help with every chunk [n_ctas] (all zero at launch); null = static
    int32_t* lists;             // per (row, head group): the number of extra partials CTAs filled for it [n_rows * n_gh], then their
                                // indices [n_rows * n_gh][kStealListCap] (all zero at launch); null = no CTA helps another
    float* part_lse;
    int n_spans, n_ctas, n_rows, n_gh;
    int lse_per_partial;        // LSE values of one span's partial(s): parts_per_span * rows_per_group
    int head_tiles;             // dynamic schedule: this many tiles at the start of every CTA's chunk (of its first span) are the
                                // owner's without a claim, so that it can stream them before it may touch the scheduling words;
                                // the span's counter then counts the tiles after them.  0 = every tile is claimed
};

// Runs in the producer warp (all 32 lanes).  issue(span_index, span, tile, slot) -> bool streams one tile (called by
// lane 0 only; false after a timed-out wait).  settle() is called by every lane before its first access to the
// scheduling words (it waits for the previous kernel of the stream unless the lane has done so already).  Returns
// false after a timeout.
template <class Issue, class Settle>
__device__ __forceinline__ bool produce_tiles(const SchedParams& p, int lane, Issue&& issue, Settle&& settle) {
    const bool dynamic = p.next != nullptr;
    const int span_begin = p.cta_span_start[blockIdx.x], span_end = p.cta_span_start[blockIdx.x + 1];
    bool ok = true;
    // All unclaimed tiles of one span. Tiles are claimed in batches that shrink as the span runs out (an eighth
    // of what is left, 8 at most), so that little is locked in when other CTAs come to help, and the claim of
    // the next batch is under way while the copies of the current one are issued. Returns the number of
    // tiles streamed (-1 after a timeout).
    auto drain = [&](int sp, int chunk, int slot, bool helping) -> int {
        const Span span = p.spans[sp];
        int n = 0;
        if (!dynamic) {
            for (int t = 0; t < span.ntiles; ++t, ++n)
                if (!issue(sp, span, span.tile0 + t, slot)) return -1;
            return n;
        }
        // the chunk's first tiles are its owner's without a claim (head_tiles): streamed before anything else
        const int head = sp == p.cta_span_start[chunk] ? min(p.head_tiles, span.ntiles) : 0;
        if (head > 0 && !helping) {
            for (int t = 0; t < head; ++t, ++n)
                if (!issue(sp, span, span.tile0 + t, slot)) return -1;
            settle();
            atomicAdd(p.next + p.n_spans + chunk, head);     // they count as claimed for CTAs looking for work
        }
        settle();
        // the owner takes an eighth of what is left per claim, a helper a quarter; the counter counts the tiles after the head
        const int avail = span.ntiles - head;
        const int shift = helping ? 2 : 3;
        auto batch = [shift](int left) { const int b = left >> shift; return b > 8 ? 8 : (b < 1 ? 1 : b); };
        int b = batch(avail - *reinterpret_cast<volatile int32_t*>(p.next + sp));
        int t0 = atomicAdd(p.next + sp, b);
        while (t0 < avail) {
            const int first = t0, last = min(t0 + b, avail);
            const int left = avail - last;                 // as far as this CTA knows
            b = batch(left);
            t0 = left > 0 ? atomicAdd(p.next + sp, b) : avail;
            atomicAdd(p.next + p.n_spans + chunk, last - first);     // what is left of the chunk, for CTAs looking for work
            for (int t = first; t < last; ++t, ++n)
                if (!issue(sp, span, span.tile0 + head + t, slot)) return -1;
        }
        return n;
    };
    // own chunk first: the partial of a span lives at the span's index
    if (lane == 0)
        for (int sp = span_begin; sp < span_end && ok; ++sp) ok = drain(sp, int(blockIdx.x), sp, false) >= 0;
    settle();
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
                while (sp >= sp_first && __ldcg(p.next + sp) >= p.spans[sp].ntiles - (sp == sp_first ? min(p.head_tiles, p.spans[sp].ntiles) : 0)) --sp;
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
            for (int i = lane; i < p.lse_per_partial; i += 32)
                p.part_lse[(int64_t(p.n_spans) + mine) * p.lse_per_partial + i] = -INFINITY;
            __syncwarp();
            ++used;
            int n = 0;
            if (lane == 0) {
                n = drain(sp, victim, p.n_spans + mine, true);
                if (n < 0) ok = false;
            }
        }
    }
    return __shfl_sync(0xffffffffu, int(ok), 0) != 0;
}

}  // namespace ipkvi
