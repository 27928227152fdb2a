// Split-K planning for the GPU-side attention (host-only): turns the per-row list of block runs into
// the tables the persistent attention kernels read.
//
// Work is counted in units of (64-token tile x head group): a head group is one KV head (x one group of
// up to 16 of its query heads) for GQA, one group of up to 16 heads for MLA.  The units are laid out in
// (row, head group, run, tile) order and cut into one contiguous, equally long chunk per CTA — one CTA
// per resident slot of the 148 SMs, so the whole launch is a single balanced wave and every CTA streams
// its chunk without a pause.  Where a chunk crosses from one (row, head group, run) to the next a new
// span starts; every span produces its own partial (O, LSE) — one per consumer warp for GQA — and the
// partials of a (row, head group) are joined by the LSE reduce (the same exact merge as Sec. 5.1, n-way).
#pragma once
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <string>
#include <vector>

#include "kernels.h"

namespace ipkvi {

constexpr int kSmCount = 148;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// When the grouped-query kernel balances its load while it runs (schedule.cuh).  Balancing makes the attention kernel
// about 2 % faster and the split reduce slower (extra partials to read, one CTA fewer per SM), so it pays only when the
// launch is long against its reduce: measured cross-over at 60-70 tiles per CTA when the reduce fits one wave of CTAs
// (16 rows x 32 heads) and at about 135 when it takes 3.5 (64 rows x 32 heads).
constexpr int kMinTilesPerCtaToBalance = 64;
constexpr int kMinTilesPerCtaPerReduceWave = 28;
inline int64_t min_tiles_per_cta_to_balance(int64_t n_rows, int n_q_heads) {
    const double waves = double(n_rows) * n_q_heads / (kSmCount * 4.0);
    return kMinTilesPerCtaToBalance + (waves > 1.0 ? int64_t(kMinTilesPerCtaPerReduceWave * (waves - 1.0)) : 0);
}

// What the bits of the device status word mean, for error messages (empty for 0).
inline std::string describe_device_status(uint32_t status) {
    std::string where;
    if (status & kStatusNoFreeStage) where += " [a producer got no free stage]";
    if (status & kStatusNoTile) where += " [a consumer got no tile]";
    if (status & kStatusCopyNotLanded) where += " [a copy did not land]";
    if (status & kStatusBadIndex) where += " [checked build: a computed address left its region]";
    if (status & ~(kStatusNoFreeStage | kStatusNoTile | kStatusCopyNotLanded | kStatusBadIndex)) where += " [unknown bits]";
    return where;
}

struct PlanSeg { int base_id; int64_t off; int64_t n_tokens; bool appended = false; bool tail_param = false; };

struct Plan {
    std::vector<Seg> segs;
    std::vector<Span> spans;
    std::vector<int32_t> cta_span_start;   // [n_ctas + 1]
    std::vector<int32_t> rg_span_start;    // [n_rows * n_gh + 1]: spans of every (row, head group), contiguous
    std::vector<int32_t> cta_tiles;        // [n_ctas]: tiles in every CTA's chunk (for the dynamic balancing of the GQA kernel)
    int n_gh = 1;
    int64_t total_tokens = 0;
    int n_ctas() const { return int(cta_span_start.size()) - 1; }
    size_t table_bytes() const {
        return align_up(segs.size() * sizeof(Seg), 16) + align_up(spans.size() * sizeof(Span), 16) +
               align_up(cta_span_start.size() * sizeof(int32_t), 16) + align_up(rg_span_start.size() * sizeof(int32_t), 16) +
               align_up(cta_tiles.size() * sizeof(int32_t), 16);
    }
    void serialize(char* dst) const {
        size_t o = 0;
        if (!segs.empty()) std::memcpy(dst + o, segs.data(), segs.size() * sizeof(Seg));
        o += align_up(segs.size() * sizeof(Seg), 16);
        if (!spans.empty()) std::memcpy(dst + o, spans.data(), spans.size() * sizeof(Span));
        o += align_up(spans.size() * sizeof(Span), 16);
        std::memcpy(dst + o, cta_span_start.data(), cta_span_start.size() * sizeof(int32_t));
        o += align_up(cta_span_start.size() * sizeof(int32_t), 16);
        std::memcpy(dst + o, rg_span_start.data(), rg_span_start.size() * sizeof(int32_t));
        o += align_up(rg_span_start.size() * sizeof(int32_t), 16);
        if (!cta_tiles.empty()) std::memcpy(dst + o, cta_tiles.data(), cta_tiles.size() * sizeof(int32_t));
    }
};

// D-window runs that all end at the same offset inside their last tile are flagged so that their token counts travel
// as one launch parameter (kSegTailParam); returns that offset (1..64), or 0 when the runs disagree or there are none.
// How many partials a span writes.  The grouped-query kernel's four consumer warps run privately; at the end of a span they
// either write a partial each, or join their states first (about a microsecond in which the CTA streams nothing, for a
// reduce that reads a quarter of the entries and ends about two microseconds sooner).  Joining pays when spans are long, or
// when a CTA has few of them and they are not tiny.  Measured per step, joined against not, by mean tiles per span (and
// spans per CTA): 116 (1.9; Mixtral shape, batch 16, 24K tokens) +0.7 %; 91 / 64 / 45 / 24 (1.4; Qwen3 shape, 32K tokens at
// CPU shares 0 / 30 / 50 / 70 %) +1.5 / +1.4 / +0.5 / +0.3 %; 81 / 57 / 40 / 24 / 17 (2.7; ragged batch of 64 at shares 0 / 30 /
// 50 / 70 / 90 %) +1.5 / +1.5 / -0.4 / -0.6 / -2.3 %; 1 (1.0; one sequence of 4K tokens) a kernel of 10.4 instead of 9.0 us.
// The compressed-latent kernel's consumer warps share one state: one partial.
constexpr int64_t kJoinWarpsFromTilesPerSpan = 48;        // long spans: always
constexpr int64_t kJoinWarpsFromTilesPerSpanIfFew = 16;   // shorter ones: if a CTA has at most 1.6 spans on average
inline int parts_per_span_for(int kind, int64_t tiles, int64_t spans, int64_t ctas) {
    if (kind == 1) return 1;
    if (spans <= 0) return 4;
    if (tiles >= kJoinWarpsFromTilesPerSpan * spans) return 1;
    if (tiles >= kJoinWarpsFromTilesPerSpanIfFew * spans && 5 * spans <= 8 * ctas) return 1;
    return 4;
}

inline int window_tail(std::vector<std::vector<PlanSeg>>& rows) {
    int tail = 0;
    for (const auto& row : rows)
        for (const PlanSeg& s : row) {
            if (s.base_id != kSegBaseWindow || s.n_tokens <= 0) continue;
            const int t = int((s.n_tokens - 1) % kTileTokens) + 1;
            if (tail == 0) tail = t;
            else if (tail != t) return 0;
        }
    if (tail == 0) return 0;
    for (auto& row : rows)
        for (PlanSeg& s : row)
            if (s.base_id == kSegBaseWindow && s.n_tokens > 0) s.tail_param = true;
    return tail;
}

// Upper bound on the number of spans build_plan can produce.  Pass 1 emits one piece per (row, head group, run), or,
// with kv_splits, at most kv_splits + 1 pieces of it (a row's runs share the row's kv_splits pieces, each run rounds up
// once); pass 2 then cuts a piece wherever a CTA's chunk ends inside it: one cut per CTA boundary, and there are never
// more CTAs than pieces (kv_splits > 0) or than CTA slots.
inline int64_t max_spans_bound(int n_rows, int n_runs, int n_gh, int kv_splits, int ctas_per_sm) {
    const int64_t slots = int64_t(kSmCount) * ctas_per_sm;
    int64_t pieces = int64_t(n_runs) * n_gh;
    if (kv_splits > 0) pieces *= int64_t(kv_splits) + 1;
    const int64_t cuts = kv_splits > 0 ? std::min(slots, pieces) : slots;
    return pieces + cuts + n_rows;
}

// rows[r] = runs of row r.  n_gh = head groups per row.  kv_splits = 0: one balanced chunk per CTA slot;
// kv_splits > 0: every (row, head group) is cut into about that many spans of equal length, one span per CTA
// while they last (more spans than slots: several spans per CTA, still balanced).
inline void build_plan(const std::vector<std::vector<PlanSeg>>& rows, int n_gh, int kv_splits, int ctas_per_sm, Plan* plan) {
    plan->segs.clear(); plan->spans.clear(); plan->cta_span_start.clear(); plan->rg_span_start.clear(); plan->cta_tiles.clear();
    plan->n_gh = n_gh;
    const int64_t slots = int64_t(kSmCount) * ctas_per_sm;
    // segments, and the tiles of every row
    std::vector<std::vector<int32_t>> row_segs(rows.size());
    int64_t total_tokens = 0, row_tiles_sum = 0, max_row_tiles = 0;
    for (size_t r = 0; r < rows.size(); ++r) {
        int64_t rt = 0;
        for (const auto& s : rows[r]) {
            if (s.n_tokens <= 0) continue;
            row_segs[r].push_back(int32_t(plan->segs.size()));
            const int64_t n_table = s.tail_param ? (s.n_tokens + kTileTokens - 1) / kTileTokens * kTileTokens : s.n_tokens;
            plan->segs.push_back(Seg{s.off, int32_t(n_table), s.base_id | (s.appended ? kSegAppended : 0) | (s.tail_param ? kSegTailParam : 0)});
            rt += (s.n_tokens + kTileTokens - 1) / kTileTokens;
            total_tokens += s.n_tokens;
        }
        row_tiles_sum += rt;
        max_row_tiles = std::max(max_row_tiles, rt);
    }
    plan->total_tokens = total_tokens;
    const int64_t units = row_tiles_sum * n_gh;
    // span length limit: kv_splits cuts rows explicitly; otherwise spans are only cut at CTA chunk boundaries
    const int64_t piece = kv_splits > 0 ? std::max<int64_t>(1, (max_row_tiles + kv_splits - 1) / kv_splits) : INT64_MAX;

    // pass 1: spans in (row, head group, run, tile) order, cut every `piece` tiles (kv_splits) ...
    struct Raw { int32_t row, gh, seg, tile0, ntiles; };
    std::vector<Raw> raw;
    for (size_t r = 0; r < rows.size(); ++r)
        for (int gh = 0; gh < n_gh; ++gh)
            for (int32_t sid : row_segs[r]) {
                const int64_t nt = (int64_t(plan->segs[sid].n_tokens) + kTileTokens - 1) / kTileTokens;
                const int64_t pieces = (piece == INT64_MAX) ? 1 : (nt + piece - 1) / piece;
                int64_t t0 = 0;
                for (int64_t k = 0; k < pieces; ++k) {
                    const int64_t cnt = nt / pieces + (k < nt % pieces ? 1 : 0);
                    raw.push_back(Raw{int32_t(r), gh, sid, int32_t(t0), int32_t(cnt)});
                    t0 += cnt;
                }
            }
    // ... pass 2: assign units to CTAs in equal contiguous chunks, cutting spans at chunk boundaries
    int64_t n_ctas = std::min<int64_t>(slots, kv_splits > 0 ? int64_t(raw.size()) : units);
    if (n_ctas < 1) n_ctas = units > 0 ? 1 : 0;
    plan->cta_span_start.push_back(0);
    int64_t done = 0;            // units assigned so far
    int64_t cta = 0;
    auto chunk_end = [&](int64_t c) { return (units * (c + 1)) / n_ctas; };   // balanced: differs by at most one unit
    for (const Raw& rw : raw) {
        int64_t t0 = rw.tile0, left = rw.ntiles;
        while (left > 0) {
            while (cta < n_ctas - 1 && done >= chunk_end(cta)) { plan->cta_span_start.push_back(int32_t(plan->spans.size())); ++cta; }
            const int64_t room = (cta == n_ctas - 1) ? left : std::min<int64_t>(left, chunk_end(cta) - done);
            plan->spans.push_back(Span{rw.row, rw.gh, rw.seg, int32_t(t0), int32_t(room)});
            t0 += room; left -= room; done += room;
        }
    }
    while (int64_t(plan->cta_span_start.size()) < n_ctas + 1) plan->cta_span_start.push_back(int32_t(plan->spans.size()));
    if (n_ctas == 0) plan->cta_span_start.assign(1, 0);
    plan->cta_tiles.assign(size_t(plan->n_ctas()), 0);
    for (int c = 0; c < plan->n_ctas(); ++c)
        for (int32_t k = plan->cta_span_start[size_t(c)]; k < plan->cta_span_start[size_t(c) + 1]; ++k)
            plan->cta_tiles[size_t(c)] += plan->spans[size_t(k)].ntiles;
    // spans of every (row, head group): contiguous because of the emission order
    plan->rg_span_start.assign(rows.size() * size_t(n_gh) + 1, 0);
    {
        size_t k = 0;
        for (size_t r = 0; r < rows.size(); ++r)
            for (int gh = 0; gh < n_gh; ++gh) {
                plan->rg_span_start[r * n_gh + gh] = int32_t(k);
                while (k < plan->spans.size() && plan->spans[k].row == int32_t(r) && plan->spans[k].gh == gh) ++k;
            }
        plan->rg_span_start[rows.size() * size_t(n_gh)] = int32_t(k);
    }
}

}  // namespace ipkvi
