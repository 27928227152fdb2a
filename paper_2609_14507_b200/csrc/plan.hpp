// Split-K planning for the GPU-side attention (host-only): turns the per-row list of block runs into
// the segment / work-item tables the kernels read.  The sequence of one row is cut into items of
// roughly equal numbers of 64-token tiles so that the grid fills the 148 SMs in whole waves; the
// partials of a row's items are joined by the LSE reduce (the same exact merge as Sec. 5.1, n-way).
#pragma once
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <vector>

#include "kernels.h"

namespace ipkvi {

constexpr int kSmCount = 148;
constexpr int kTargetTilesPerItem = 16;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct PlanSeg { int base_id; int64_t off; int64_t n_tokens; };

struct Plan {
    std::vector<Seg> segs;
    std::vector<Item> items;
    std::vector<int32_t> row_item_start;
    int64_t total_tokens = 0;
    size_t table_bytes() const {
        return align_up(segs.size() * sizeof(Seg), 16) + align_up(items.size() * sizeof(Item), 16) +
               align_up(row_item_start.size() * sizeof(int32_t), 16);
    }
    void serialize(char* dst) const {
        size_t o = 0;
        if (!segs.empty()) std::memcpy(dst + o, segs.data(), segs.size() * sizeof(Seg));
        o += align_up(segs.size() * sizeof(Seg), 16);
        if (!items.empty()) std::memcpy(dst + o, items.data(), items.size() * sizeof(Item));
        o += align_up(items.size() * sizeof(Item), 16);
        std::memcpy(dst + o, row_item_start.data(), row_item_start.size() * sizeof(int32_t));
    }
};

// Number of pieces a run of `nt` tiles is cut into when items hold at most `per` tiles, and the largest piece.
inline int64_t pieces_of(int64_t nt, int64_t per) { return (nt + per - 1) / per; }

// Tiles per item. With kv_splits > 0 the longest row is cut into that many pieces. Otherwise the size is
// searched so that the grid (items x heads_per_tile CTAs, ctas_per_sm resident per SM) runs in as few
// equally loaded waves as possible: cost = waves x (largest piece + a fixed per-CTA overhead in tile units).
inline int tiles_per_item(const std::vector<int64_t>& seg_tiles, int64_t max_row_tiles, int heads_per_tile,
                          int kv_splits, int ctas_per_sm) {
    if (kv_splits > 0) return int(std::max<int64_t>(1, (max_row_tiles + kv_splits - 1) / kv_splits));
    const int64_t slots = int64_t(kSmCount) * ctas_per_sm;
    int64_t longest = 1;
    for (int64_t nt : seg_tiles) longest = std::max(longest, nt);
    int best = 1;
    double best_cost = 1e300;
    const int64_t hi = std::min<int64_t>(longest, 4 * kTargetTilesPerItem);
    for (int64_t per = 1; per <= hi; ++per) {
        int64_t items = 0, biggest = 0;
        for (int64_t nt : seg_tiles) {
            const int64_t pc = pieces_of(nt, per);
            items += pc;
            biggest = std::max(biggest, (nt + pc - 1) / pc);
        }
        const int64_t waves = (items * heads_per_tile + slots - 1) / slots;
        const double cost = double(waves) * (double(biggest) + 2.0);     // ~2 tiles of fixed cost per CTA
        if (cost < best_cost - 1e-9 || (cost < best_cost + 1e-9 && per > best)) { best_cost = cost; best = int(per); }
    }
    return best;
}

// rows[r] = segments of row r. Produces the device tables' host image.
inline void build_plan(const std::vector<std::vector<PlanSeg>>& rows, int heads_per_tile, int kv_splits, int ctas_per_sm, Plan* plan) {
    plan->segs.clear(); plan->items.clear(); plan->row_item_start.clear();
    int64_t max_row_tiles = 0, total_tokens = 0;
    std::vector<int64_t> seg_tiles;
    for (const auto& row : rows) {
        int64_t rt = 0;
        for (const auto& s : row) {
            if (s.n_tokens <= 0) continue;
            const int64_t nt = (s.n_tokens + kTileTokens - 1) / kTileTokens;
            seg_tiles.push_back(nt);
            rt += nt;
            total_tokens += s.n_tokens;
        }
        max_row_tiles = std::max(max_row_tiles, rt);
    }
    plan->total_tokens = total_tokens;
    const int per = tiles_per_item(seg_tiles, max_row_tiles, heads_per_tile, kv_splits, ctas_per_sm);
    for (size_t r = 0; r < rows.size(); ++r) {
        plan->row_item_start.push_back(int32_t(plan->items.size()));
        for (const auto& s : rows[r]) {
            if (s.n_tokens <= 0) continue;
            const int32_t seg_id = int32_t(plan->segs.size());
            plan->segs.push_back(Seg{s.off, int32_t(s.n_tokens), s.base_id});
            const int64_t nt = (s.n_tokens + kTileTokens - 1) / kTileTokens;
            // equal-sized pieces, so that no piece is a short straggler
            const int64_t pieces = (nt + per - 1) / per;
            int64_t t0 = 0;
            for (int64_t k = 0; k < pieces; ++k) {
                const int64_t cnt = nt / pieces + (k < nt % pieces ? 1 : 0);
                plan->items.push_back(Item{int32_t(r), seg_id, int32_t(t0), int32_t(cnt)});
                t0 += cnt;
            }
        }
    }
    plan->row_item_start.push_back(int32_t(plan->items.size()));
}

}  // namespace ipkvi
