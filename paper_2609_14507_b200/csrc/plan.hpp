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
constexpr int kCtasPerSm = 2;
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

inline int tiles_per_item(int64_t total_tiles, int64_t max_row_tiles, int heads_per_tile, int kv_splits) {
    if (kv_splits > 0) return int(std::max<int64_t>(1, (max_row_tiles + kv_splits - 1) / kv_splits));
    // Fill the machine in whole waves: the grid is (items x heads_per_tile) CTAs, kCtasPerSm resident per SM.
    const int64_t slots = int64_t(kSmCount) * kCtasPerSm;
    const int64_t work = total_tiles * heads_per_tile;
    const int64_t waves = std::max<int64_t>(1, (work + slots * kTargetTilesPerItem - 1) / (slots * kTargetTilesPerItem));
    const int64_t per = (work + slots * waves - 1) / (slots * waves);
    return int(std::max<int64_t>(1, per));
}

// rows[r] = segments of row r. Produces the device tables' host image.
inline void build_plan(const std::vector<std::vector<PlanSeg>>& rows, int heads_per_tile, int kv_splits, Plan* plan) {
    plan->segs.clear(); plan->items.clear(); plan->row_item_start.clear();
    int64_t total_tiles = 0, max_row_tiles = 0, total_tokens = 0;
    for (const auto& row : rows) {
        int64_t rt = 0;
        for (const auto& s : row) { rt += (s.n_tokens + kTileTokens - 1) / kTileTokens; total_tokens += s.n_tokens; }
        total_tiles += rt;
        max_row_tiles = std::max(max_row_tiles, rt);
    }
    plan->total_tokens = total_tokens;
    const int per = tiles_per_item(total_tiles, max_row_tiles, heads_per_tile, kv_splits);
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
