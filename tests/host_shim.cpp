// Test-only C shim over the product's host-side headers (router.hpp, plan.hpp, layout.cuh) so that
// the routing state machine, the split-K planner and the block-layout arithmetic can be exercised on
// a machine without a GPU.  Compiled by tests/host_shim.py with g++; not part of the library.
#include <cstdint>
#include <cstring>
#include <vector>

#include "../paper_2609_14507_b200/csrc/plan.hpp"
#include "../paper_2609_14507_b200/csrc/ring.hpp"
#include "../paper_2609_14507_b200/csrc/router.hpp"

using namespace ipkvi;

extern "C" {

void* shim_router_new(int64_t block, int64_t window, int64_t num, int64_t den) { return new SeqRouter(block, window, num, den); }
void shim_router_free(void* r) { delete static_cast<SeqRouter*>(r); }
void shim_router_set_share(void* r, int64_t num) { static_cast<SeqRouter*>(r)->set_share(num); }
void shim_router_bulk(void* r, int64_t n, int64_t num0, int64_t den0) {
    Run out[2];
    static_cast<SeqRouter*>(r)->bulk(n, num0, den0, out);
}
void shim_router_flush(void* r) { static_cast<SeqRouter*>(r)->evict(); }
// the library's append: evict a full window first, then stage
void shim_router_append(void* r) {
    SeqRouter* s = static_cast<SeqRouter*>(r);
    if (s->window_full()) s->evict();
    s->stage();
}
int64_t shim_router_len(void* r) { return static_cast<SeqRouter*>(r)->length(); }
void shim_router_counts(void* r, int64_t* c) {
    SeqRouter* s = static_cast<SeqRouter*>(r);
    c[0] = s->tokens_in(REGION_U); c[1] = s->tokens_in(REGION_P); c[2] = s->tokens_in(REGION_W);
    c[3] = s->blocks_used(REGION_U); c[4] = s->blocks_used(REGION_P);
    c[5] = s->evictions(); c[6] = s->evictions_cpu();
}
void shim_router_dump(void* r, int8_t* region, int64_t* blk, int32_t* off) {
    SeqRouter* s = static_cast<SeqRouter*>(r);
    for (int64_t t = 0; t < s->length(); ++t) {
        int32_t g, o;
        int64_t b;
        s->locate(t, &g, &b, &o);
        region[t] = int8_t(g); blk[t] = b; off[t] = o;
    }
}

int64_t shim_min_tiles_to_balance(int64_t n_rows, int n_q_heads) { return min_tiles_per_cta_to_balance(n_rows, n_q_heads); }

// plan: rows given as flat (row_start[n_rows+1], n_tokens[n_segs]); fills the span table and the two index arrays
int shim_plan(int n_rows, const int32_t* row_start, const int64_t* seg_tokens, int n_gh, int kv_splits, int ctas_per_sm,
              int cap_spans, int32_t* span_fields /* [cap][5] */, int32_t* cta_span_start /* [<= 148*ctas_per_sm + 1] */,
              int* n_ctas_out, int32_t* rg_span_start /* [n_rows*n_gh + 1] */, int32_t* seg_tokens_out, int* n_segs_out,
              int32_t* cta_tiles /* [<= 148*ctas_per_sm] */, int64_t* table_bytes_out) {
    std::vector<std::vector<PlanSeg>> rows(n_rows);
    for (int r = 0; r < n_rows; ++r)
        for (int k = row_start[r]; k < row_start[r + 1]; ++k) rows[r].push_back(PlanSeg{0, int64_t(k) * 4096, seg_tokens[k]});
    Plan plan;
    build_plan(rows, n_gh, kv_splits, ctas_per_sm, &plan);
    const int n = int(plan.spans.size());
    if (n > cap_spans) return -n;
    int n_runs = 0;
    for (int r = 0; r < n_rows; ++r) n_runs += row_start[r + 1] - row_start[r];
    if (n > max_spans_bound(n_rows, n_runs, n_gh, kv_splits, ctas_per_sm)) return -1000000;   // the bound must hold
    for (int i = 0; i < n; ++i) {
        const Span& sp = plan.spans[i];
        int32_t* f = span_fields + 5 * i;
        f[0] = sp.row; f[1] = sp.gh; f[2] = sp.seg; f[3] = sp.tile0; f[4] = sp.ntiles;
    }
    *n_ctas_out = plan.n_ctas();
    for (size_t c = 0; c < plan.cta_span_start.size(); ++c) cta_span_start[c] = plan.cta_span_start[c];
    for (size_t c = 0; c < plan.rg_span_start.size(); ++c) rg_span_start[c] = plan.rg_span_start[c];
    for (size_t c = 0; c < plan.cta_tiles.size(); ++c) cta_tiles[c] = plan.cta_tiles[c];
    {   // the serialised image has exactly table_bytes() bytes: write it into a guarded buffer
        const size_t tb = plan.table_bytes();
        std::vector<char> img(tb + 64, char(0x5a));
        plan.serialize(img.data());
        for (size_t i = tb; i < tb + 64; ++i) if (img[i] != char(0x5a)) return -2000000;
        *table_bytes_out = int64_t(tb);
    }
    *n_segs_out = int(plan.segs.size());
    for (size_t k = 0; k < plan.segs.size(); ++k) seg_tokens_out[k] = plan.segs[k].n_tokens;
    return n;
}

// the text the library puts behind IPKV_ETIMEOUT for a device status word
int shim_describe_status(uint32_t status, char* out, int cap) {
    const std::string s = describe_device_status(status);
    if (int(s.size()) + 1 > cap) return -1;
    std::memcpy(out, s.c_str(), s.size() + 1);
    return int(s.size());
}
uint32_t shim_status_bit(int which) { return which == 0 ? kStatusNoFreeStage : which == 1 ? kStatusNoTile : kStatusCopyNotLanded; }

// resident ring: slot of P block j of every sequence, for the newest blocks when `used[s]` P blocks exist.
// out_slots gets, sequence after sequence, the slots of blocks [first_resident, used); returns how many were written.
int64_t shim_ring_slots(int n_seqs, int64_t uniform_tokens, const int64_t* tokens_by_seq, int64_t bt, const int64_t* used,
                        int64_t* out_slots, int64_t cap_out, int64_t* total_out, int64_t* caps_out) {
    RingMap m;
    m.init(n_seqs, uniform_tokens, tokens_by_seq, bt);
    *total_out = m.total();
    int64_t n = 0;
    for (int s = 0; s < n_seqs; ++s) {
        caps_out[s] = m.blocks(s);
        if (m.blocks(s) == 0) continue;
        for (int64_t j = m.first_resident(s, used[s]); j < used[s]; ++j) {
            if (n >= cap_out) return -1;
            out_slots[n++] = m.slot(s, j);
        }
    }
    return n;
}

// Two consecutive decode steps of a batch: window runs of `fill` and `fill + 1` tokens behind a resident run each.
// Partials per span of a launch whose rows hold `tokens[r]` tokens each (one run per row): the rule of plan.hpp applied to
// the plan that is actually built.
int shim_parts_per_span(int kind, int n_rows, const int64_t* tokens, int n_gh, int ctas_per_sm) {
    std::vector<std::vector<PlanSeg>> rows(n_rows);
    for (int r = 0; r < n_rows; ++r) rows[r].push_back(PlanSeg{0, int64_t(r) << 26, tokens[r]});
    Plan plan;
    build_plan(rows, n_gh, 0, ctas_per_sm, &plan);
    int64_t tiles = 0;
    for (const Span& sp : plan.spans) tiles += sp.ntiles;
    return parts_per_span_for(kind, tiles, int64_t(plan.spans.size()), int64_t(plan.n_ctas()));
}

int shim_parts_rule(int kind, int64_t tiles, int64_t spans, int64_t ctas) { return parts_per_span_for(kind, tiles, spans, ctas); }

// Returns the launch parameter win_tail of the first step and, in *same_table, whether the two steps' serialised launch
// tables are byte-identical (they must be, unless a window grows into a new tile, when the plan itself changes).
int shim_window_tail(int n_rows, const int64_t* resident_tokens, const int64_t* window_fill, int n_gh, int ctas_per_sm, int* same_table,
                     int* tail_next_out) {
    std::vector<char> img[2];
    int tails[2] = {0, 0};
    for (int step = 0; step < 2; ++step) {
        std::vector<std::vector<PlanSeg>> rows(n_rows);
        for (int r = 0; r < n_rows; ++r) {
            if (resident_tokens[r] > 0) rows[r].push_back(PlanSeg{0, int64_t(r) << 24, resident_tokens[r]});
            if (window_fill[r] + step > 0) rows[r].push_back(PlanSeg{kSegBaseWindow, int64_t(r) << 16, window_fill[r] + step});
        }
        tails[step] = window_tail(rows);
        Plan plan;
        build_plan(rows, n_gh, 0, ctas_per_sm, &plan);
        img[step].assign(plan.table_bytes(), 0);
        plan.serialize(img[step].data());
        int64_t want = 0;
        for (int r = 0; r < n_rows; ++r) want += resident_tokens[r] + window_fill[r] + step;
        if (plan.total_tokens != want) return -1;                   // the real counts stay the plan's counts
    }
    *same_table = img[0] == img[1] ? 1 : 0;
    *tail_next_out = tails[1];
    return tails[0];
}

int64_t shim_tile_chunk_offset(int32_t bt, int32_t t, int32_t chunk) { return tile_chunk_offset(bt, t, chunk); }
int64_t shim_plain_chunk_offset(int32_t d, int32_t t, int32_t chunk) { return plain_chunk_offset(d, t, chunk); }
int64_t shim_block_bytes(int32_t hkv, int32_t dqk, int32_t dv_stored, int32_t bt) {
    BlockGeom g{hkv, dqk, dv_stored, bt};
    return g.block_bytes();
}

}  // extern "C"
