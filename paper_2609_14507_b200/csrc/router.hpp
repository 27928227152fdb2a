// Write-time router: the pure-integer state of one (layer, sequence) of the four-region format.
//
// Follows Sec. 4.1 (regions, fixed-size blocks), Sec. 4.2 (prefill routed in one shot; decode tokens
// staged in the D-window and evicted as whole batches that never move again) and Sec. 5.3 (successive
// batches routed so that the running fraction of CPU-placed batches equals the marginal share p).
// Host-only C++; no floating point anywhere, so every index is reproducible bit for bit.
#pragma once
#include <cstdint>
#include <vector>

namespace ipkvi {

enum Region : int32_t { REGION_U = 0, REGION_P = 1, REGION_W = 2 };

// A placed run of consecutive tokens: contiguous blocks of one region, starting on a block boundary.
struct Run {
    int32_t region;
    int64_t first_token;
    int64_t n_tokens;
    int64_t first_block;
};

class SeqRouter {
public:
    SeqRouter() = default;
    SeqRouter(int64_t block, int64_t window, int64_t num, int64_t den) { init(block, window, num, den); }

    void init(int64_t block, int64_t window, int64_t num, int64_t den) {
        block_ = block; window_ = window; num_ = num; den_ = den;
        clear();
    }
    void clear() {
        credit_ = den_ / 2;   // centred start: batch k goes to U iff round-half-up(k*p) steps up
        len_ = 0; win_first_ = 0;
        blocks_used_[0] = blocks_used_[1] = 0;
        tokens_in_[0] = tokens_in_[1] = 0;
        evictions_ = evictions_cpu_ = 0;
        runs_.clear();
    }
    void set_share(int64_t num) { num_ = num; }

    int64_t length() const { return len_; }
    int64_t window_fill() const { return len_ - win_first_; }
    int64_t window_first() const { return win_first_; }
    bool window_full() const { return window_fill() == window_; }
    int64_t blocks_used(int region) const { return blocks_used_[region]; }
    int64_t tokens_in(int region) const { return region == REGION_W ? window_fill() : tokens_in_[region]; }
    int64_t evictions() const { return evictions_; }
    int64_t evictions_cpu() const { return evictions_cpu_; }
    const std::vector<Run>& runs() const { return runs_; }
    int64_t block() const { return block_; }

    // How many tokens of an n-token prefill at share num0/den0 the CPU side takes: whole blocks, floored.
    int64_t prefill_cpu_tokens(int64_t n, int64_t num0, int64_t den0) const {
        const int64_t whole_blocks = n / block_;
        return block_ * ((whole_blocks * num0) / den0);
    }

    // Blocks a run of `count` tokens occupies.
    int64_t blocks_for(int64_t count) const { return (count + block_ - 1) / block_; }

    // Prefill: returns the number of runs written to out[0..1] (U run first if non-empty, then P).
    int bulk(int64_t n, int64_t num0, int64_t den0, Run out[2]) {
        const int64_t cpu = prefill_cpu_tokens(n, num0, den0);
        int k = 0;
        if (cpu > 0) out[k++] = place(REGION_U, 0, cpu);
        if (n - cpu > 0) out[k++] = place(REGION_P, cpu, n - cpu);
        len_ = win_first_ = n;
        return k;
    }

    // Which side the next eviction batch would go to, without changing state.
    int peek_eviction_side() const { return (credit_ + num_ >= den_) ? REGION_U : REGION_P; }

    // Evict the window as one batch. Returns the placed run (n_tokens == 0 if the window was empty).
    Run evict() {
        Run none{REGION_W, win_first_, 0, 0};
        const int64_t fill = window_fill();
        if (fill == 0) return none;
        int side = REGION_P;
        credit_ += num_;
        if (credit_ >= den_) { credit_ -= den_; side = REGION_U; }
        Run r = place(side, win_first_, fill);
        win_first_ = len_;
        evictions_ += 1;
        evictions_cpu_ += (side == REGION_U);
        return r;
    }

    // Stage one new decode token; the caller evicts first when window_full(). Returns its window slot.
    int64_t stage() {
        const int64_t slot = window_fill();
        len_ += 1;
        return slot;
    }

    // Locate a token. Returns false if out of range.
    bool locate(int64_t token, int32_t* region, int64_t* region_block, int32_t* offset) const {
        if (token < 0 || token >= len_) return false;
        if (token >= win_first_) {
            *region = REGION_W; *region_block = 0; *offset = static_cast<int32_t>(token - win_first_);
            return true;
        }
        // runs_ is ordered by first_token and covers [0, win_first_) without gaps
        size_t lo = 0, hi = runs_.size();
        while (hi - lo > 1) {
            const size_t mid = (lo + hi) / 2;
            if (runs_[mid].first_token <= token) lo = mid; else hi = mid;
        }
        const Run& r = runs_[lo];
        const int64_t rel = token - r.first_token;
        *region = r.region;
        *region_block = r.first_block + rel / block_;
        *offset = static_cast<int32_t>(rel % block_);
        return true;
    }

private:
    Run place(int region, int64_t first, int64_t count) {
        Run r{region, first, count, blocks_used_[region]};
        blocks_used_[region] += blocks_for(count);
        tokens_in_[region] += count;
        runs_.push_back(r);
        return r;
    }

    int64_t block_ = 1, window_ = 1, num_ = 0, den_ = 1;
    int64_t credit_ = 0;
    int64_t len_ = 0, win_first_ = 0;
    int64_t blocks_used_[2] = {0, 0};
    int64_t tokens_in_[2] = {0, 0};
    int64_t evictions_ = 0, evictions_cpu_ = 0;
    std::vector<Run> runs_;
};

}  // namespace ipkvi
