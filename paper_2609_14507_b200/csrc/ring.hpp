// How the device ring of resident P blocks of one layer is divided among the sequences (host-only).
//
// The ring is a cache of region P (Sec. 4.1: fixed-size blocks are the unit of placement): sequence s owns
// cap[s] consecutive block slots of every layer's ring, and P block j of that sequence, while it is one of the
// newest cap[s], lives in slot start[s] + j mod cap[s].  With one capacity for all sequences a ragged batch
// would reserve the longest sequence's ring for every sequence; with a capacity per sequence the ring holds
// what the batch needs.
#pragma once
#include <algorithm>
#include <cstdint>
#include <vector>

namespace ipkvi {

struct RingMap {
    std::vector<int64_t> cap;      // [n_seqs] block slots of every sequence
    std::vector<int64_t> start;    // [n_seqs + 1] first slot of every sequence's part; start[n_seqs] = slots per layer

    // tokens_by_seq may be null: every sequence then gets uniform_tokens. Capacities are rounded up to whole blocks.
    void init(int n_seqs, int64_t uniform_tokens, const int64_t* tokens_by_seq, int64_t block_tokens) {
        cap.assign(size_t(n_seqs), 0);
        start.assign(size_t(n_seqs) + 1, 0);
        for (int s = 0; s < n_seqs; ++s) {
            const int64_t t = tokens_by_seq ? tokens_by_seq[s] : uniform_tokens;
            cap[size_t(s)] = t > 0 ? (t + block_tokens - 1) / block_tokens : 0;
            start[size_t(s) + 1] = start[size_t(s)] + cap[size_t(s)];
        }
    }
    int64_t total() const { return start.empty() ? 0 : start.back(); }
    int64_t blocks(int seq) const { return cap[size_t(seq)]; }
    int64_t first_slot(int seq) const { return start[size_t(seq)]; }
    // slot (counted from the layer's first slot) of P block j of `seq`; only meaningful while the block is resident
    int64_t slot(int seq, int64_t j) const { return start[size_t(seq)] + j % cap[size_t(seq)]; }
    // with `used` P blocks in existence, blocks [0, first_resident) are no longer (or never were) in the ring
    int64_t first_resident(int seq, int64_t used) const { return std::max<int64_t>(0, used - cap[size_t(seq)]); }
};

}  // namespace ipkvi
