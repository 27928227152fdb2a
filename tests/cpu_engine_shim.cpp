// Test-only C interface over the product's CPU-side attention engine (csrc/cpu_engine.cpp), so that it can be
// checked against the oracle without a GPU.  Builds PLAIN-layout blocks (per KV head: K rows then V rows) from
// token-major inputs, as the library's prefill routing leaves them in the unpinned region.
#include <chrono>
#include <cstdint>
#include <cstring>
#include <vector>

#include "../paper_2609_14507_b200/csrc/cpu_engine.h"

using namespace ipkvi;

extern "C" {

// k [n][Hkv][dqk], v [n][Hkv][dv] (NULL: the value aliases the first dv columns of K) as bf16 bits; the tokens are cut
// into runs of run_tokens[i] tokens, each run starting on a fresh block. q [Hq][dqk]. One query row.
int shim_cpu_attend(int Hq, int Hkv, int dqk, int dv, int bt, float scale, int64_t n, const uint16_t* k, const uint16_t* v,
                    int n_runs, const int64_t* run_tokens, const uint16_t* q, float* o_out, float* lse_out, int n_threads,
                    int reps, double* best_seconds /* may be NULL */) {
    const int dvs = v ? dv : 0;
    const int64_t head_bytes = int64_t(bt) * (dqk + dvs) * 2, block_bytes = head_bytes * Hkv;
    std::vector<std::vector<char>> bufs;
    bufs.resize(size_t(n_runs));
    std::vector<CpuRun> runs;
    runs.resize(size_t(n_runs));
    int64_t t0 = 0;
    for (int r = 0; r < n_runs; ++r) {
        const int64_t nt = run_tokens[r], nb = (nt + bt - 1) / bt;
        bufs[size_t(r)].assign(size_t(nb * block_bytes), char(0x7f));          // unwritten rows hold NaN patterns
        for (int64_t t = 0; t < nt; ++t) {
            const int64_t blk = t / bt, off = t - blk * bt;
            for (int g = 0; g < Hkv; ++g) {
                char* head = bufs[size_t(r)].data() + blk * block_bytes + g * head_bytes;
                std::memcpy(head + off * dqk * 2, k + ((t0 + t) * Hkv + g) * dqk, size_t(dqk) * 2);
                if (v) std::memcpy(head + int64_t(bt) * dqk * 2 + off * dv * 2, v + ((t0 + t) * Hkv + g) * dv, size_t(dv) * 2);
            }
        }
        runs[size_t(r)] = CpuRun{bufs[size_t(r)].data(), nt};
        t0 += nt;
    }
    if (t0 != n) return -2;
    const int32_t row_run_start[2] = {0, n_runs};
    CpuShape sh{Hq, Hkv, dqk, dv, dvs, bt, scale};
    int rc = 0;
    double best = 1e30;
    for (int i = 0; i < (reps > 0 ? reps : 1) && rc == 0; ++i) {
        const auto t_a = std::chrono::steady_clock::now();
        rc = cpu_attend_batch(sh, 1, q, runs.data(), row_run_start, o_out, lse_out, n_threads);
        const double dt = std::chrono::duration<double>(std::chrono::steady_clock::now() - t_a).count();
        if (dt < best) best = dt;
    }
    if (best_seconds) *best_seconds = best;
    return rc;
}

}  // extern "C"
