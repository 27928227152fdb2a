// CPU-side in-place attention over the unpinned compute region (Sec. 6.1): the engine that produces the
// CPU partial (O, LSE) which ipkv_merge joins with the GPU partial.
//
// Follows the paper's CPU kernel in spirit, written for whatever vector width the host has (the compiler
// clones the hot loop for AVX-512, AVX2 and baseline x86-64 and picks one at load time):
//   * zero-copy: K/V are read where write-time routing put them — PLAIN blocks of region U, per KV head
//     K[bt][dqk] then V[bt][dv], addressed with strides, never gathered into a contiguous copy;
//   * scores are never materialised beyond a 16-token tile; online softmax keeps a running max and sum per
//     query head (fp32); the output accumulators of a head group (G x dv fp32) stay in L1;
//   * all query heads of a group share one read of each K/V row (bf16 widened to fp32 once per tile);
//   * compressed-latent (MLA) variant: one latent row per token is shared by all heads, and the value is the
//     row's first dv columns, so the widened tile is used for both the score and the output phase.
// Work is split over (row, KV head, token chunk) items run by OpenMP threads; the chunk partials of a
// (row, KV head) are joined with the same exact LSE merge.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

#include "cpu_engine.h"

namespace ipkvi {

namespace {

constexpr int kTile = 16;          // tokens widened and scored at a time
constexpr int kMaxDim = 576;
constexpr int kMaxGroup = 128;     // query heads sharing one KV head (MLA: all heads)

#if defined(__x86_64__) && defined(__GNUC__) && !defined(__clang__)
#define IPKV_CLONES __attribute__((target_clones("avx512f", "avx2,fma", "default")))
#else
#define IPKV_CLONES
#endif

inline void widen(const uint16_t* src, float* dst, int n) {
    for (int i = 0; i < n; ++i) {
        const uint32_t w = uint32_t(src[i]) << 16;
        std::memcpy(dst + i, &w, 4);
    }
}

struct Partial {            // online-softmax state of one (row, KV head, chunk): per head m, l; O is unnormalised
    std::vector<float> m, l, o;
};

// One item: tokens [t_begin, t_end) of the concatenated CPU-side runs of a row, for KV head g.
IPKV_CLONES
void attend_chunk(const CpuShape& sh, const float* qf /*[G][dqk], pre-scaled*/, int G, int g,
                  const CpuRun* runs, int n_runs, int64_t t_begin, int64_t t_end, float* m, float* l, float* o) {
    const int dqk = sh.dim_qk, dv = sh.dim_v;
    const bool alias_v = sh.dim_v_stored == 0;
    const int64_t head_bytes = int64_t(sh.bt) * (dqk + sh.dim_v_stored) * 2;
    const int64_t block_bytes = head_bytes * sh.n_kv_heads;
    alignas(64) float kf[kTile * kMaxDim];
    alignas(64) float vf_store[kTile * kMaxDim];
    float s[kMaxGroup][kTile];
    for (int h = 0; h < G; ++h) { m[h] = -std::numeric_limits<float>::infinity(); l[h] = 0.f; }
    std::fill(o, o + size_t(G) * dv, 0.f);

    int64_t run_first = 0;                       // token index of the current run's first token
    for (int r = 0; r < n_runs; ++r) {
        const int64_t run_last = run_first + runs[r].n_tokens;
        const int64_t lo = std::max(t_begin, run_first), hi = std::min(t_end, run_last);
        for (int64_t t0 = lo; t0 < hi; t0 += kTile) {
            const int nt = int(std::min<int64_t>(kTile, hi - t0));
            // widen the tile's K rows (and V rows) once; every head of the group reuses them
            for (int j = 0; j < nt; ++j) {
                const int64_t rel = t0 + j - run_first;
                const int64_t blk = rel / sh.bt, off = rel - blk * sh.bt;
                const char* head = runs[r].blocks + blk * block_bytes + int64_t(g) * head_bytes;
                widen(reinterpret_cast<const uint16_t*>(head + off * dqk * 2), kf + j * dqk, dqk);
                if (!alias_v)
                    widen(reinterpret_cast<const uint16_t*>(head + int64_t(sh.bt) * dqk * 2 + off * dv * 2), vf_store + j * dv, dv);
            }
            const float* vf = alias_v ? kf : vf_store;
            const int vpitch = alias_v ? dqk : dv;
            for (int h = 0; h < G; ++h) {
                const float* qh = qf + size_t(h) * dqk;
                float mx = -std::numeric_limits<float>::infinity();
                for (int j = 0; j < nt; ++j) {
                    const float* kr = kf + j * dqk;
                    float acc = 0.f;
#pragma omp simd reduction(+ : acc)
                    for (int i = 0; i < dqk; ++i) acc += qh[i] * kr[i];
                    s[h][j] = acc;
                    mx = std::max(mx, acc);
                }
                const float mn = std::max(m[h], mx);
                const float alpha = std::exp(m[h] - mn);          // exp(-inf) = 0 on the first tile
                float* oh = o + size_t(h) * dv;
                if (alpha != 1.f) {
#pragma omp simd
                    for (int c = 0; c < dv; ++c) oh[c] *= alpha;
                }
                float lsum = 0.f;
                for (int j = 0; j < nt; ++j) {
                    const float pj = std::exp(s[h][j] - mn);
                    lsum += pj;
                    const float* vr = vf + j * vpitch;
#pragma omp simd
                    for (int c = 0; c < dv; ++c) oh[c] += pj * vr[c];
                }
                l[h] = l[h] * alpha + lsum;
                m[h] = mn;
            }
        }
        run_first = run_last;
    }
}

}  // namespace

int cpu_attend_batch(const CpuShape& sh, int n_rows, const uint16_t* q, const CpuRun* runs, const int32_t* row_run_start,
                     float* o_out, float* lse_out, int n_threads) {
    const int G = sh.n_q_heads / sh.n_kv_heads;
    if (G > kMaxGroup || sh.dim_qk > kMaxDim || sh.dim_v > kMaxDim) return -1;
    struct Item { int row, g; int64_t t0, t1; };
    std::vector<Item> items;
    std::vector<int> first_item(size_t(n_rows) * sh.n_kv_heads + 1, 0);
    const int64_t chunk = 2048;
    for (int r = 0; r < n_rows; ++r) {
        int64_t total = 0;
        for (int k = row_run_start[r]; k < row_run_start[r + 1]; ++k) total += runs[k].n_tokens;
        for (int g = 0; g < sh.n_kv_heads; ++g) {
            first_item[size_t(r) * sh.n_kv_heads + g] = int(items.size());
            for (int64_t t0 = 0; t0 < total; t0 += chunk) items.push_back(Item{r, g, t0, std::min(total, t0 + chunk)});
        }
    }
    first_item.back() = int(items.size());
    std::vector<Partial> parts(items.size());
    // widened, pre-scaled queries: [row][Hq][dqk]
    std::vector<float> qf(size_t(n_rows) * sh.n_q_heads * sh.dim_qk);
    for (size_t i = 0; i < qf.size(); ++i) {
        const uint32_t w = uint32_t(q[i]) << 16;
        float f;
        std::memcpy(&f, &w, 4);
        qf[i] = f * sh.scale;
    }
#ifdef _OPENMP
    const int threads = n_threads > 0 ? n_threads : omp_get_max_threads();
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads)
#else
    (void)n_threads;
#endif
    for (int64_t i = 0; i < int64_t(items.size()); ++i) {
        const Item& it = items[size_t(i)];
        Partial& p = parts[size_t(i)];
        p.m.resize(G); p.l.resize(G); p.o.resize(size_t(G) * sh.dim_v);
        attend_chunk(sh, qf.data() + (size_t(it.row) * sh.n_q_heads + size_t(it.g) * G) * sh.dim_qk, G, it.g,
                     runs + row_run_start[it.row], row_run_start[it.row + 1] - row_run_start[it.row], it.t0, it.t1,
                     p.m.data(), p.l.data(), p.o.data());
    }
    // join the chunk partials of every (row, head): exact LSE merge, natural-log LSE out
    for (int r = 0; r < n_rows; ++r)
        for (int g = 0; g < sh.n_kv_heads; ++g) {
            const int i0 = first_item[size_t(r) * sh.n_kv_heads + g], i1 = first_item[size_t(r) * sh.n_kv_heads + g + 1];
            for (int h = 0; h < G; ++h) {
                const size_t row = size_t(r) * sh.n_q_heads + size_t(g) * G + h;
                float* oo = o_out + row * sh.dim_v;
                float M = -std::numeric_limits<float>::infinity();
                for (int i = i0; i < i1; ++i) M = std::max(M, parts[i].m[h]);
                std::fill(oo, oo + sh.dim_v, 0.f);
                if (M == -std::numeric_limits<float>::infinity()) { lse_out[row] = M; continue; }
                double L = 0.0;
                for (int i = i0; i < i1; ++i) {
                    const float w = std::exp(parts[i].m[h] - M);
                    if (w == 0.f) continue;
                    L += double(parts[i].l[h]) * w;
                    const float* po = parts[i].o.data() + size_t(h) * sh.dim_v;
                    for (int c = 0; c < sh.dim_v; ++c) oo[c] += w * po[c];
                }
                const float inv = float(1.0 / L);
                for (int c = 0; c < sh.dim_v; ++c) oo[c] *= inv;
                lse_out[row] = M + float(std::log(L));
            }
        }
    return 0;
}

int cpu_engine_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // namespace ipkvi
