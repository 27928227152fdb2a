// CPU-side in-place attention over the unpinned compute region (Sec. 6.1): the engine that produces the
// CPU partial (O, LSE) which ipkv_merge joins with the GPU partial.
//
// Follows the paper's CPU kernel in spirit, written for whatever the host has (the tile kernel, cpu_engine_kernel.cpp, is
// compiled for AVX-512, AVX2 + FMA and baseline x86-64; cpu_engine_amx.cpp does the two contractions on the AMX tile unit
// where there is one; the best available is picked at first use, IPKV_CPU_KERNEL=amx|v4|v3|base overrides for tests):
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

#if defined(__x86_64__) && defined(__linux__)
#include <cpuid.h>
#include <sys/syscall.h>
#include <unistd.h>
#endif
#include <cstdlib>

#include "cpu_engine.h"

namespace ipkvi {

// cpu_engine_kernel.cpp, compiled per instruction-set level, and cpu_engine_amx.cpp: one item each; the queries come
// widened and pre-scaled (fp32) and as their bf16 bits
#define IPKV_CHUNK_ARGS const CpuShape&, const float*, const uint16_t*, int, int, const CpuRun*, int, int64_t, int64_t, float*, float*, float*
void attend_chunk_amx(IPKV_CHUNK_ARGS);
void attend_chunk_v4(IPKV_CHUNK_ARGS);
void attend_chunk_v3(IPKV_CHUNK_ARGS);
void attend_chunk_base(IPKV_CHUNK_ARGS);

namespace {

using ChunkFn = void (*)(IPKV_CHUNK_ARGS);

bool cpu_has_avx512() {
#if defined(__x86_64__) && defined(__GNUC__)
    __builtin_cpu_init();
    return __builtin_cpu_supports("avx512f") && __builtin_cpu_supports("avx512bw") && __builtin_cpu_supports("avx512dq") &&
           __builtin_cpu_supports("avx512vl");
#else
    return false;
#endif
}

// AMX: the CPU must have the tile unit with bf16 products, and the kernel must grant this process the tile state.
bool amx_usable() {
#if defined(__x86_64__) && defined(__linux__)
    if (!cpu_has_avx512()) return false;
    unsigned a = 0, b = 0, c = 0, d = 0;
    if (!__get_cpuid_count(7, 0, &a, &b, &c, &d)) return false;
    if (!((d >> 22) & 1u) || !((d >> 24) & 1u)) return false;                 // AMX-BF16, AMX-TILE
    constexpr long kArchReqXcompPerm = 0x1023, kXfeatureXtiledata = 18;
    return syscall(SYS_arch_prctl, kArchReqXcompPerm, kXfeatureXtiledata) == 0;
#else
    return false;
#endif
}

struct Kernels {
    ChunkFn vec;        // the vector kernel for this host: any shape
    ChunkFn amx;        // null where there is no tile unit: at most 16 heads a call, dimensions in multiples of 32
};

Kernels pick_kernels() {
    Kernels k{attend_chunk_base, nullptr};
#if defined(__x86_64__) && defined(__GNUC__)
    __builtin_cpu_init();
    if (cpu_has_avx512()) k.vec = attend_chunk_v4;
    else if (__builtin_cpu_supports("avx2") && __builtin_cpu_supports("fma")) k.vec = attend_chunk_v3;
    if (amx_usable()) k.amx = attend_chunk_amx;
    if (const char* want = std::getenv("IPKV_CPU_KERNEL")) {                  // tests: a lower level than the host's best
        const bool avx512 = cpu_has_avx512(), avx2 = __builtin_cpu_supports("avx2") && __builtin_cpu_supports("fma");
        if (!std::strcmp(want, "v4") && avx512) { k.vec = attend_chunk_v4; k.amx = nullptr; }
        else if (!std::strcmp(want, "v3") && avx2) { k.vec = attend_chunk_v3; k.amx = nullptr; }
        else if (!std::strcmp(want, "base")) { k.vec = attend_chunk_base; k.amx = nullptr; }
    }
#endif
    return k;
}

struct Partial {            // online-softmax state of one (row, KV head, chunk): per head m, l; O is unnormalised
    std::vector<float> m, l, o;
};

}  // namespace

int cpu_attend_batch(const CpuShape& sh, int n_rows, const uint16_t* q, const CpuRun* runs, const int32_t* row_run_start,
                     float* o_out, float* lse_out, int n_threads) {
    const int G = sh.n_q_heads / sh.n_kv_heads;
    if (G > kCpuMaxGroup || sh.dim_qk > kCpuMaxDim || sh.dim_v > kCpuMaxDim || sh.dim_qk % 16 != 0 || sh.dim_v % 16 != 0) return -1;
    static const Kernels kernels = pick_kernels();
    // the tile-unit kernel takes 16 query heads at a time: a wider group is done in slices (its rows are then read once per
    // slice, the later times from cache)
    const bool use_amx = kernels.amx && sh.dim_qk % 32 == 0 && sh.dim_v % 32 == 0;
    const ChunkFn attend = use_amx ? kernels.amx : kernels.vec;
    const int slice = use_amx ? 16 : G;
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
        const size_t q_off = (size_t(it.row) * sh.n_q_heads + size_t(it.g) * G) * sh.dim_qk;
        for (int h0 = 0; h0 < G; h0 += slice)
            attend(sh, qf.data() + q_off + size_t(h0) * sh.dim_qk, q + q_off + size_t(h0) * sh.dim_qk, std::min(slice, G - h0), it.g,
                   runs + row_run_start[it.row], row_run_start[it.row + 1] - row_run_start[it.row], it.t0, it.t1,
                   p.m.data() + h0, p.l.data() + h0, p.o.data() + size_t(h0) * sh.dim_v);
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

const char* cpu_engine_kernel_name(const CpuShape& sh) {
    static const Kernels kernels = pick_kernels();
    if (kernels.amx && sh.dim_qk % 32 == 0 && sh.dim_v % 32 == 0) return "amx";
    return kernels.vec == attend_chunk_v4 ? "v4" : kernels.vec == attend_chunk_v3 ? "v3" : "base";
}

int cpu_engine_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // namespace ipkvi
