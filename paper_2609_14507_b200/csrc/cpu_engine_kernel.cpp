// The tile kernel of the CPU-side in-place attention engine (see cpu_engine.cpp).  This file is compiled once per
// instruction-set level (x86-64-v4 = AVX-512, x86-64-v3 = AVX2 + FMA, baseline), each time with IPKV_CPU_KERNEL set to
// the name of the function it defines; cpu_engine.cpp picks one at run time.  (Function multi-versioning by attribute
// gave 2-3x slower code here than a translation unit compiled for the level.)
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>

#include "cpu_engine.h"

#ifndef IPKV_CPU_KERNEL
#define IPKV_CPU_KERNEL attend_chunk_base
#endif

namespace ipkvi {

namespace {

constexpr int kTile = 16;          // tokens widened and scored at a time
constexpr int kPrefetchTiles = 4;  // how far ahead of the tile in work the K/V rows are requested
constexpr int kMaxDim = kCpuMaxDim;
constexpr int kMaxGroup = kCpuMaxGroup;


// 16 fp32 lanes as one value: GCC lowers it to one AVX-512 register, two AVX2 registers or four SSE registers,
// whichever level this file is being compiled for.
typedef float v16f __attribute__((vector_size(64)));
typedef int32_t v16i __attribute__((vector_size(64)));

__attribute__((always_inline)) inline v16f vload(const float* p) { v16f v; std::memcpy(&v, p, sizeof v); return v; }
__attribute__((always_inline)) inline void vstore(float* p, v16f v) { std::memcpy(p, &v, sizeof v); }
__attribute__((always_inline)) inline v16f vsplat(float x) { return v16f{x, x, x, x, x, x, x, x, x, x, x, x, x, x, x, x}; }
__attribute__((always_inline)) inline float hsum(v16f v) {
    float s = 0.f;
    for (int i = 0; i < 16; ++i) s += v[i];
    return s;
}
typedef float v8f __attribute__((vector_size(32)));
typedef float v4f __attribute__((vector_size(16)));
// The lane sums of four vectors at once: halve each twice, then two rounds of pairwise adds across the four.
__attribute__((always_inline)) inline v4f hsum4(v16f a, v16f b, v16f c, v16f d) {
    auto half8 = [](v16f v) { return __builtin_shufflevector(v, v, 0, 1, 2, 3, 4, 5, 6, 7) + __builtin_shufflevector(v, v, 8, 9, 10, 11, 12, 13, 14, 15); };
    auto half4 = [](v8f v) { return __builtin_shufflevector(v, v, 0, 1, 2, 3) + __builtin_shufflevector(v, v, 4, 5, 6, 7); };
    const v4f x0 = half4(half8(a)), x1 = half4(half8(b)), x2 = half4(half8(c)), x3 = half4(half8(d));
    const v4f y0 = __builtin_shufflevector(x0, x1, 0, 2, 4, 6) + __builtin_shufflevector(x0, x1, 1, 3, 5, 7);   // a01 a23 b01 b23
    const v4f y1 = __builtin_shufflevector(x2, x3, 0, 2, 4, 6) + __builtin_shufflevector(x2, x3, 1, 3, 5, 7);   // c01 c23 d01 d23
    return __builtin_shufflevector(y0, y1, 0, 2, 4, 6) + __builtin_shufflevector(y0, y1, 1, 3, 5, 7);           // a b c d
}
__attribute__((always_inline)) inline float hmax(v16f v) {
    float s = v[0];
    for (int i = 1; i < 16; ++i) s = std::max(s, v[i]);
    return s;
}
// exp(x) for x <= 0 (softmax weights), 16 lanes: 2^(x log2 e) with the integer part moved into the exponent field and a
// degree-5 polynomial for the fraction in [-0.5, 0.5] (relative error about 2e-7); anything below -87 becomes 0.
__attribute__((always_inline)) inline v16f vexp_nonpos(v16f x) {
    const v16f lo = vsplat(-87.f);
    const v16i keep = x > lo;                      // lanes that do not underflow (-inf and NaN-free inputs only)
    x = (x > lo) ? x : lo;
    const v16f t = x * vsplat(1.4426950408889634f);
    const v16f r = t + vsplat(12582912.f);         // 1.5 * 2^23: rounds t to the nearest integer in the low mantissa bits
    const v16f n = r - vsplat(12582912.f);
    const v16f f = t - n;
    v16f p = vsplat(1.3333558146e-3f);
    p = p * f + vsplat(9.6181291076e-3f);
    p = p * f + vsplat(5.5504108664e-2f);
    p = p * f + vsplat(2.4022650696e-1f);
    p = p * f + vsplat(6.9314718056e-1f);
    p = p * f + vsplat(1.f);
    const v16i e = (__builtin_convertvector(n, v16i) + 127) << 23;
    v16f scale;
    std::memcpy(&scale, &e, sizeof scale);
    const v16f y = p * scale;
    return keep ? y : vsplat(0.f);
}

typedef uint16_t v16h __attribute__((vector_size(32)));
// bf16 -> fp32, 16 values at a time (n is a multiple of 16): zero-extend, shift into the high half.
__attribute__((always_inline)) inline void widen(const uint16_t* src, float* dst, int n) {
    for (int i = 0; i < n; i += 16) {
        v16h h;
        std::memcpy(&h, src + i, sizeof h);
        const v16i w = __builtin_convertvector(h, v16i) << 16;
        std::memcpy(dst + i, &w, sizeof w);
    }
}
// The K/V rows are read once, in order, a few KB per tile: the rows two tiles ahead are requested while the current
// tile is being worked on (measured without this: 40 000 cycles per 16-token tile spent waiting for the rows, against
// 6 000 for all the arithmetic).
__attribute__((always_inline)) inline void prefetch_rows(const char* p, int bytes) {
    for (int b = 0; b < bytes; b += 64) __builtin_prefetch(p + b, 0, 0);
}


// One item: tokens [t_begin, t_end) of the concatenated CPU-side runs of a row, for KV head g.
// Per 16-token tile: K and V rows widened to fp32 once; scores as 2 heads x 4 tokens register blocks over the head
// dimension; softmax weights 16 tokens at a time; O += P V as 4 heads x 16 columns register blocks, so that every
// widened K/V value loaded from L1 feeds several multiply-adds.
}  // namespace

void IPKV_CPU_KERNEL(const CpuShape& sh, const float* qf /*[G][dqk], pre-scaled*/, const uint16_t* /*bf16 bits: not used here*/, int G, int g,
                  const CpuRun* runs, int n_runs, int64_t t_begin, int64_t t_end, float* m, float* l, float* o) {
    const int dqk = sh.dim_qk, dv = sh.dim_v;
    const bool alias_v = sh.dim_v_stored == 0;
    const int64_t head_bytes = int64_t(sh.bt) * (dqk + sh.dim_v_stored) * 2;
    const int64_t block_bytes = head_bytes * sh.n_kv_heads;
    alignas(64) float kf[kTile * kMaxDim];
    alignas(64) float vf_store[kTile * kMaxDim];
    alignas(64) float s[kMaxGroup][kTile];
    float alpha[kMaxGroup];
    for (int h = 0; h < G; ++h) { m[h] = -std::numeric_limits<float>::infinity(); l[h] = 0.f; }
    std::fill(o, o + size_t(G) * dv, 0.f);
    const float ninf = -std::numeric_limits<float>::infinity();

    int64_t run_first = 0;                       // token index of the current run's first token
    for (int r = 0; r < n_runs; ++r) {
        const int64_t run_last = run_first + runs[r].n_tokens;
        const int64_t lo = std::max(t_begin, run_first), hi = std::min(t_end, run_last);
        for (int64_t t0 = lo; t0 < hi; t0 += kTile) {
            const int nt = int(std::min<int64_t>(kTile, hi - t0));
            // widen the tile's K rows (and V rows) once; every head of the group reuses them. Rows past the end: zeros.
            for (int j = 0; j < nt; ++j) {
                const int64_t rel = t0 + j - run_first;
                const int64_t blk = rel / sh.bt, off = rel - blk * sh.bt;
                const char* head = runs[r].blocks + blk * block_bytes + int64_t(g) * head_bytes;
                const char* krow = head + off * dqk * 2;
                const char* vrow = head + int64_t(sh.bt) * dqk * 2 + off * dv * 2;
                prefetch_rows(krow + kPrefetchTiles * kTile * dqk * 2, dqk * 2);
                widen(reinterpret_cast<const uint16_t*>(krow), kf + j * dqk, dqk);
                if (!alias_v) {
                    prefetch_rows(vrow + kPrefetchTiles * kTile * dv * 2, dv * 2);
                    widen(reinterpret_cast<const uint16_t*>(vrow), vf_store + j * dv, dv);
                }
            }
            if (nt < kTile) {
                std::fill(kf + nt * dqk, kf + kTile * dqk, 0.f);
                if (!alias_v) std::fill(vf_store + nt * dv, vf_store + kTile * dv, 0.f);
            }
            const float* vf = alias_v ? kf : vf_store;
            const int vpitch = alias_v ? dqk : dv;

            // ---- scores: s[h][j] = q_h . k_j ----
            for (int h = 0; h < G; h += 2) {
                const float* q0 = qf + size_t(h) * dqk;
                const float* q1 = qf + size_t(std::min(h + 1, G - 1)) * dqk;
                for (int j = 0; j < kTile; j += 4) {
                    const float* k0 = kf + (j + 0) * dqk;
                    const float* k1 = kf + (j + 1) * dqk;
                    const float* k2 = kf + (j + 2) * dqk;
                    const float* k3 = kf + (j + 3) * dqk;
                    v16f a00 = vsplat(0.f), a01 = a00, a02 = a00, a03 = a00, a10 = a00, a11 = a00, a12 = a00, a13 = a00;
                    for (int i = 0; i < dqk; i += 16) {
                        const v16f x0 = vload(q0 + i), x1 = vload(q1 + i);
                        const v16f y0 = vload(k0 + i), y1 = vload(k1 + i), y2 = vload(k2 + i), y3 = vload(k3 + i);
                        a00 += x0 * y0; a01 += x0 * y1; a02 += x0 * y2; a03 += x0 * y3;
                        a10 += x1 * y0; a11 += x1 * y1; a12 += x1 * y2; a13 += x1 * y3;
                    }
                    const v4f r0 = hsum4(a00, a01, a02, a03);
                    std::memcpy(&s[h][j], &r0, sizeof r0);
                    if (h + 1 < G) {
                        const v4f r1 = hsum4(a10, a11, a12, a13);
                        std::memcpy(&s[h + 1][j], &r1, sizeof r1);
                    }
                }
            }
            // ---- online softmax, 16 tokens of a head at a time ----
            for (int h = 0; h < G; ++h) {
                v16f sv = vload(s[h]);
                if (nt < kTile)
                    for (int j = nt; j < kTile; ++j) sv[j] = ninf;
                const float mx = hmax(sv);
                const float mn = std::max(m[h], mx);
                alpha[h] = std::exp(m[h] - mn);                   // exp(-inf) = 0 on the first tile
                const v16f pv = vexp_nonpos(sv - vsplat(mn));
                vstore(s[h], pv);
                l[h] = l[h] * alpha[h] + hsum(pv);
                m[h] = mn;
            }
            // ---- O[h] = O[h] * alpha_h + sum_j p[h][j] V[j] ----
            for (int h = 0; h < G; h += 4) {
                const int h1 = std::min(h + 1, G - 1), h2 = std::min(h + 2, G - 1), h3 = std::min(h + 3, G - 1);
                float* o0 = o + size_t(h) * dv; float* o1 = o + size_t(h1) * dv; float* o2 = o + size_t(h2) * dv; float* o3 = o + size_t(h3) * dv;
                for (int c = 0; c < dv; c += 16) {
                    v16f a0 = vload(o0 + c) * vsplat(alpha[h]), a1 = vload(o1 + c) * vsplat(alpha[h1]);
                    v16f a2 = vload(o2 + c) * vsplat(alpha[h2]), a3 = vload(o3 + c) * vsplat(alpha[h3]);
                    for (int j = 0; j < kTile; ++j) {
                        const v16f vv = vload(vf + j * vpitch + c);
                        a0 += vsplat(s[h][j]) * vv; a1 += vsplat(s[h1][j]) * vv; a2 += vsplat(s[h2][j]) * vv; a3 += vsplat(s[h3][j]) * vv;
                    }
                    vstore(o0 + c, a0);
                    if (h + 1 < G) vstore(o1 + c, a1);
                    if (h + 2 < G) vstore(o2 + c, a2);
                    if (h + 3 < G) vstore(o3 + c, a3);
                }
            }
        }
        run_first = run_last;
    }
}

}  // namespace ipkvi
