// The CPU-side engine's tile kernel for hosts with AMX (Sapphire Rapids and later): the same item as
// cpu_engine_kernel.cpp computes — tokens [t_begin, t_end) of a row's CPU-side runs for one KV head, all query heads of
// the group — with the two contractions on the tile matrix unit and everything else in AVX-512.
//
// Per step of 32 tokens:
//   scores   S[token][head] = K[token][:] . Q[head][:]    A = K rows, 16 tokens x 32 bf16 columns, loaded with the row
//            pitch straight from the PLAIN block where write-time routing put them (Sec. 6.1: in place, no gather);
//            B = the query tile in pair-interleaved form, prepared once per item; fp32 accumulation in a tile.
//   softmax  16 query heads side by side in the lanes of a vector: running maximum, sum and the weights of a token row
//            need no horizontal operation at all.
//   output   O[head][:] += P[head][token] V[token][:]     A = the weights, transposed to head-major and split into a bf16
//            head and a bf16 remainder (about 16 significant bits, as in the GPU kernels); B = the V rows of a token pair
//            interleaved column by column (one two-source permute per 32 columns); accumulators [16 heads][dv] fp32 in L1,
//            four column blocks of them in tiles at a time.
// The arithmetic is a few dozen cycles per token and KV head, so the kernel runs at the rate the rows arrive from memory:
// they are requested two steps ahead, across block boundaries.
//
// Compiled with -march=x86-64-v4 -mamx-tile -mamx-bf16; cpu_engine.cpp uses it only where the CPU has AMX and the kernel
// grants the tile state (arch_prctl), for head dimensions that are multiples of 32; at most 16 query heads a call (a wider
// group is done in slices).
#include <immintrin.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <limits>

#include "cpu_engine.h"

namespace ipkvi {

namespace {

constexpr int kStep = 32;                // tokens per step: the K dimension of one output-tile product
constexpr int kHeads = 16;               // rows of the weight tile; groups with fewer heads leave rows empty
constexpr int kMaxDim = kCpuMaxDim;

struct alignas(64) TileConfig {
    uint8_t palette, start_row;
    uint8_t reserved[14];
    uint16_t colsb[16];
    uint8_t rows[16];
};

// exp(x) for x <= 0, 16 lanes (the polynomial of cpu_engine_kernel.cpp): anything below -87 becomes 0.
inline __m512 exp_nonpos(__m512 x) {
    const __m512 lo = _mm512_set1_ps(-87.f);
    const __mmask16 keep = _mm512_cmp_ps_mask(x, lo, _CMP_GT_OQ);
    x = _mm512_max_ps(x, lo);
    const __m512 t = _mm512_mul_ps(x, _mm512_set1_ps(1.4426950408889634f));
    const __m512 n = _mm512_roundscale_ps(t, _MM_FROUND_TO_NEAREST_INT | _MM_FROUND_NO_EXC);
    const __m512 f = _mm512_sub_ps(t, n);
    __m512 p = _mm512_set1_ps(1.3333558146e-3f);
    p = _mm512_fmadd_ps(p, f, _mm512_set1_ps(9.6181291076e-3f));
    p = _mm512_fmadd_ps(p, f, _mm512_set1_ps(5.5504108664e-2f));
    p = _mm512_fmadd_ps(p, f, _mm512_set1_ps(2.4022650696e-1f));
    p = _mm512_fmadd_ps(p, f, _mm512_set1_ps(6.9314718056e-1f));
    p = _mm512_fmadd_ps(p, f, _mm512_set1_ps(1.f));
    const __m512i e = _mm512_slli_epi32(_mm512_add_epi32(_mm512_cvtps_epi32(n), _mm512_set1_epi32(127)), 23);
    return _mm512_maskz_mul_ps(keep, p, _mm512_castsi512_ps(e));
}

// rows[i][j] -> rows[j][i] for a 16 x 16 block of fp32
inline void transpose16(__m512 (&r)[16]) {
    __m512 t[16];
    for (int i = 0; i < 8; ++i) {
        t[2 * i] = _mm512_unpacklo_ps(r[2 * i], r[2 * i + 1]);
        t[2 * i + 1] = _mm512_unpackhi_ps(r[2 * i], r[2 * i + 1]);
    }
    for (int i = 0; i < 4; ++i) {
        r[4 * i + 0] = _mm512_castpd_ps(_mm512_unpacklo_pd(_mm512_castps_pd(t[4 * i]), _mm512_castps_pd(t[4 * i + 2])));
        r[4 * i + 1] = _mm512_castpd_ps(_mm512_unpackhi_pd(_mm512_castps_pd(t[4 * i]), _mm512_castps_pd(t[4 * i + 2])));
        r[4 * i + 2] = _mm512_castpd_ps(_mm512_unpacklo_pd(_mm512_castps_pd(t[4 * i + 1]), _mm512_castps_pd(t[4 * i + 3])));
        r[4 * i + 3] = _mm512_castpd_ps(_mm512_unpackhi_pd(_mm512_castps_pd(t[4 * i + 1]), _mm512_castps_pd(t[4 * i + 3])));
    }
    for (int i = 0; i < 2; ++i)
        for (int j = 0; j < 4; ++j) {
            t[8 * i + j] = _mm512_shuffle_f32x4(r[8 * i + j], r[8 * i + j + 4], 0x88);
            t[8 * i + j + 4] = _mm512_shuffle_f32x4(r[8 * i + j], r[8 * i + j + 4], 0xdd);
        }
    for (int j = 0; j < 8; ++j) {
        r[j] = _mm512_shuffle_f32x4(t[j], t[j + 8], 0x88);
        r[j + 8] = _mm512_shuffle_f32x4(t[j], t[j + 8], 0xdd);
    }
}

// fp32 (finite, any sign) -> bf16 bits in the low half of every lane, round to nearest even
inline __m512i to_bf16_bits(__m512 x) {
    const __m512i u = _mm512_castps_si512(x);
    const __m512i odd = _mm512_and_si512(_mm512_srli_epi32(u, 16), _mm512_set1_epi32(1));
    return _mm512_srli_epi32(_mm512_add_epi32(u, _mm512_add_epi32(odd, _mm512_set1_epi32(0x7fff))), 16);
}

}  // namespace

void attend_chunk_amx(const CpuShape& sh, const float* /*qf*/, const uint16_t* qh /*[G][dqk] bf16, not scaled*/, int G, int g,
                      const CpuRun* runs, int n_runs, int64_t t_begin, int64_t t_end, float* m, float* l, float* o) {
    const int dqk = sh.dim_qk, dv = sh.dim_v;
    const bool alias_v = sh.dim_v_stored == 0;
    const int64_t head_bytes = int64_t(sh.bt) * (dqk + sh.dim_v_stored) * 2;
    const int64_t block_bytes = head_bytes * sh.n_kv_heads;
    const int kpitch = dqk * 2, vpitch = alias_v ? dqk * 2 : dv * 2;
    const int n_kc = dqk / 32, n_cb = dv / 16;

    TileConfig cfg;
    std::memset(&cfg, 0, sizeof cfg);
    cfg.palette = 1;
    for (int i = 0; i < 8; ++i) { cfg.colsb[i] = 64; cfg.rows[i] = 16; }
    _tile_loadconfig(&cfg);

    // the query tile, pair-interleaved: qv[kc][r][h] = (q[h][32 kc + 2 r], q[h][32 kc + 2 r + 1]); heads past G are zero
    alignas(64) uint16_t qv[(kMaxDim / 32) * 16 * 32];
    std::memset(qv, 0, size_t(n_kc) * 16 * 32 * 2);
    for (int h = 0; h < G; ++h)
        for (int c = 0; c < dqk; ++c) qv[((c >> 5) * 16 + ((c & 31) >> 1)) * 32 + h * 2 + (c & 1)] = qh[size_t(h) * dqk + c];

    alignas(64) float sbuf[kStep][kHeads];                   // raw scores of a step, token-major
    alignas(64) uint16_t p_hi[kHeads][kStep], p_lo[kHeads][kStep];
    alignas(64) uint16_t kstage[kStep * kMaxDim];            // a step's K rows when they are not 32 contiguous rows of a block
    alignas(64) uint16_t vn[(kMaxDim / 16) * 16 * 32];       // a step's V rows, pair-interleaved: vn[cb][r] = 16 columns x 2 tokens
    alignas(64) float obuf[kHeads * kMaxDim];
    std::memset(obuf, 0, size_t(kHeads) * dv * 4);
    std::memset(kstage, 0, sizeof kstage);
    const __m512 scale = _mm512_set1_ps(sh.scale);
    const __m512 ninf = _mm512_set1_ps(-std::numeric_limits<float>::infinity());
    __m512 m_run = ninf, l_run = _mm512_setzero_ps();
    // pair interleave of two rows of 32 bf16: (a0, b0, a1, b1, ...) for the low and the high 16 columns
    alignas(64) uint16_t idx_lo[32], idx_hi[32];
    for (int i = 0; i < 16; ++i) {
        idx_lo[2 * i] = uint16_t(i); idx_lo[2 * i + 1] = uint16_t(32 + i);
        idx_hi[2 * i] = uint16_t(16 + i); idx_hi[2 * i + 1] = uint16_t(48 + i);
    }
    const __m512i perm_lo = _mm512_load_si512(idx_lo), perm_hi = _mm512_load_si512(idx_hi);

    int64_t run_first = 0;
    for (int r = 0; r < n_runs; ++r) {
        const int64_t run_last = run_first + runs[r].n_tokens;
        const int64_t lo = std::max(t_begin, run_first), hi = std::min(t_end, run_last);
        // where the K and V rows of `count` consecutive tokens of this run are (one division, then steps)
        auto rows_of = [&](int64_t rel, int count, const char** kr, const char** vr) {
            const int64_t blk = rel / sh.bt;
            int64_t off = rel - blk * sh.bt;
            const char* head = runs[r].blocks + blk * block_bytes + int64_t(g) * head_bytes;
            for (int j = 0; j < count; ++j) {
                kr[j] = head + off * kpitch;
                vr[j] = alias_v ? kr[j] : head + int64_t(sh.bt) * kpitch + off * vpitch;
                if (++off == sh.bt) { off = 0; head += block_bytes; }
            }
        };
        for (int64_t t0 = lo; t0 < hi; t0 += kStep) {
            const int nt = int(std::min<int64_t>(kStep, hi - t0));
            const int64_t rel0 = t0 - run_first;
            const char* krow[kStep];
            const char* vrow[kStep];
            // The rows two steps ahead, wherever their block is.  They are requested a few lines at a time between the phases
            // below: a core has a dozen line-fill buffers, and hundreds of requests issued in one go would wait for them
            // while nothing else runs.
            const char* pf_k[kStep];
            const char* pf_v[kStep];
            int pf_rows = 0, pf_row = 0, pf_byte = 0;
            {
                const int64_t rel = rel0 + 2 * kStep;
                pf_rows = int(std::max<int64_t>(0, std::min<int64_t>(kStep, runs[r].n_tokens - rel)));
                if (pf_rows > 0) rows_of(rel, pf_rows, pf_k, pf_v);
            }
            const int pf_row_bytes = kpitch + (alias_v ? 0 : vpitch);
            const int pf_slots = n_kc + kStep / 2 + (n_cb + 3) / 4;
            const int pf_lines = (pf_rows * pf_row_bytes / 64 + pf_slots - 1) / pf_slots;
            auto prefetch_some = [&]() {
                for (int i = 0; i < pf_lines && pf_row < pf_rows; ++i) {
                    const char* p = pf_byte < kpitch ? pf_k[pf_row] + pf_byte : pf_v[pf_row] + (pf_byte - kpitch);
                    _mm_prefetch(p, _MM_HINT_T0);
                    pf_byte += 64;
                    if (pf_byte >= pf_row_bytes) { pf_byte = 0; ++pf_row; }
                }
            };
            rows_of(rel0, nt, krow, vrow);
            const bool contiguous = nt == kStep && krow[kStep - 1] == krow[0] + int64_t(kStep - 1) * kpitch;
            const char* kbase;
            if (contiguous) {
                kbase = krow[0];
            } else {
                for (int j = 0; j < kStep; ++j) {
                    if (j < nt) std::memcpy(kstage + size_t(j) * dqk, krow[j], size_t(kpitch));
                    else std::memset(kstage + size_t(j) * dqk, 0, size_t(kpitch));
                }
                kbase = reinterpret_cast<const char*>(kstage);
            }
            // ---- scores ----
            _tile_zero(0);
            _tile_zero(1);
            for (int kc = 0; kc < n_kc; ++kc) {
                _tile_loadd(7, qv + size_t(kc) * 16 * 32, 64);
                _tile_loadd(6, kbase + kc * 64, kpitch);
                _tile_dpbf16ps(0, 6, 7);
                _tile_loadd(5, kbase + 16 * kpitch + kc * 64, kpitch);
                _tile_dpbf16ps(1, 5, 7);
                prefetch_some();
            }
            _tile_stored(0, sbuf[0], 64);
            _tile_stored(1, sbuf[16], 64);
            // ---- online softmax: lanes are query heads ----
            __m512 sv[kStep];
            __m512 mx = ninf;
            for (int j = 0; j < kStep; ++j) {
                sv[j] = j < nt ? _mm512_mul_ps(_mm512_load_ps(sbuf[j]), scale) : ninf;
                mx = _mm512_max_ps(mx, sv[j]);
            }
            const __m512 mn = _mm512_max_ps(m_run, mx);
            const __m512 alpha = exp_nonpos(_mm512_sub_ps(m_run, mn));     // exp(-inf) = 0 on the first step
            __m512 lsum = _mm512_setzero_ps();
            for (int j = 0; j < kStep; ++j) {
                sv[j] = exp_nonpos(_mm512_sub_ps(sv[j], mn));
                lsum = _mm512_add_ps(lsum, sv[j]);
            }
            l_run = _mm512_fmadd_ps(l_run, alpha, lsum);
            m_run = mn;
            // weights to head-major bf16 head and remainder
            for (int half = 0; half < 2; ++half) {
                __m512 blk[16];
                for (int j = 0; j < 16; ++j) blk[j] = sv[half * 16 + j];
                transpose16(blk);                                            // blk[h] = 16 tokens of head h
                for (int h = 0; h < kHeads; ++h) {
                    const __m512i hb = to_bf16_bits(blk[h]);
                    const __m512 hf = _mm512_castsi512_ps(_mm512_slli_epi32(hb, 16));
                    const __m512i lb = to_bf16_bits(_mm512_sub_ps(blk[h], hf));
                    _mm256_store_si256(reinterpret_cast<__m256i*>(&p_hi[h][half * 16]), _mm512_cvtepi32_epi16(hb));
                    _mm256_store_si256(reinterpret_cast<__m256i*>(&p_lo[h][half * 16]), _mm512_cvtepi32_epi16(lb));
                }
            }
            // ---- V rows of every token pair, interleaved column by column ----
            for (int pr = 0; pr < kStep / 2; ++pr) {
                const int j0 = 2 * pr, j1 = 2 * pr + 1;
                const char* v0 = j0 < nt ? vrow[j0] : nullptr;
                const char* v1 = j1 < nt ? vrow[j1] : nullptr;
                prefetch_some();
                for (int c = 0; c < dv; c += 32) {
                    const __m512i a = v0 ? _mm512_loadu_si512(v0 + c * 2) : _mm512_setzero_si512();
                    const __m512i b = v1 ? _mm512_loadu_si512(v1 + c * 2) : _mm512_setzero_si512();
                    _mm512_store_si512(vn + (size_t(c / 16) * 16 + pr) * 32, _mm512_permutex2var_epi16(a, perm_lo, b));
                    _mm512_store_si512(vn + (size_t(c / 16 + 1) * 16 + pr) * 32, _mm512_permutex2var_epi16(a, perm_hi, b));
                }
            }
            // ---- O = O * alpha + P V ----
            if (_mm512_cmp_ps_mask(alpha, _mm512_set1_ps(1.f), _CMP_NEQ_UQ)) {
                alignas(64) float av[16];
                _mm512_store_ps(av, alpha);
                for (int h = 0; h < G; ++h) {
                    if (av[h] == 1.f) continue;
                    const __m512 a = _mm512_set1_ps(av[h]);
                    float* row = obuf + size_t(h) * dv;
                    for (int c = 0; c < dv; c += 16) _mm512_store_ps(row + c, _mm512_mul_ps(_mm512_load_ps(row + c), a));
                }
            }
            _tile_loadd(4, p_hi, 64);
            _tile_loadd(5, p_lo, 64);
            for (int cb0 = 0; cb0 < n_cb; cb0 += 4) {
                const int nb = std::min(4, n_cb - cb0);
                prefetch_some();
                // (tile numbers are immediates: the four column blocks are written out)
                _tile_loadd(0, obuf + (cb0 + 0) * 16, dv * 4);
                _tile_loadd(6, vn + size_t(cb0 + 0) * 16 * 32, 64);
                _tile_dpbf16ps(0, 4, 6);
                _tile_dpbf16ps(0, 5, 6);
                _tile_stored(0, obuf + (cb0 + 0) * 16, dv * 4);
                if (nb > 1) {
                    _tile_loadd(1, obuf + (cb0 + 1) * 16, dv * 4);
                    _tile_loadd(7, vn + size_t(cb0 + 1) * 16 * 32, 64);
                    _tile_dpbf16ps(1, 4, 7);
                    _tile_dpbf16ps(1, 5, 7);
                    _tile_stored(1, obuf + (cb0 + 1) * 16, dv * 4);
                }
                if (nb > 2) {
                    _tile_loadd(2, obuf + (cb0 + 2) * 16, dv * 4);
                    _tile_loadd(6, vn + size_t(cb0 + 2) * 16 * 32, 64);
                    _tile_dpbf16ps(2, 4, 6);
                    _tile_dpbf16ps(2, 5, 6);
                    _tile_stored(2, obuf + (cb0 + 2) * 16, dv * 4);
                }
                if (nb > 3) {
                    _tile_loadd(3, obuf + (cb0 + 3) * 16, dv * 4);
                    _tile_loadd(7, vn + size_t(cb0 + 3) * 16 * 32, 64);
                    _tile_dpbf16ps(3, 4, 7);
                    _tile_dpbf16ps(3, 5, 7);
                    _tile_stored(3, obuf + (cb0 + 3) * 16, dv * 4);
                }
            }
        }
        run_first = run_last;
    }
    _tile_release();
    alignas(64) float mv[16], lv[16];
    _mm512_store_ps(mv, m_run);
    _mm512_store_ps(lv, l_run);
    for (int h = 0; h < G; ++h) {
        m[h] = mv[h];
        l[h] = lv[h];
        std::memcpy(o + size_t(h) * dv, obuf + size_t(h) * dv, size_t(dv) * 4);
    }
}

}  // namespace ipkvi
