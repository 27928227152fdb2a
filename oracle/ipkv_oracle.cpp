// TEST INFRASTRUCTURE — not part of the product.
//
// Plain, slow, float64 CPU oracle for the sequence-split decode-attention path of the
// InplaceKVCache / WriteScope method.  Only the test-suite, the smoke check and the
// benchmark's CPU-baseline leg may load this library; the CUDA library never does, and
// the two share no source.
//
//   O1  oracle_attend      full softmax attention of one decode query over a token SET
//                          (the textbook definition; the paper's Sec. 4.3 guarantee (iv)
//                          and Sec. 5.1 say the method is exact, so the definition IS the
//                          expected result).  Two passes, no online softmax, no tiling.
//   O2  oracle_merge       exact log-sum-exp join of partial (O, LSE) pairs computed over
//                          disjoint token sets (Sec. 4.2 "merged via LSE rescaling",
//                          Sec. 5.1 "merge exactly").
//   O3  oracle_route_*     pure-integer simulator of write-time routing into the four
//                          regions (Sec. 4.1 regions and blocks, Sec. 4.2 prefill one-shot
//                          routing, D-window staging and whole-batch eviction, Sec. 5.3
//                          constant marginal share p).
//
// Readings the paper leaves open and this oracle fixes (parity for these choices is
// "unpinned by the paper": any consistent choice satisfies every printed statement):
//   * the phase / tie-break of the per-batch routing rule: an integer error-diffusion
//     accumulator started at floor(den/2) (round-half-up of k*p);
//   * the flush fires lazily, at the start of the append that finds the window full;
//   * block size is a parameter; the prefill CPU share is the OLDEST tokens, floored to
//     whole blocks.
//
// bf16 values travel as raw uint16 bit patterns and are widened exactly to double.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

inline double bf16_to_double(uint16_t bits) {
    uint32_t w = static_cast<uint32_t>(bits) << 16;
    float f;
    std::memcpy(&f, &w, sizeof f);
    return static_cast<double>(f);
}

const double NEG_INF = -std::numeric_limits<double>::infinity();

}  // namespace

extern "C" {

int oracle_num_threads() {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

// O1.  Attention of one sequence's decode query over the token set idx[0..n_idx).
//   q  [Hq][dqk]            bf16 bits
//   k  [n_store][Hkv][dqk]  bf16 bits, token-major
//   v  [n_store][Hkv][dv]   bf16 bits; NULL means the compressed-latent (MLA) case where
//                           V[j] = K[j][0:dv]  (Sec. 6.1, compressed-MLA variant: every head
//                           shares one latent, the value is its leading columns)
//   query head h reads KV head floor(h / (Hq/Hkv))  (contiguous GQA groups)
//   scores are scale * <q_h, K_j>;  LSE is the natural log of the sum of exp(scores)
//   Empty set: O = 0, LSE = -inf.
// Returns 0, or -1 on bad arguments.
int oracle_attend(const uint16_t* q, const uint16_t* k, const uint16_t* v,
                  int Hq, int Hkv, int dqk, int dv,
                  const int64_t* idx, int64_t n_idx, double scale,
                  double* O, double* lse) {
    if (!q || !O || !lse || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || dqk <= 0 || dv <= 0) return -1;
    if (n_idx < 0 || (n_idx > 0 && (!k || !idx))) return -1;
    if (!v && dv > dqk) return -1;
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int h = 0; h < Hq; ++h) {
        const int g = h / G;
        double* Oh = O + static_cast<int64_t>(h) * dv;
        for (int c = 0; c < dv; ++c) Oh[c] = 0.0;
        if (n_idx == 0) {
            lse[h] = NEG_INF;
            continue;
        }
        std::vector<double> qd(dqk), s(static_cast<size_t>(n_idx));
        for (int i = 0; i < dqk; ++i) qd[i] = bf16_to_double(q[static_cast<int64_t>(h) * dqk + i]);
        // pass 1: all scores, then their maximum
        double m = NEG_INF;
        for (int64_t j = 0; j < n_idx; ++j) {
            const uint16_t* kj = k + (idx[j] * Hkv + g) * static_cast<int64_t>(dqk);
            double acc = 0.0;
            for (int i = 0; i < dqk; ++i) acc += qd[i] * bf16_to_double(kj[i]);
            s[j] = scale * acc;
            if (s[j] > m) m = s[j];
        }
        // pass 2: weights, normaliser, weighted values
        double l = 0.0;
        for (int64_t j = 0; j < n_idx; ++j) {
            const double w = std::exp(s[j] - m);
            l += w;
            const uint16_t* vj = v ? v + (idx[j] * Hkv + g) * static_cast<int64_t>(dv)
                                   : k + (idx[j] * Hkv + g) * static_cast<int64_t>(dqk);
            for (int c = 0; c < dv; ++c) Oh[c] += w * bf16_to_double(vj[c]);
        }
        for (int c = 0; c < dv; ++c) Oh[c] /= l;
        lse[h] = m + std::log(l);
    }
    return 0;
}

// O2.  n-way exact merge of row-aligned partials over disjoint token sets.
//   O_parts[i]  [n_rows][dv], lse_parts[i] [n_rows]
//   LSE = m + ln sum_i exp(LSE_i - m), m = max_i LSE_i;  O = sum_i exp(LSE_i - LSE) O_i
//   Parts with LSE_i = -inf contribute nothing; all -inf gives (0, -inf).
int oracle_merge(int n_rows, int dv, int n_parts,
                 const double* const* O_parts, const double* const* lse_parts,
                 double* O, double* lse) {
    if (n_rows < 0 || dv <= 0 || n_parts < 0 || !O || !lse) return -1;
    for (int r = 0; r < n_rows; ++r) {
        double m = NEG_INF;
        for (int i = 0; i < n_parts; ++i)
            if (lse_parts[i][r] > m) m = lse_parts[i][r];
        double* Or = O + static_cast<int64_t>(r) * dv;
        for (int c = 0; c < dv; ++c) Or[c] = 0.0;
        if (m == NEG_INF) {
            lse[r] = NEG_INF;
            continue;
        }
        double z = 0.0;
        for (int i = 0; i < n_parts; ++i) z += std::exp(lse_parts[i][r] - m);
        const double L = m + std::log(z);
        for (int i = 0; i < n_parts; ++i) {
            if (lse_parts[i][r] == NEG_INF) continue;
            const double w = std::exp(lse_parts[i][r] - L);
            const double* Oi = O_parts[i] + static_cast<int64_t>(r) * dv;
            for (int c = 0; c < dv; ++c) Or[c] += w * Oi[c];
        }
        lse[r] = L;
    }
    return 0;
}

// O3.  Routing simulator for ONE (layer, sequence); all integers.
struct oracle_route {
    int64_t block, D, num, den, acc;
    std::vector<int8_t> region;   // per token: 0 = U (host unpinned, CPU compute),
                                  //            1 = P (host pinned, GPU load), 2 = W (D-window)
    std::vector<int64_t> blk;     // ordinal of the token's block inside its region
    std::vector<int32_t> off;     // offset of the token inside that block (W: slot index)
    int64_t u_blocks, p_blocks;   // blocks handed out so far in U and P
    int64_t w0;                   // first token held by the window; window = [w0, n)
    int64_t n_flush, n_flush_cpu;
};

oracle_route* oracle_route_new(int64_t block, int64_t D, int64_t num, int64_t den) {
    if (block <= 0 || D <= 0 || D % block != 0 || den <= 0 || num < 0 || num > den) return nullptr;
    oracle_route* r = new oracle_route();
    r->block = block; r->D = D; r->num = num; r->den = den; r->acc = den / 2;
    r->u_blocks = r->p_blocks = 0; r->w0 = 0; r->n_flush = r->n_flush_cpu = 0;
    return r;
}

void oracle_route_free(oracle_route* r) { delete r; }

int oracle_route_set_share(oracle_route* r, int64_t num) {
    if (!r || num < 0 || num > r->den) return -1;
    r->num = num;
    return 0;
}

// place tokens [first, first+count) into region reg, starting at its next block boundary
static void place_run(oracle_route* r, int reg, int64_t first, int64_t count) {
    int64_t& next = (reg == 0) ? r->u_blocks : r->p_blocks;
    for (int64_t t = 0; t < count; ++t) {
        r->region[first + t] = static_cast<int8_t>(reg);
        r->blk[first + t] = next + t / r->block;
        r->off[first + t] = static_cast<int32_t>(t % r->block);
    }
    next += (count + r->block - 1) / r->block;
}

// Prefill: n0 tokens in one shot at share num0/den0; legal only on an empty sequence.
// CPU gets the oldest n_cpu = block * floor(floor(n0/block) * num0 / den0) tokens.
int oracle_route_bulk(oracle_route* r, int64_t n0, int64_t num0, int64_t den0) {
    if (!r || !r->region.empty() || n0 < 0 || den0 <= 0 || num0 < 0 || num0 > den0) return -1;
    const int64_t n_cpu = r->block * (((n0 / r->block) * num0) / den0);
    r->region.resize(n0); r->blk.resize(n0); r->off.resize(n0);
    place_run(r, 0, 0, n_cpu);
    place_run(r, 1, n_cpu, n0 - n_cpu);
    r->w0 = n0;
    return 0;
}

// Evict the whole window as one batch; destination by error diffusion at share num/den.
int oracle_route_flush(oracle_route* r) {
    if (!r) return -1;
    const int64_t n = static_cast<int64_t>(r->region.size());
    const int64_t cnt = n - r->w0;
    if (cnt == 0) return 0;
    r->acc += r->num;
    int dest = 1;
    if (r->acc >= r->den) { r->acc -= r->den; dest = 0; }
    place_run(r, dest, r->w0, cnt);
    r->w0 = n;
    r->n_flush += 1;
    r->n_flush_cpu += (dest == 0);
    return 0;
}

// Decode: one new token; a full window is evicted first, so the newest token is always in W.
int oracle_route_append(oracle_route* r) {
    if (!r) return -1;
    int64_t n = static_cast<int64_t>(r->region.size());
    if (n - r->w0 == r->D) oracle_route_flush(r);
    r->region.push_back(2);
    r->blk.push_back(0);
    r->off.push_back(static_cast<int32_t>(n - r->w0));
    return 0;
}

int64_t oracle_route_len(const oracle_route* r) { return r ? static_cast<int64_t>(r->region.size()) : -1; }

// counts[0..2] = tokens in U, P, W; counts[3..4] = blocks handed out in U, P;
// counts[5..6] = flushes so far, of which to U.
int oracle_route_counts(const oracle_route* r, int64_t counts[7]) {
    if (!r) return -1;
    counts[0] = counts[1] = counts[2] = 0;
    for (int8_t g : r->region) counts[g] += 1;
    counts[3] = r->u_blocks; counts[4] = r->p_blocks;
    counts[5] = r->n_flush; counts[6] = r->n_flush_cpu;
    return 0;
}

int oracle_route_dump(const oracle_route* r, int8_t* region, int64_t* blk, int32_t* off) {
    if (!r) return -1;
    const size_t n = r->region.size();
    if (n) {
        std::memcpy(region, r->region.data(), n * sizeof(int8_t));
        std::memcpy(blk, r->blk.data(), n * sizeof(int64_t));
        std::memcpy(off, r->off.data(), n * sizeof(int32_t));
    }
    return 0;
}

}  // extern "C"
