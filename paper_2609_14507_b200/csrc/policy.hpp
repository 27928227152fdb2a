// Roofline share policy (Sec. 5.2-5.3): the analytic latency model of the two engines, the balanced CPU
// share it implies, and the online feedback that tracks the CPU's per-token cost.
//
//   Eq. 1   T_CPU(r) = r A L + C_CPU,   T_GPU(r) = (1 - r) B L + C_GPU,   T = max(T_CPU, T_GPU) + T_merge
//   Eq. 2   r(L) = min(1, max(0, B / (A + B) + Delta / ((A + B) L))),   Delta = C_GPU - C_CPU
//   marginal share of decode eviction batches: p = B / (A + B), the limit of r(L)
//   feedback: the CPU engine's per-step latency is averaged over a sliding window of steps and A is
//   back-computed from T_CPU = A * (CPU-side tokens) + C_CPU; B is calibrated once.
//
// Host-only; its output is an integer numerator for the router, so routing itself stays integer-exact.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <vector>

namespace ipkvi {

struct RooflineParams {
    double A, B;          // seconds per KV token: CPU in-place read cost, GPU transfer cost
    double C_cpu, C_gpu;  // fixed per-step overheads, seconds
};

inline double engine_time_cpu(const RooflineParams& m, double r, double L) { return r * m.A * L + m.C_cpu; }
inline double engine_time_gpu(const RooflineParams& m, double r, double L) { return (1.0 - r) * m.B * L + m.C_gpu; }
inline double step_time(const RooflineParams& m, double r, double L, double t_merge) {
    return std::max(engine_time_cpu(m, r, L), engine_time_gpu(m, r, L)) + t_merge;
}
inline double marginal_share(const RooflineParams& m) { return m.B / (m.A + m.B); }
inline double balanced_share(const RooflineParams& m, double L) {
    if (!(L > 0.0)) return std::min(1.0, std::max(0.0, marginal_share(m)));
    const double r = m.B / (m.A + m.B) + (m.C_gpu - m.C_cpu) / ((m.A + m.B) * L);
    return std::min(1.0, std::max(0.0, r));
}

class SharePolicy {
public:
    SharePolicy(const RooflineParams& m, int window_steps, int share_den)
        : m_(m), den_(share_den), win_(size_t(std::max(1, window_steps))) {}

    const RooflineParams& model() const { return m_; }
    int den() const { return den_; }
    int samples() const { return int(std::min(count_, win_.size())); }

    // One decode step of the CPU engine: its latency and the number of CPU-side KV tokens it attended.
    void observe(double cpu_seconds, double cpu_tokens) {
        Sample& s = win_[count_ % win_.size()];
        if (count_ >= win_.size()) { sum_t_ -= s.t; sum_n_ -= s.n; }
        s.t = cpu_seconds; s.n = cpu_tokens;
        sum_t_ += cpu_seconds; sum_n_ += cpu_tokens;
        ++count_;
    }

    // Back-compute A from the sliding averages and return the numerator of the marginal share p = B / (A + B)
    // over den (round to nearest). Without samples (or with no CPU-side tokens yet) A keeps its calibrated value.
    int update() {
        const double n = double(samples());
        if (n > 0 && sum_n_ > 0.0) {
            const double a = (sum_t_ - n * m_.C_cpu) / sum_n_;
            if (a > 0.0 && std::isfinite(a)) m_.A = a;
        }
        return numerator(marginal_share(m_));
    }

    // Prefill share R(L0) = r(L0) as a numerator over den.
    int prefill_numerator(double L0) const { return numerator(balanced_share(m_, L0)); }

private:
    int numerator(double share) const {
        const long v = std::lround(share * den_);
        return int(std::min<long>(den_, std::max<long>(0, v)));
    }
    struct Sample { double t = 0.0, n = 0.0; };
    RooflineParams m_;
    int den_;
    std::vector<Sample> win_;
    size_t count_ = 0;
    double sum_t_ = 0.0, sum_n_ = 0.0;
};

}  // namespace ipkvi
