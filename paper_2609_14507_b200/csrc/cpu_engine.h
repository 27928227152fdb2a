// Interface of the CPU-side in-place attention engine (cpu_engine.cpp), used by the C ABI.
#pragma once
#include <cstdint>

namespace ipkvi {

constexpr int kCpuMaxDim = 576;      // widest head dimension the tile kernel holds
constexpr int kCpuMaxGroup = 128;    // most query heads sharing one KV head (compressed latent: all heads)

struct CpuShape {
    int n_q_heads, n_kv_heads, dim_qk, dim_v;
    int dim_v_stored;     // 0 for the compressed-latent kind: V aliases the first dim_v columns of K
    int bt;               // tokens per block
    float scale;
};
// A run of contiguous PLAIN-layout blocks in host memory holding n_tokens tokens.
struct CpuRun {
    const char* blocks;
    int64_t n_tokens;
};

// Attention of n_rows queries (bf16 bits, [n_rows][Hq][dqk]) over the runs of each row; fp32 normalised O
// [n_rows][Hq][dv] and natural-log LSE [n_rows][Hq]. Returns 0, or -1 for unsupported shapes.
int cpu_attend_batch(const CpuShape& sh, int n_rows, const uint16_t* q, const CpuRun* runs, const int32_t* row_run_start,
                     float* o_out, float* lse_out, int n_threads);
int cpu_engine_threads();
// Which tile kernel cpu_attend_batch uses for this shape on this host: "amx", "v4", "v3" or "base".
const char* cpu_engine_kernel_name(const CpuShape& sh);

}  // namespace ipkvi
