// Internal launch interface between the host scheduler (api.cu) and the CUDA kernels.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <cstdlib>

#include "layout.cuh"

namespace ipkvi {

// One run of contiguous TILE-layout blocks that a row attends to; address = bases[base_id] + off.
struct Seg {
    int64_t off;
    int32_t n_tokens;
    int32_t base_id;     // index into bases (low byte); kSegAppended: the run's last token is written by this launch
};
// Fused append (grouped-query kernel): the last token of a flagged run is not in memory yet. The launch carries the
// new K/V rows; the consumer warp that owns the token's 16-token slice writes them into the shared-memory tile once
// its copy has landed (and into the run itself, for the launches to come), then computes as usual.
constexpr int32_t kSegAppended = 0x100;
constexpr int32_t kSegBaseMask = 0xff;
// The run's token count in the table is rounded up to whole 64-token tiles; the real count is that minus 64 plus the
// launch parameter win_tail (1..64).  Set on the D-window runs of a launch when all of them end at the same offset inside
// their last tile, which is the case while a batch decodes in lockstep: the table then stays the same from step to step
// (only win_tail moves) until a window grows into a new tile or is evicted, and need not be uploaded again.
constexpr int32_t kSegTailParam = 0x200;
constexpr int32_t kSegBaseWindow = 1;     // bases[1] is the layer's D-window (bases[0] the resident ring, bases[2] the slots)
// One span of split-K work: tiles [tile0, tile0 + ntiles) of segment `seg` for query row `row` and head
// group `gh`.  A CTA processes a contiguous range of spans back to back; the partial(s) a span produces are
// stored at the span's own index.
struct Span {
    int32_t row, gh, seg, tile0, ntiles;
};

constexpr int kMaxBases = 4;

// Bits of the device status word: which bounded wait of a kernel gave up.
constexpr uint32_t kStatusNoFreeStage = 1u;     // the producer waited for the consumers to release a stage
constexpr uint32_t kStatusNoTile = 2u;          // a consumer waited for a tile (or the end marker) to arrive
constexpr uint32_t kStatusCopyNotLanded = 4u;   // the producer waited for its last copies before leaving
constexpr uint32_t kStatusBadIndex = 8u;        // bounds-checked build only: a computed address left its region (the access was not made)

// Bounds-checked build (-DIPKV_CHECKED; the stand-in for a memory checker): every source address the attention kernels
// compute for a copy, every partial row they store and every window slot the append paths write is compared with the
// extent of the region it must lie in.  A violation sets kStatusBadIndex in the status word and the access is redirected
// to the start of the region (reads) or dropped (writes): nothing traps, nothing reads or writes out of bounds.
#ifdef IPKV_CHECKED
constexpr bool kChecked = true;
#else
constexpr bool kChecked = false;
#endif

struct AttnLaunch {
    int kind;                       // 0 = GQA, 1 = compressed latent (MLA)
    int n_q_heads, n_kv_heads, dim_qk, dim_v, bt;
    float scale;                    // softmax scale applied to fp32 scores
    const void* q;                  // [n_rows][Hq][dqk] bf16
    const char* bases[kMaxBases];
    const Seg* segs;                // device tables (see plan.hpp)
    const Span* spans;
    const int32_t* cta_span_start;  // [n_ctas + 1]
    const int32_t* rg_span_start;   // [n_rows * n_gh + 1]
    const int32_t* cta_tiles;       // [n_ctas] tiles per chunk
    int n_spans, n_ctas, n_rows, n_gh;
    float* part_o;                  // [n_spans * parts_per_span][rows_per_group][dv]
    float* part_lse;                // [n_spans * parts_per_span][rows_per_group]
    const float* acc_o;             // optional earlier partial to fold in, [n_rows][Hq][dv]
    const float* acc_lse;
    float* out_o;                   // [n_rows][Hq][dv]
    float* out_lse;                 // [n_rows][Hq]
    uint32_t* status;               // device word, OR-ed with an error bit if a bounded wait gives up
    const void* append_k;           // fused append: [n_rows][n_kv_heads][dim_qk] bf16 new K rows (null: none)
    const void* append_v;           // [n_rows][n_kv_heads][dim_v]
    int64_t base_bytes[kMaxBases];  // extent of the memory behind every base (0: unknown, not checked); used by the checked build
    int64_t part_rows;              // rows of (O, LSE) partial storage behind part_o / part_lse
    int parts_per_span;             // partials every span writes in this launch (plan.hpp: parts_per_span_for)
    int win_tail;                   // valid tokens in the last tile of the runs flagged kSegTailParam (1..64)
    int plain_launch;               // 1: the tables were written by the kernel right in front of this launch: no launch overlap
    int early_tiles;                // nonzero: no ring byte this launch reads (2: no window byte either) was written by the kernel
                                    // before it in the stream, so the first copies of such tiles may be issued before that
                                    // kernel has completed (see launch.cuh)
    // Dynamic load balancing of the GQA kernel (all null = static schedule with bit-reproducible results): a CTA
    // that has finished its chunk takes tiles from the spans that are furthest behind and accumulates them into
    // extra partials of its own, stored after the spans' partials (kStealSlots per CTA) and listed per (row, head group).
    int32_t* steal_next;            // [n_spans + 2 * n_ctas]: tiles claimed so far of every span, tiles claimed of every CTA's
                                    // chunk, CTAs that came to help with every chunk; zero when the kernel starts
    int32_t* steal_lists;           // [n_rows * n_gh] number of extra partials of every (row, head group), then
                                    // [n_rows * n_gh][kStealListCap] their indices; zero when the kernel starts
    int32_t* steal_clear;           // words the split reduce sets to zero for the launch after this one
    int steal_clear_words;
};
constexpr int kStealSlots = 4;      // extra partials a CTA can fill
constexpr int kStealListCap = 16;   // extra partials a (row, head group) can take

// Geometry of the partial buffers: query heads per head group (rows of one partial), head groups per row,
// partials per span at most (sizes the scratch; one per consumer warp for GQA unless the launch joins them, one for MLA), resident CTAs per SM.
struct PartGeom {
    int rows_per_group, n_gh, parts_per_span, ctas_per_sm;
};

inline PartGeom part_geom(int kind, int Hq, int Hkv) {
    PartGeom g;
    if (kind == 1) { g.rows_per_group = 16; g.n_gh = (Hq + 15) / 16; g.parts_per_span = 1; g.ctas_per_sm = 1; }
    else {
        const int G = Hq / Hkv;
        g.rows_per_group = G < 16 ? G : 16;
        g.n_gh = Hkv * ((G + 15) / 16);
        g.parts_per_span = 4;
        g.ctas_per_sm = 2;
    }
    return g;
}

// Split-K attention: partial (O, LSE) per span, rows = the query heads of the span's group.
cudaError_t launch_attend(const AttnLaunch& a, cudaStream_t s);
// Second pass: per (row, head) LSE-reduce the partials of its head group's spans (and acc_*, if given) into out_*.
cudaError_t launch_split_reduce(const AttnLaunch& a, cudaStream_t s);

constexpr int kMaxMergeParts = 8;
struct MergeLaunch {
    const float* o[kMaxMergeParts];
    const float* lse[kMaxMergeParts];
    int n_parts, n_rows, dim_v;
    void* out_o;
    int out_is_bf16;
    float* out_lse;                 // may be null
};
cudaError_t launch_merge(const MergeLaunch& m, cudaStream_t s);

// Token-major K/V -> blocks. dst_token0 = token offset (in the destination's block space) of src token 0.
cudaError_t launch_pack(const BlockGeom& g, int layout_tile, const void* k, const void* v, int64_t n_tokens,
                        void* dst, int64_t dst_token0, cudaStream_t s);
// TILE-layout blocks -> PLAIN-layout blocks (eviction of a window batch to the CPU-compute region).
cudaError_t launch_tile_to_plain(const BlockGeom& g, const void* src, void* dst, int64_t n_blocks, cudaStream_t s);

// Several device-to-device copies in one launch (refreshing the resident ring after an eviction): 16-byte chunks.
constexpr int kCopySpansPerLaunch = 64;
struct CopySpans {
    const char* src[kCopySpansPerLaunch];
    char* dst[kCopySpansPerLaunch];
    int64_t bytes[kCopySpansPerLaunch];      // multiples of 16
};
cudaError_t launch_copy_spans(const CopySpans& spans, int n, cudaStream_t s);
// Writes `bytes` (a multiple of 16) of host data to device memory with kernels that carry the data as launch
// parameters: unlike a copy from pageable memory, such a launch keeps nothing but a value, so it can be recorded
// into a CUDA graph and replayed after the host buffer is gone.
cudaError_t launch_upload_by_value(void* dst_dev, const void* src_host, size_t bytes, cudaStream_t s);

// Self-test: a one-CTA kernel whose consumer waits `limit_ns` for a tile that is announced and never copied, gives up
// and ORs kStatusNoTile into *status (probe.cu).
cudaError_t launch_expire_wait(uint32_t* status, uint64_t limit_ns, cudaStream_t s);

constexpr int kAppendRowsPerLaunch = 64;
struct AppendRows {
    int64_t dst_off[kAppendRowsPerLaunch];   // byte offset of the row's window (first block) from w_base
    int32_t slot[kAppendRowsPerLaunch];      // token slot inside the window
};
// One new token per row into its D-window (TILE layout). k/v point at the first row of this launch.
// w_bytes / status: extent of the layer's windows and the status word, for the bounds-checked build (0 / null: unchecked).
cudaError_t launch_append(const BlockGeom& g, const void* k, const void* v, int dim_v_src, char* w_base,
                          const AppendRows& rows, int n_rows, cudaStream_t s, int64_t w_bytes = 0, uint32_t* status = nullptr);

}  // namespace ipkvi
