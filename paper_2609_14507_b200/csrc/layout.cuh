// Block layouts of the four-region format (Sec. 4.1: "each region is internally organized in
// fixed-size blocks") and the index arithmetic shared by the host scheduler and the kernels.
//
// PLAIN (region U, read by a CPU engine): per KV head, K[bt][dqk] then V[bt][dv], row-major.
// TILE  (P, W, PP, resident ring; read by the GPU): per KV head, K plane then V plane; a plane of
//   width d is d/64 panels of bt rows x 128 bytes, and inside a row the 16-byte chunk c of token
//   offset t sits at chunk position c ^ (t & 7).  A 64-token tile of one head therefore reaches
//   shared memory by plain contiguous bulk copies and is read by ldmatrix without bank conflicts.
#pragma once
#include <cstdint>

#if defined(__CUDACC__)
#define IPKV_HD __host__ __device__ __forceinline__
#else
#define IPKV_HD inline
#endif

namespace ipkvi {

constexpr int kTileTokens = 64;   // tokens per shared-memory tile of the attention kernels
constexpr int kPanelCols = 64;    // bf16 columns per panel (128 bytes)

struct BlockGeom {
    int32_t n_kv_heads, dim_qk, dim_v_stored;   // dim_v_stored = 0 for the compressed-latent kind
    int32_t bt;                                 // tokens per block
    IPKV_HD int64_t k_plane_bytes() const { return int64_t(bt) * dim_qk * 2; }
    IPKV_HD int64_t v_plane_bytes() const { return int64_t(bt) * dim_v_stored * 2; }
    IPKV_HD int64_t head_bytes() const { return k_plane_bytes() + v_plane_bytes(); }
    IPKV_HD int64_t block_bytes() const { return head_bytes() * n_kv_heads; }
};

// Byte offset inside a TILE-layout plane of the 16-byte chunk `chunk` (0 .. d/8-1) of token offset t.
IPKV_HD int64_t tile_chunk_offset(int32_t bt, int32_t t, int32_t chunk) {
    return int64_t(chunk >> 3) * (int64_t(bt) * 128) + int64_t(t) * 128 + (((chunk & 7) ^ (t & 7)) << 4);
}
// Byte offset inside a PLAIN-layout plane of width d.
IPKV_HD int64_t plain_chunk_offset(int32_t d, int32_t t, int32_t chunk) {
    return (int64_t(t) * d + int64_t(chunk) * 8) * 2;
}

}  // namespace ipkvi
