// Data-movement kernels of write-time routing (Sec. 4.2): every K/V entry is laid out once, at write
// time, in the layout of the region that will consume it, and never reorganised afterwards.
//   pack_kernel          prefill K/V (token-major) -> blocks of the destination region's layout
//   append_kernel        one new decode token per sequence -> its D-window slot (TILE layout)
//   tile_to_plain_kernel an evicted window batch, TILE -> PLAIN, on its way to the CPU-compute region
// All three move 16-byte chunks; one thread per chunk, consecutive threads on consecutive source chunks.
// (Also here: upload_by_value_kernel, which writes launch tables carried as kernel parameters, for calls recorded into a
// CUDA graph.)
#include <cstring>

#include "kernels.h"
#include "launch.cuh"
#include "ptx.cuh"

namespace ipkvi {

namespace {

__global__ void pack_kernel(BlockGeom g, int layout_tile, const uint4* __restrict__ k, const uint4* __restrict__ v,
                            int64_t n_tokens, char* __restrict__ dst, int64_t dst_token0) {
    const int kc = g.dim_qk / 8, vc = g.dim_v_stored / 8;       // chunks per row
    const int per_head = kc + vc;
    const int64_t per_token = int64_t(per_head) * g.n_kv_heads;
    const int64_t total = n_tokens * per_token;
    for (int64_t i = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; i < total; i += int64_t(gridDim.x) * blockDim.x) {
        const int64_t t = i / per_token;
        const int rem = int(i - t * per_token);
        // source order inside a token: all K chunks of all heads, then all V chunks of all heads
        int head, chunk;
        bool is_v;
        if (rem < kc * g.n_kv_heads) { is_v = false; head = rem / kc; chunk = rem - head * kc; }
        else { const int r2 = rem - kc * g.n_kv_heads; is_v = true; head = r2 / vc; chunk = r2 - head * vc; }
        const uint4 val = is_v ? v[(t * g.n_kv_heads + head) * vc + chunk] : k[(t * g.n_kv_heads + head) * kc + chunk];
        const int64_t td = dst_token0 + t;
        const int64_t blk = td / g.bt;
        const int toff = int(td - blk * g.bt);
        int64_t off = blk * g.block_bytes() + int64_t(head) * g.head_bytes() + (is_v ? g.k_plane_bytes() : 0);
        off += layout_tile ? tile_chunk_offset(g.bt, toff, chunk)
                           : plain_chunk_offset(is_v ? g.dim_v_stored : g.dim_qk, toff, chunk);
        *reinterpret_cast<uint4*>(dst + off) = val;
    }
}

__global__ void tile_to_plain_kernel(BlockGeom g, const char* __restrict__ src, char* __restrict__ dst, int64_t n_blocks) {
    const int64_t chunks_per_block = g.block_bytes() / 16;
    const int64_t total = n_blocks * chunks_per_block;
    const int kc = g.dim_qk / 8, vc = g.dim_v_stored / 8;
    const int64_t head_chunks = int64_t(g.bt) * (kc + vc);
    for (int64_t i = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; i < total; i += int64_t(gridDim.x) * blockDim.x) {
        // enumerate the PLAIN destination in order (coalesced writes), gather from the TILE source
        const int64_t blk = i / chunks_per_block;
        int64_t r = i - blk * chunks_per_block;
        const int head = int(r / head_chunks);
        r -= head * head_chunks;
        const bool is_v = r >= int64_t(g.bt) * kc;
        if (is_v) r -= int64_t(g.bt) * kc;
        const int c = is_v ? vc : kc;
        const int t = int(r / c), chunk = int(r - int64_t(t) * c);
        const int64_t base = blk * g.block_bytes() + int64_t(head) * g.head_bytes() + (is_v ? g.k_plane_bytes() : 0);
        const uint4 val = *reinterpret_cast<const uint4*>(src + base + tile_chunk_offset(g.bt, t, chunk));
        *reinterpret_cast<uint4*>(dst + base + plain_chunk_offset(is_v ? g.dim_v_stored : g.dim_qk, t, chunk)) = val;
    }
}

__global__ void append_kernel(BlockGeom g, const uint4* __restrict__ k, const uint4* __restrict__ v,
                              char* __restrict__ w_base, AppendRows rows, int64_t w_bytes, uint32_t* status) {
    ptx::grid_dependency_wait();       // launched so that it may come in under the previous kernel's tail (launch.cuh)
    ptx::grid_launch_dependents();
    const int row = blockIdx.x;
    const int kc = g.dim_qk / 8, vc = g.dim_v_stored / 8;
    const int per_token = (kc + vc) * g.n_kv_heads;
    const int slot = rows.slot[row];
    const int64_t blk = slot / g.bt;
    const int toff = slot - int(blk) * g.bt;
    char* win = w_base + rows.dst_off[row] + blk * g.block_bytes();
    if (kChecked && w_bytes > 0 && (slot < 0 || rows.dst_off[row] < 0 || rows.dst_off[row] + (blk + 1) * g.block_bytes() > w_bytes)) {
        if (threadIdx.x == 0) atomicOr(status, kStatusBadIndex);      // the slot's block must lie inside the layer's windows
        return;
    }
    for (int i = threadIdx.x; i < per_token; i += blockDim.x) {
        int head, chunk;
        bool is_v;
        if (i < kc * g.n_kv_heads) { is_v = false; head = i / kc; chunk = i - head * kc; }
        else { const int r2 = i - kc * g.n_kv_heads; is_v = true; head = r2 / vc; chunk = r2 - head * vc; }
        const uint4 val = is_v ? v[(int64_t(row) * g.n_kv_heads + head) * vc + chunk]
                               : k[(int64_t(row) * g.n_kv_heads + head) * kc + chunk];
        const int64_t off = int64_t(head) * g.head_bytes() + (is_v ? g.k_plane_bytes() : 0) + tile_chunk_offset(g.bt, toff, chunk);
        *reinterpret_cast<uint4*>(win + off) = val;
    }
}

__global__ void copy_spans_kernel(CopySpans sp) {
    const int k = blockIdx.y;
    const uint4* src = reinterpret_cast<const uint4*>(sp.src[k]);
    uint4* dst = reinterpret_cast<uint4*>(sp.dst[k]);
    const int64_t n = sp.bytes[k] / 16;
    for (int64_t i = blockIdx.x * int64_t(blockDim.x) + threadIdx.x; i < n; i += int64_t(gridDim.x) * blockDim.x) dst[i] = src[i];
}

constexpr int kUploadChunk = 16384;             // bytes of data per launch (kernel parameters may be up to 32 764 bytes on this architecture)
struct UploadChunk { uint4 v[kUploadChunk / 16]; };

__global__ void upload_by_value_kernel(UploadChunk c, uint4* dst, int n16) {
    ptx::grid_dependency_wait();
    ptx::grid_launch_dependents();
    for (int i = threadIdx.x; i < n16; i += blockDim.x) dst[i] = c.v[i];
}

int grid_for(int64_t total, int threads) {
    int64_t b = (total + threads - 1) / threads;
    const int64_t cap = 148 * 16;
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return int(b);
}

}  // namespace

cudaError_t launch_pack(const BlockGeom& g, int layout_tile, const void* k, const void* v, int64_t n_tokens,
                        void* dst, int64_t dst_token0, cudaStream_t s) {
    if (n_tokens <= 0) return cudaSuccess;
    const int64_t total = n_tokens * g.n_kv_heads * ((g.dim_qk + g.dim_v_stored) / 8);
    pack_kernel<<<grid_for(total, 256), 256, 0, s>>>(g, layout_tile, static_cast<const uint4*>(k), static_cast<const uint4*>(v),
                                                     n_tokens, static_cast<char*>(dst), dst_token0);
    return cudaGetLastError();
}

cudaError_t launch_tile_to_plain(const BlockGeom& g, const void* src, void* dst, int64_t n_blocks, cudaStream_t s) {
    if (n_blocks <= 0) return cudaSuccess;
    const int64_t total = n_blocks * (g.block_bytes() / 16);
    tile_to_plain_kernel<<<grid_for(total, 256), 256, 0, s>>>(g, static_cast<const char*>(src), static_cast<char*>(dst), n_blocks);
    return cudaGetLastError();
}

cudaError_t launch_copy_spans(const CopySpans& spans, int n, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    int64_t longest = 0;
    for (int i = 0; i < n; ++i) longest = spans.bytes[i] > longest ? spans.bytes[i] : longest;
    dim3 grid(grid_for(longest / 16, 256) > 64 ? 64 : grid_for(longest / 16, 256), n);
    copy_spans_kernel<<<grid, 256, 0, s>>>(spans);
    return cudaGetLastError();
}

cudaError_t launch_upload_by_value(void* dst_dev, const void* src_host, size_t bytes, cudaStream_t s) {
    if (bytes % 16 != 0) return cudaErrorInvalidValue;
    for (size_t off = 0; off < bytes; off += kUploadChunk) {
        const size_t n = bytes - off < size_t(kUploadChunk) ? bytes - off : size_t(kUploadChunk);
        UploadChunk c;
        std::memcpy(c.v, static_cast<const char*>(src_host) + off, n);
        upload_by_value_kernel<<<1, 128, 0, s>>>(c, reinterpret_cast<uint4*>(static_cast<char*>(dst_dev) + off), int(n / 16));
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t launch_append(const BlockGeom& g, const void* k, const void* v, int /*dim_v_src*/, char* w_base,
                          const AppendRows& rows, int n_rows, cudaStream_t s, int64_t w_bytes, uint32_t* status) {
    if (n_rows <= 0) return cudaSuccess;
    return launch_overlapped(append_kernel, n_rows, 128, size_t(0), s, g, static_cast<const uint4*>(k), static_cast<const uint4*>(v), w_base, rows,
                             w_bytes, status);
}

}  // namespace ipkvi
