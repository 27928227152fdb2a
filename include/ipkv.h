/* ipkv.h — C ABI of the sequence-split decode-attention path over a write-time-partitioned KV cache.
 *
 * The library implements, for one NVIDIA B200 (sm_100a), the hot path of the InplaceKVCache /
 * WriteScope method:
 *
 *   1. write-time routing of every new K/V token into the four-region layout
 *      (device affinity x access pattern; Sec. 4.1, Sec. 4.2 of the paper),
 *   2. attention of one decode query per sequence over the GPU-side share of the sequence,
 *      producing a partial (O, LSE) per query head (Sec. 5.1),
 *   3. the exact log-sum-exp join of that partial with the partial of the CPU-side share
 *      (Sec. 4.2, Sec. 5.1).
 *
 * Conventions
 *   - Every function returns an ipkv_status; nothing throws, aborts, traps the device or keeps
 *     process-global state.  ipkv_last_error() gives the text of the last failure on a handle.
 *   - "dev" pointers are device memory of the handle's device, "host" pointers are host memory.
 *   - All bf16 tensors are raw 16-bit patterns.  Scores are softmax_scale * <q, k>; LSE is the
 *     NATURAL log of the sum of exp(scores); partial outputs O are normalised (divided by their own
 *     softmax denominator).  An empty token set gives O = 0, LSE = -inf.
 *   - Query head h reads KV head floor(h / (n_q_heads / n_kv_heads)).
 *   - Calls are asynchronous on the CUDA stream they are given (a cudaStream_t passed as void*;
 *     NULL is the legacy default stream).  Host-visible results (U / P contents, statistics) are
 *     valid after that stream has been synchronised.  One host thread per handle at a time, and the
 *     calls on one handle must be ordered on the device: use one stream, or order streams with events
 *     (the handle's scratch memory and staging buffers are shared by consecutive calls).
 *   - No CPU fallback exists: without a usable CUDA device every compute entry point fails with
 *     IPKV_ECUDA.
 *
 * Regions (Sec. 4.1).  U: host, unpinned, read by a CPU attention engine.  P: host, pinned, source of
 * host-to-device loads.  W: device, the D-window that stages the newest decode tokens.  PP: device,
 * overwrite-reused slots that P chunks are streamed through ("ping-pong").  On a GPU whose memory can
 * hold part of the GPU-side share, `resident_tokens_per_seq` keeps the newest P blocks of each
 * sequence in a device-side ring (a cache of P; P stays the authoritative copy) so that they need no
 * per-step load; with 0 the layout is exactly the paper's (W + PP only).
 *
 * Block layouts.  A block holds `block_tokens` consecutive tokens of one (layer, sequence).
 *   PLAIN (region U): for each KV head g: K[block_tokens][dim_qk] then V[block_tokens][dim_v],
 *     row-major bf16.
 *   TILE (regions P, W, PP and the resident ring): for each KV head g: the K plane then the V plane.
 *     A plane of width d is d/64 panels; a panel is block_tokens rows of 128 bytes (64 bf16 columns);
 *     inside a row the 16-byte chunk c (0..7) of token offset t sits at chunk position c ^ (t & 7).
 *     Byte offset of column x of token offset t in a plane:
 *       (x/64)*block_tokens*128 + t*128 + ((((x%64)/8) ^ (t&7))*16) + (x%8)*2.
 *     This is the bank-conflict-free shared-memory operand layout of the attention kernel, so a
 *     block travels host -> device -> shared memory as plain contiguous copies.
 *   The compressed-latent kind (IPKV_MLA) stores only the K plane (dim_qk = latent + rope columns);
 *   its V is the first dim_v columns of the same row (Sec. 6.1) and no V plane exists.
 */
#ifndef IPKV_H
#define IPKV_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ipkv ipkv_t; /* opaque; owned by the library */

typedef enum {
  IPKV_OK = 0,
  IPKV_EINVAL = 1,    /* bad argument                                            */
  IPKV_ENOMEM = 2,    /* an allocation failed or a caller buffer is too small    */
  IPKV_ERANGE = 3,    /* a region or the sequence capacity would be exceeded     */
  IPKV_ESTATE = 4,    /* call not legal in the current state                     */
  IPKV_ECUDA = 5,     /* a CUDA call failed (or no device)                       */
  IPKV_ETIMEOUT = 6,  /* a bounded wait inside a kernel gave up                  */
  IPKV_EINTERNAL = 7
} ipkv_status;

typedef enum { IPKV_GQA = 0, IPKV_MLA = 1 } ipkv_kind;
typedef enum { IPKV_REGION_U = 0, IPKV_REGION_P = 1, IPKV_REGION_W = 2 } ipkv_region;
typedef enum { IPKV_LAYOUT_PLAIN = 0, IPKV_LAYOUT_TILE = 1 } ipkv_layout;

/* flags */
#define IPKV_FLAG_NO_HOST_U 1u /* U contents are not kept (routing indices still are): for callers whose
                                  CPU engine keeps its own copy, and for benchmarks                       */
#define IPKV_FLAG_NO_HOST_P 2u /* no host copy of P: every P block must stay device-resident, otherwise
                                  an append fails with IPKV_ERANGE                                        */
#define IPKV_FLAG_GROW_P 4u    /* P grows batch by batch instead of being pinned in full by create (Sec. 4.3,
                                  Sec. 7.7): create pins p_initial_tokens_per_seq per (layer, sequence) — the
                                  prefill share — and a helper thread pins room for every later eviction batch
                                  (window_tokens per (layer, sequence), all layers and sequences in one
                                  allocation, faulted in and then page-locked a layer's range at a time so that
                                  no single driver call is long) one eviction window before the batch lands.
                                  max_p_tokens_per_seq
                                  stays the hard capacity.  Needs chunk_tokens % window_tokens == 0 and
                                  p_initial_tokens_per_seq % chunk_tokens == 0; p_host_pinned must be NULL.      */

/* The paper's PartitionSpec (Sec. 4.3): the four regions, block granularity, eviction batch size, and
 * the share that the roofline policy of Sec. 5.3 would supply, here as an exact rational. */
typedef struct {
  uint32_t struct_size;           /* = sizeof(ipkv_config)                                             */
  int32_t kind;                   /* ipkv_kind                                                         */
  int32_t n_layers, max_seqs;
  int32_t n_q_heads, n_kv_heads;  /* IPKV_MLA: n_kv_heads = 1                                          */
  int32_t dim_qk, dim_v;          /* multiples of 64. GQA kernels: 64 or 128, equal; MLA: 576 / 512    */
  int32_t block_tokens;           /* 16, 32 or a multiple of 64 (paper: "fixed-size blocks", Sec. 4.1) */
  int32_t window_tokens;          /* D, multiple of block_tokens (Sec. 4.2; 256 in the paper)          */
  int32_t chunk_tokens;           /* tokens per sequence in one PP slot, multiple of block_tokens       */
  int32_t n_slots;                /* >= 2; 2 is the paper's ping-pong                                  */
  int64_t max_u_tokens_per_seq;   /* capacity of U per (layer, sequence)                               */
  int64_t max_p_tokens_per_seq;   /* capacity of P per (layer, sequence)                               */
  int64_t resident_tokens_per_seq;/* device ring for the newest P blocks; 0 = stream everything        */
  int64_t p_initial_tokens_per_seq;/* IPKV_FLAG_GROW_P: part of P pinned by create; ignored otherwise   */
  float softmax_scale;            /* 0 => 1/sqrt(dim_qk)                                               */
  int32_t share_num, share_den;   /* marginal CPU share p = num/den of decode eviction batches         */
  int32_t device;                 /* CUDA device ordinal                                               */
  uint32_t flags;
  /* Optional caller-provided memory (e.g. torch tensors); NULL => the library allocates.
     Sizes come from ipkv_query_sizes; a smaller buffer fails with IPKV_ENOMEM. The caller keeps
     ownership and must keep the memory alive until ipkv_destroy. Device buffers are zeroed by create. */
  void* u_host;        size_t u_bytes;
  void* p_host_pinned; size_t p_bytes;
  void* w_dev;         size_t w_bytes;
  void* resident_dev;  size_t resident_bytes;
  void* pp_dev;        size_t pp_bytes;
  /* Optional ring capacity per sequence: host array [max_seqs] of token counts, read by ipkv_query_sizes and
     ipkv_create only (it need not outlive them); NULL => resident_tokens_per_seq for every sequence.  Every layer's
     ring is one run of block slots divided among the sequences in this proportion, so a ragged batch reserves what
     each sequence needs instead of the longest sequence's ring for all (Sec. 4.1: blocks are the unit of placement). */
  const int64_t* resident_tokens_by_seq;
} ipkv_config;

/* out_bytes[0..4] = U, P, W, resident ring, PP slots.  (Table 2 of the paper is these sizes.)
 * With IPKV_FLAG_GROW_P out_bytes[1] is what create pins; P then grows up to its capacity. */
ipkv_status ipkv_query_sizes(const ipkv_config* cfg, size_t out_bytes[5]);

/* The paper's `init` (Sec. 4.3): sizes the regions and pre-allocates them. */
ipkv_status ipkv_create(const ipkv_config* cfg, ipkv_t** out);
ipkv_status ipkv_destroy(ipkv_t* h);

/* Marginal CPU share for later eviction batches (Sec. 5.3); same denominator as at creation. */
ipkv_status ipkv_set_share(ipkv_t* h, int32_t num);

/* Forget one sequence (seq >= 0) or all (seq = -1): its blocks are reused in place (Sec. 4.2). */
ipkv_status ipkv_reset(ipkv_t* h, int32_t seq);

/* Prefill routing in one shot (Sec. 4.2): legal only on an empty (layer, sequence).
 * k_dev [n_tokens][n_kv_heads][dim_qk], v_dev [n_tokens][n_kv_heads][dim_v] bf16 on the device
 * (v_dev = NULL for IPKV_MLA).  The oldest n_cpu = block_tokens * floor(floor(n_tokens/block_tokens)
 * * num0/den0) tokens go to U, the rest to P (and into the resident ring as far as it reaches).
 * The inputs may be reused once work queued on `stream` so far has completed. */
ipkv_status ipkv_append_bulk(ipkv_t* h, int32_t layer, int32_t seq, const void* k_dev, const void* v_dev,
                             int64_t n_tokens, int32_t num0, int32_t den0, void* stream);

/* The paper's `append` for decode (Sec. 4.2): one new token for each listed sequence goes into its
 * D-window; a window that is already full is flushed first, so the newest token is always GPU-side.
 * seq_ids: host, n_seq distinct ids.  k_dev [n_seq][n_kv_heads][dim_qk], v_dev [n_seq][n_kv_heads][dim_v]. */
ipkv_status ipkv_append(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq,
                        const void* k_dev, const void* v_dev, void* stream);

/* The paper's `flush` (Sec. 4.2, 4.3): evict the window of (layer, seq) as one whole batch to U or P;
 * the side follows the integer error-diffusion rule  acc += num; if (acc >= den) { acc -= den; U } else P
 * with acc starting at den/2, which holds the running fraction of CPU-placed batches at num/den
 * (Sec. 5.3).  layer = -1 / seq = -1 mean all.  A placed batch never moves again.  No-op on an empty window. */
ipkv_status ipkv_flush(ipkv_t* h, int32_t layer, int32_t seq, void* stream);

/* By default the grouped-query kernel balances its load while it runs: a CTA that finishes its share of the
 * tiles early (some SMs get more memory bandwidth than others) takes over tiles of the CTAs that are behind.
 * Which tiles end up in which partial then differs from launch to launch, so the fp32 results can differ in the
 * last bits between two identical calls.  This flag keeps the fixed assignment: bit-reproducible, a few
 * percent slower.  (The stateless entry points below always use the fixed assignment.) */
#define IPKV_ATTEND_STATIC_SCHEDULE 1
/* The balancing is switched on by the library when the launch is long enough for it to pay (from 64 tiles of 64
 * tokens per CTA, more when the batch is large); this flag switches it on for any size (tests use it to exercise the path on small inputs). */
#define IPKV_ATTEND_BALANCE 2
/* Stream ordering.  The attention, split-reduce and append kernels are launched so that each may become resident while the previous
 * kernel of its stream drains (programmatic dependent launch); it waits for that kernel to complete before it reads
 * or writes anything a previous kernel could have touched, so the results are those of plain stream order, behind
 * the library's own kernels and behind the caller's.  An attention launch whose K/V bytes the library knows to be
 * settled (nothing it enqueued since the launch before the previous one wrote them) also starts its first copies
 * before that wait.  The environment variables IPKV_NO_LAUNCH_OVERLAP and IPKV_NO_EARLY_COPIES (any value, read once
 * per process) restore plain launches / switch the early copies off.  IPKV_PARTS_PER_SPAN=1 or 4 (a test hook, read
 * once) fixes how many partials the grouped-query kernel writes per span (1: its warps join their states first), which
 * the library otherwise chooses per launch by the length of the spans; the results agree within rounding. */

typedef struct {
  int32_t kv_splits;   /* 0 = automatic; otherwise the number of sequence chunks per (sequence, KV head) */
  int32_t flags;       /* IPKV_ATTEND_* bits                                                          */
  void* side_stream;   /* stream for host-to-device chunk copies; NULL = the handle's own             */
  /* Optional extra partial over a disjoint token set (typically the CPU-side partial, already on the
     device): [n_seq][n_q_heads][dim_v] and [n_seq][n_q_heads] fp32.  When both are given it is folded in by
     the same exact LSE join inside the split reduce, so the outputs are the MERGED (O, LSE) and no separate
     ipkv_merge launch is needed for this step (Sec. 4.2: one join per step, performed on the GPU).        */
  const float* fold_o_dev;
  const float* fold_lse_dev;
  /* Optional fused decode append (ipkv_attend_gpu only): one new token for each listed sequence,
     k [n_seq][n_kv_heads][dim_qk], v [n_seq][n_kv_heads][dim_v] (NULL for IPKV_MLA), appended exactly as ipkv_append
     would (full windows are evicted first) and attended by the same call.  Where the kernel can, it writes the new
     rows into the D-window itself (grouped-query caches with block_tokens >= 64: the warp that owns the token's slice
     of the tile patches the tile in shared memory and stores the rows to the window), which saves the append launch of
     every layer; otherwise the library launches its append kernel first.  The result is the same either way.   */
  const void* append_k_dev;
  const void* append_v_dev;
} ipkv_attend_opts;

/* Attention over the GPU-side share (Sec. 5.1): the D-window plus every P token, device-resident ones
 * read in place and the others streamed through the PP slots on the side stream while the resident part
 * is being computed.  Which tokens are attended is fixed by the format at write time, never an argument.
 * q_dev [n_seq][n_q_heads][dim_qk] bf16.  Outputs (fp32, device): o_part [n_seq][n_q_heads][dim_v],
 * lse_part [n_seq][n_q_heads].  opts may be NULL. */
ipkv_status ipkv_attend_gpu(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq,
                            const void* q_dev, const ipkv_attend_opts* opts,
                            float* o_part_dev, float* lse_part_dev, void* stream);

/* Block-sparse variant (Sec. 4.4): every row attends its D-window (if include_window != 0) plus the listed WHOLE P
 * blocks only — the set a block-level top-k selection would return.  p_blocks: host array of block ordinals inside
 * region P (as ipkv_views / ipkv_locate report them), the blocks of row r at p_blocks[row_block_start[r] ..
 * row_block_start[r+1]), strictly increasing within a row.  Device-resident blocks are read in place; host-only blocks
 * are gathered, one memcpy per block, into a contiguous pinned staging buffer the size of a PP slot and reach the
 * device with one DMA per slot, the gather of the next slot overlapping the DMA of the current one.
 * Other arguments and outputs as ipkv_attend_gpu. */
ipkv_status ipkv_attend_gpu_sparse(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* q_dev,
                                   const int64_t* p_blocks, const int32_t* row_block_start, int32_t include_window,
                                   const ipkv_attend_opts* opts, float* o_part_dev, float* lse_part_dev, void* stream);

/* CPU-side engine (Sec. 6.1): in-place attention over the CPU-side share, i.e. the tokens routed to region U,
 * read where they lie (PLAIN blocks, no copy).  This is the paper's second engine, not a fallback for the GPU
 * path: it attends a disjoint token range and its partial is joined by ipkv_merge / the fold option.
 * q_host [n_seq][n_q_heads][dim_qk] bf16 in host memory; o_part_host [n_seq][n_q_heads][dim_v] and
 * lse_part_host [n_seq][n_q_heads] fp32 in host memory (in pinned memory ipkv_merge reads them where they are).
 * The call runs synchronously on the calling thread plus OpenMP workers (n_threads <= 0: all cores).  The tile
 * kernel is chosen at first use: the AMX tile unit where the CPU has one and the operating system grants its state,
 * else AVX-512, AVX2 or baseline vector code; the environment variable IPKV_CPU_KERNEL=v4|v3|base forces a lower
 * level (tests).  The levels agree within fp32 rounding.
 * U is filled by device-to-host copies queued by the append / flush calls: synchronise their stream first.
 * This call may run on a second host thread while ipkv_attend_gpu / ipkv_merge of the same handle run on the first
 * (the paper's step: both engines at once, one join): it only reads the routing state.  No call that changes routing
 * (append, flush, set_share, reset) may run at the same time.
 * Fails with IPKV_ESTATE if U contents are not kept (IPKV_FLAG_NO_HOST_U). */
ipkv_status ipkv_attend_cpu(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* q_host,
                            float* o_part_host, float* lse_part_host, int32_t n_threads);

/* Exact n-way log-sum-exp join (Sec. 4.2, 5.1) of row-aligned partials over disjoint token sets:
 *   LSE = m + ln sum_i exp(LSE_i - m), m = max_i LSE_i;  O = sum_i exp(LSE_i - LSE) * O_i.
 * o_parts[i] [n_rows][dim_v] fp32, lse_parts[i] [n_rows] fp32; the pointer arrays are host memory;
 * each part may be device memory or host memory.  A part in pinned (page-locked or registered) host memory is
 * read by the kernel where it is, in stream order: it must stay unchanged until the call's work on `stream`
 * has completed.  A part in pageable host memory is copied on `stream` first.  1 <= n_parts <= 8.
 * o_out_dev is fp32, or bf16 (round to nearest even) when o_out_is_bf16 != 0.  lse_out_dev may be NULL.
 * h may be NULL only if no part is pageable host memory. */
ipkv_status ipkv_merge(ipkv_t* h, int32_t n_rows, int32_t dim_v, int32_t n_parts,
                       const float* const* o_parts, const float* const* lse_parts,
                       void* o_out_dev, int32_t o_out_is_bf16, float* lse_out_dev, void* stream);

/* The paper's `views` (Sec. 4.3): zero-copy description of where a (layer, sequence) lives.
 * One extent per placed run (prefill share, each eviction batch) plus one for the window, in token order. */
typedef struct {
  int32_t region;        /* ipkv_region                                                        */
  int32_t layout;        /* ipkv_layout of the blocks                                          */
  int64_t first_token;   /* first token index of the run in the sequence                       */
  int64_t n_tokens;
  int64_t region_block;  /* ordinal of the run's first block inside its region (W: 0)          */
  const void* host_ptr;  /* first block in U or P host memory, NULL if none                    */
  const void* dev_ptr;   /* first block on the device (W, or a fully resident P run), else NULL */
  int64_t block_bytes;   /* consecutive blocks of a run are contiguous at this pitch           */
} ipkv_extent;

ipkv_status ipkv_views(ipkv_t* h, int32_t layer, int32_t seq, ipkv_extent* out, int32_t cap, int32_t* n_out);

/* Where one token lives: region, block ordinal in the region, offset in the block (W: slot index). */
ipkv_status ipkv_locate(ipkv_t* h, int32_t layer, int32_t seq, int64_t token,
                        int32_t* region, int64_t* region_block, int32_t* offset_in_block);

/* Token counts of (layer, seq): counts[0..2] = tokens in U, P, W; counts[3] = P tokens that are
 * device-resident; counts[4..5] = eviction batches so far, of which CPU-placed. */
ipkv_status ipkv_counts(ipkv_t* h, int32_t layer, int32_t seq, int64_t counts[6]);

/* Copy the K (and V) row of one token, de-swizzled to plain [n_kv_heads][dim] order, into host buffers
 * (synchronises the device; for tests and debugging).  v_out may be NULL. */
ipkv_status ipkv_read_token(ipkv_t* h, int32_t layer, int32_t seq, int64_t token, void* k_out, void* v_out);

typedef struct {
  uint64_t attend_calls, attend_kernels, reduce_kernels, merge_kernels, append_kernels, pack_kernels;
  uint64_t kv_bytes_attended;   /* tokens * bytes per token, summed over attend calls            */
  uint64_t h2d_bytes, d2h_bytes, d2d_bytes;
  uint64_t flushes, flushes_to_u;
  uint64_t fused_appends;       /* ipkv_attend_gpu calls whose kernel wrote the appended rows itself     */
  uint64_t early_launches;      /* attention launches allowed to fill their copy ring before the previous kernel
                                   of the stream had completed (no K/V byte they read could still be in flight) */
  /* IPKV_FLAG_GROW_P: segments pinned so far, their bytes, the page-locking time spent (by create for the
     first, by the helper thread for the rest), and how often / how long a call had to wait for a segment
     that was not pinned yet (0 when the one-window lookahead covers the pinning, as Sec. 7.7 expects).  */
  uint64_t p_segments, p_pinned_bytes, p_pin_us, p_grow_waits, p_grow_wait_us;
  uint64_t p_register_us, p_register_calls, p_register_max_us;  /* the page-locking calls alone: total, count, longest */
  uint32_t device_status;       /* nonzero after a kernel's bounded wait gave up (synchronises): bit 0 a producer
                                   got no free stage, bit 1 a consumer got no tile, bit 2 a copy did not land;
                                   bit 3 (bounds-checked build) a computed address left its region             */
} ipkv_stats;
/* Synchronises the device and fills *out.  If a bounded wait inside one of the handle's kernels gave up since the last
 * call, *out is still filled (device_status says which wait), the call returns IPKV_ETIMEOUT (the results of the
 * attention calls since the last ipkv_get_stats are then invalid) and the device word is cleared, so the calls that
 * follow are judged on their own. */
ipkv_status ipkv_get_stats(ipkv_t* h, ipkv_stats* out);

/* Self-test of the failure path (no counterpart in the paper): enqueues a one-CTA kernel in which a consumer thread
 * waits limit_us microseconds (1 .. 1 000 000) for a tile that is announced on its stage barrier and never copied.
 * The wait runs out, the kernel records "a consumer got no tile" in the handle's status word and returns; nothing
 * faults and nothing spins without a limit.  The next ipkv_get_stats then returns IPKV_ETIMEOUT, the one after it
 * IPKV_OK.  The attention kernels' own waits use the same routine with a limit of two seconds. */
ipkv_status ipkv_selftest_expire_wait(ipkv_t* h, uint32_t limit_us, void* stream);

/* Self-test of the host-side failure path (no counterpart in the paper): the next attention launch of this handle is
 * refused on the host before anything reaches the GPU and its call returns IPKV_ECUDA.  If that call carried a fused
 * append, the routing state already counts the new tokens; the library then writes their rows with its append kernel,
 * so the windows hold what the routing says and the next calls see every token. */
ipkv_status ipkv_selftest_fail_next_launch(ipkv_t* h);

/* Bounds-checked build (libipkv_checked.so, compiled with -DIPKV_CHECKED; ipkv_version() says so): every source address
 * the attention kernels compute for a copy, every partial row they store and every window slot the append paths write is
 * compared with the extent of its region, and the ring destinations the host computes for the packing and ring-refresh
 * kernels with the sequence's part of the ring.  A violation is recorded (device_status bit 3), the access is not made (a read
 * is redirected to the region's first bytes, a write is dropped), and the next ipkv_get_stats returns IPKV_EINTERNAL.
 * This self-test call (no counterpart in the paper) declares region base_id of the handle (0 resident ring of a layer,
 * 1 D-windows of a layer, 2 PP slots) to be only `bytes` long (0 restores the real extent): launches that reach
 * beyond then trip the check while touching nothing but valid memory.  IPKV_ESTATE in the ordinary build. */
ipkv_status ipkv_selftest_declare_bounds(ipkv_t* h, int32_t base_id, int64_t bytes);

/* ---- roofline share policy (host only; Sec. 5.2-5.3) ------------------------------------------------
 * Eq. 1: T_CPU(r) = r*A*L + C_cpu, T_GPU(r) = (1-r)*B*L + C_gpu, T = max(T_CPU, T_GPU) + T_merge.
 * Eq. 2: r(L) = clamp01(B/(A+B) + (C_gpu - C_cpu)/((A+B)*L)); marginal share p = B/(A+B).
 * A, B in seconds per KV token, overheads in seconds.  The policy keeps a sliding window of the CPU engine's
 * per-step latencies (the paper uses 256 steps), back-computes A from them and returns the numerator of p over
 * `share_den` for ipkv_set_share; B is calibrated once.  None of these calls touches a GPU. */
typedef struct ipkv_policy ipkv_policy_t;
typedef struct { double A, B, C_cpu, C_gpu; } ipkv_roofline;
double ipkv_roofline_share(const ipkv_roofline* m, double L);                                   /* Eq. 2 */
double ipkv_roofline_step_time(const ipkv_roofline* m, double r, double L, double t_merge,
                               double* t_cpu_out, double* t_gpu_out);                           /* Eq. 1 */
ipkv_status ipkv_policy_create(const ipkv_roofline* m, int32_t window_steps, int32_t share_den, ipkv_policy_t** out);
ipkv_status ipkv_policy_destroy(ipkv_policy_t* p);
/* one decode step of the CPU engine: its latency and the CPU-side KV tokens it attended */
ipkv_status ipkv_policy_observe(ipkv_policy_t* p, double cpu_seconds, double cpu_tokens);
/* re-estimate A, return the numerator of p = B/(A+B) over share_den and the current model */
ipkv_status ipkv_policy_update(ipkv_policy_t* p, int32_t* share_num_out, ipkv_roofline* model_out);
/* prefill share R(L0) = r(L0) as a numerator over share_den */
ipkv_status ipkv_policy_prefill_share(const ipkv_policy_t* p, double L0, int32_t* share_num_out);

/* Kernel timing for benchmarks.  While enabled, every attention-kernel launch of ipkv_attend_gpu is
 * bracketed by a pair of CUDA events on the launching stream.  ipkv_profile_read synchronises the device,
 * returns the summed kernel time (milliseconds) and the number of launches since the last read, and resets
 * both.  At most 8192 launches are kept between two reads; later ones are counted but not timed. */
/* on: 0 off, 1 attention kernels, 2 split-reduce kernels instead; plus 256 * n to bracket only every n-th launch (an
 * event between two kernels keeps the second from starting while the first drains, which costs the step several
 * microseconds per bracketed launch). */
ipkv_status ipkv_profile_enable(ipkv_t* h, int32_t on);
ipkv_status ipkv_profile_read(ipkv_t* h, double* attend_kernel_ms, int64_t* n_timed, int64_t* n_launches);

/* Measurement aid (no counterpart in the paper): the rate, in GB/s, at which the SMs of `device` read `bytes` bytes
 * (>= 64 MB; use more than the L2 holds) of freshly allocated device memory through the same bulk-copy / mbarrier ring
 * the attention kernels use, with no arithmetic.  Decode attention only reads the KV bytes, a copy reads and writes
 * them: this is the read-only ceiling shown beside the copy bandwidth.  Allocates 2 x bytes for the duration of the
 * call, runs 3 warm-up and `reps` timed launches (CUDA events), returns the best and the mean. */
ipkv_status ipkv_probe_read_bandwidth(int32_t device, size_t bytes, int32_t reps, double* best_gbs, double* mean_gbs);

/* Measurement aid (no counterpart in the paper): the cost of small fifth-generation tensor-core instructions on `device`.
 * One CTA, one issuing thread: n_mma back-to-back tcgen05.mma of shape M x N x 16 (bf16 in, fp32 accumulate in tensor
 * memory, operands in shared memory) and one commit.  issue_cycles: SM clocks until the last instruction and the commit
 * were issued; total_cycles: until the commit's barrier completed; best of `reps` launches.  Shapes M 64 / 128 x N 16 /
 * 64 / 256 with n_mma 1, 8, 36 into one accumulator, and 36 rotating over four accumulators where they fit: the fixed
 * cost per instruction and the throughput separate.  Fills out[0 .. *n_out). */
typedef struct { int32_t m, n, n_mma, accumulators; int64_t issue_cycles, total_cycles; } ipkv_umma_timing;
ipkv_status ipkv_probe_umma(int32_t device, int32_t reps, ipkv_umma_timing* out, int32_t cap, int32_t* n_out);

/* ---- stateless kernel entry points (no handle) ------------------------------------------------- */

typedef struct {
  int32_t kind;                   /* ipkv_kind */
  int32_t n_q_heads, n_kv_heads, dim_qk, dim_v, block_tokens;
  float softmax_scale;            /* 0 => 1/sqrt(dim_qk) */
} ipkv_attn_shape;

typedef struct {
  const void* blocks_dev;  /* first block of a run of contiguous TILE-layout blocks on the device; every
                              block of the run must be fully allocated and hold finite values           */
  int64_t n_tokens;        /* valid tokens in the run (the last block may be partly filled)           */
} ipkv_run;

/* Scratch needed by ipkv_attend_runs for n_rows rows, n_runs runs in total holding total_tokens tokens. */
ipkv_status ipkv_attend_scratch_bytes(const ipkv_attn_shape* shape, int32_t n_rows, int32_t n_runs,
                                      int64_t total_tokens, int32_t kv_splits, size_t* out_bytes);

/* Split-K decode attention (Sec. 5.1, GPU side) of n_rows queries, row r over the union of the runs
 * runs[row_run_start[r] .. row_run_start[r+1]).  runs and row_run_start are host arrays.
 * scratch_dev: device memory of at least ipkv_attend_scratch_bytes (256-byte aligned), private to this
 * call until the work queued on `stream` has completed.  Outputs as in ipkv_attend_gpu.
 * status_dev: optional device uint32 that is OR-ed with the bits below if a bounded wait inside a kernel gave up
 * (bit 0: the copy engine's thread found no free stage; bit 1: a consumer's tile did not arrive; bit 2: a copy had
 * not landed when its CTA left); the results of that call are then invalid.  With NULL a timeout goes unreported. */
ipkv_status ipkv_attend_runs(const ipkv_attn_shape* shape, int32_t n_rows,
                             const ipkv_run* runs, const int32_t* row_run_start,
                             const void* q_dev, int32_t kv_splits,
                             void* scratch_dev, size_t scratch_bytes,
                             float* o_part_dev, float* lse_part_dev, uint32_t* status_dev, void* stream);

/* Same computation and arguments as ipkv_attend_runs, but without a scratch argument: the scratch lives in a
 * fixed 16 MiB array inside the library's device image.  (The paper has no counterpart; this exists for hosts
 * that must not allocate device memory where they call attention: servers that give all memory to their own
 * pool at start-up, latency-critical loops that cannot afford cudaMalloc's device-wide synchronisation,
 * plug-ins whose contract forbids allocation.)  The call allocates nothing on the device: no cudaMalloc,
 * no cudaFree, no allocating library routine.
 *   - Limit: the call needs ipkv_attend_scratch_bytes(shape, n_rows, n_runs, total tokens, kv_splits) bytes;
 *     if that exceeds ipkv_noalloc_scratch_limit() (16 MiB) it returns IPKV_ERANGE and does nothing.
 *     A larger kv_splits or batch needs more; use ipkv_attend_runs with your own scratch then.
 *   - The array is one per GPU.  The first call on a device resolves its device address (cudaGetSymbolAddress, with
 *     that device current); with CUDA's lazy module loading that is also the moment the driver sets the 16 MiB aside
 *     on that GPU, which keeps them until the process exits.  So make one warm-up call per device at start-up, before
 *     the memory is handed to a pool (afterwards the first call could fail with IPKV_ECUDA) and outside any stream
 *     capture.  The address is remembered per device ordinal: after a cudaDeviceReset the library must be reloaded.
 *   - The launch tables (a few KB) go up with a cudaMemcpyAsync from a temporary pageable host image: the runtime
 *     stages it before the call returns, so the call is asynchronous to the GPU but not free of host-side work.
 *   - All calls on a device share the array and each finds the previous call's bytes in it; nothing needs
 *     clearing between calls, but two calls whose work overlaps on the GPU (different streams without an
 *     ordering event, or another host thread) race on it.  Order them.
 * status_dev as in ipkv_attend_runs. */
ipkv_status ipkv_attend_runs_noalloc(const ipkv_attn_shape* shape, int32_t n_rows,
                                     const ipkv_run* runs, const int32_t* row_run_start,
                                     const void* q_dev, int32_t kv_splits,
                                     float* o_part_dev, float* lse_part_dev, uint32_t* status_dev, void* stream);
size_t ipkv_noalloc_scratch_limit(void);

/* Re-lay token-major K/V ([n_tokens][n_kv_heads][dim]) into consecutive blocks of the given layout
 * starting at token offset 0 of dst_dev (device to device; used by tests and by callers that build
 * blocks themselves).  v_dev = NULL for IPKV_MLA. */
ipkv_status ipkv_pack_blocks(const ipkv_attn_shape* shape, int32_t layout, const void* k_dev, const void* v_dev,
                             int64_t n_tokens, void* dst_dev, void* stream);

/* Bytes of one block for a shape. */
int64_t ipkv_block_bytes(const ipkv_attn_shape* shape);

const char* ipkv_status_str(ipkv_status s);
const char* ipkv_last_error(const ipkv_t* h);
const char* ipkv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* IPKV_H */
