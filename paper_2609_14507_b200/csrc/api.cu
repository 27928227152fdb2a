// C ABI of the library (include/ipkv.h): the handle, the host-side scheduler that turns the routing
// state into kernel launches and copies, and the stateless entry points.
//
// Decode step of one layer (Sec. 4.2, Sec. 5.1):
//   ipkv_append      router -> append kernel (new token into the D-window); a full window is evicted first
//                    (whole batch, device -> host on the idle D2H direction, TILE -> PLAIN for U)
//   ipkv_attend_gpu  split-K attention over the resident ring and the D-window; P chunks that are not
//                    device-resident are copied H2D into PP slots on a side stream, each slot attended as
//                    soon as its copy has landed and folded into the running partial
//   ipkv_merge       LSE join with the CPU-side partial
#include <cuda_runtime.h>
#include <sys/mman.h>

#include <algorithm>
#include <chrono>
#include <cmath>
#include <condition_variable>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <thread>
#include <vector>

#include "../../include/ipkv.h"
#include "cpu_engine.h"
#include "kernels.h"
#include "plan.hpp"
#include "ring.hpp"
#include "policy.hpp"
#include "router.hpp"

namespace ipkvi {
cudaError_t launch_attend_gqa(const AttnLaunch& a, cudaStream_t s);
cudaError_t launch_attend_mla(const AttnLaunch& a, cudaStream_t s);

cudaError_t launch_attend(const AttnLaunch& a, cudaStream_t s) {
    return a.kind == IPKV_MLA ? launch_attend_mla(a, s) : launch_attend_gqa(a, s);
}
}  // namespace ipkvi

using namespace ipkvi;

namespace {


struct PRun {            // maximal run of P blocks that the attention kernel can walk as one segment
    int64_t first_block;
    int64_t n_tokens;
};

struct SeqState {
    SeqRouter router;
    std::vector<PRun> p_runs;
};


// Bytes of the partial buffers for n_spans spans.
size_t partial_bytes(size_t n_spans, const PartGeom& pg, int dv) {
    const size_t rows = n_spans * size_t(pg.parts_per_span) * pg.rows_per_group;
    return align_up(rows * dv * sizeof(float), 256) + align_up(rows * sizeof(float), 256);
}

bool shape_ok(int kind, int Hq, int Hkv, int dqk, int dv, int bt, std::string* why) {
    auto fail = [&](const char* m) { if (why) *why = m; return false; };
    if (Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) return fail("n_q_heads must be a positive multiple of n_kv_heads");
    if (!(bt == 16 || bt == 32 || (bt > 0 && bt % 64 == 0))) return fail("block_tokens must be 16, 32 or a multiple of 64");
    if (kind == IPKV_GQA) {
        if (!((dqk == 128 && dv == 128) || (dqk == 64 && dv == 64))) return fail("GQA kernels support dim_qk = dim_v in {64, 128}");
    } else if (kind == IPKV_MLA) {
        if (Hkv != 1) return fail("the compressed-latent kind has one shared KV head");
        if (dqk != 576 || dv != 512) return fail("the compressed-latent kernel supports dim_qk 576 / dim_v 512");
        if (Hq > 128) return fail("the compressed-latent kernel supports at most 128 query heads");
    } else {
        return fail("unknown kind");
    }
    return true;
}

BlockGeom make_geom(int kind, int Hkv, int dqk, int dv, int bt) {
    BlockGeom g;
    g.n_kv_heads = Hkv; g.dim_qk = dqk; g.dim_v_stored = (kind == IPKV_MLA) ? 0 : dv; g.bt = bt;
    return g;
}

}  // namespace

// ---- the handle ---------------------------------------------------------------------------------
struct ipkv {
    ipkv_config cfg;
    BlockGeom geom;
    float scale = 0.f;
    int64_t bb = 0;                 // block bytes
    int64_t u_cap = 0, p_cap = 0;   // blocks per (layer, seq)
    RingMap rmap;                   // resident ring: block slots of every sequence inside a layer's ring
    int64_t w_blocks = 0, chunk_blocks = 0;
    size_t sizes[5] = {0, 0, 0, 0, 0};
    char *u_host = nullptr, *p_host = nullptr, *w_dev = nullptr, *res_dev = nullptr, *pp_dev = nullptr;
    bool own[5] = {false, false, false, false, false};
    // Pin-ahead growth of P (Sec. 4.3, Sec. 7.7): P is a list of pinned segments, each holding the same range
    // of block ordinals of every (layer, sequence) as [layer][seq][nb].  Segment 0 (the prefill share) is pinned
    // by create; every later segment holds one eviction batch and is pinned by a helper thread one window
    // before its first batch lands, so the page-locking never sits on the decode path.
    struct PSegment { char* base = nullptr; int64_t b0 = 0, nb = 0; };
    bool grow_p = false;
    std::vector<PSegment> pseg;          // every segment P can ever have; `base` is set once, by the pinning thread
    std::mutex pmu;
    std::condition_variable pcv;
    int p_requested = 0, p_ready = 0;    // segments [0, p_ready) are usable, [p_ready, p_requested) are being pinned
    bool p_failed = false, p_quit = false;
    int p_waiters = 0;                   // calls blocked in p_ensure: the pinning thread then stops pacing itself
    uint64_t p_tick = 0;                 // decode steps seen (appends to layer 0): the pinning thread's pace
    std::thread p_thread;
    uint64_t p_pinned_bytes = 0, p_pin_us = 0, p_register_us = 0, p_register_calls = 0, p_register_max_us = 0;   // under pmu
    std::vector<SeqState> st;
    // staging for layout conversion on the way to host memory
    char* staging = nullptr;
    size_t staging_bytes = 0;
    // split-K scratch: descriptor tables + partials
    char* scratch = nullptr;
    size_t scratch_bytes = 0;
    char* table_pinned = nullptr;   // ring of pinned table images, mirrored at the same offsets on the device
    char* table_dev = nullptr;
    size_t table_cap = 0, table_head = 0;
    static constexpr int kTableParts = 8;
    cudaEvent_t table_ev[kTableParts] = {};
    bool table_ev_set[kTableParts] = {};
    int table_part = 0;
    std::vector<char> last_table;
    size_t last_table_off = 0;
    cudaStream_t last_table_stream = nullptr;
    bool last_table_valid = false;
    // merge staging for host-side partials
    char* merge_stage = nullptr;
    size_t merge_stage_bytes = 0;
    uint32_t* status_dev = nullptr;
    // scheduling words of the dynamically balanced attention kernel: two sets used by alternate launches; the
    // split reduce of one launch zeroes the set of the next
    // the plan of the previous launch and what it was built from: a launch over the same runs (every layer of a decode step,
    // and the next steps while the windows stay inside their tiles) reuses it without planning or serialising anything
    Plan last_plan;
    std::vector<int64_t> plan_sig_scratch;
    std::vector<int64_t> last_plan_sig;
    bool fail_next_launch = false;                   // self-test: the next attention launch is refused on the host
    int32_t* steal_dev = nullptr;
    static constexpr int kStealWords = 1 << 16;     // per set
    int steal_dirty[2] = {0, 0};                     // words a launch has written in each set
    unsigned steal_epoch = 0;
    // write-back of evicted windows on the idle D2H direction: a device snapshot of every window (same shape as W),
    // a copy stream, one "snapshot in use" event per layer, and a pinned bounce buffer for the unpinned region
    char* wb_stage = nullptr;
    char* wb_bounce = nullptr;
    cudaStream_t copy = nullptr;
    cudaEvent_t ev_wb = nullptr, ev_copy = nullptr;
    std::vector<cudaEvent_t> wb_busy;
    std::vector<char> wb_busy_set;
    cudaStream_t side = nullptr;
    // block-sparse path: two pinned gather buffers of one PP slot each, and the event of the DMA that last read each
    char* gather[2] = {nullptr, nullptr};
    cudaEvent_t gather_done[2] = {nullptr, nullptr};
    bool gather_busy[2] = {false, false};
    std::vector<cudaEvent_t> slot_ready, slot_free;
    std::vector<char> slot_free_set;
    cudaEvent_t ev_main = nullptr;
    cudaEvent_t ev_p_host = nullptr;       // after the last copy into P's host memory that a compute stream carried (prefill)
    bool ev_p_host_set = false;
    // Which attention launches may start their first copies before the previous kernel of the stream has completed
    // (AttnLaunch::early_tiles).  launch_seq counts the attention launches enqueued so far; kv_written_at[layer] is the
    // value it must have reached before a launch on that layer may do so: one whole attention + reduce pair has then
    // been enqueued, on the same stream, after the last operation that wrote the layer's device-side K/V.  The D-window
    // is written by every append and the ring only by evictions, so the two are tracked apart: a launch right behind an
    // append kernel may still start early on its ring tiles.
    uint64_t launch_seq = 0;
    std::vector<uint64_t> kv_written_at;     // resident ring of the layer
    std::vector<uint64_t> w_written_at;      // D-window of the layer
    cudaStream_t launch_stream = nullptr;
    bool launch_stream_valid = false;
    ipkv_stats stats;
    std::string err;
    // optional kernel timing
    bool prof_on = false;
    bool prof_reduce = false;              // time the split reduce instead of the attention kernel
    int prof_stride = 1;                   // time every prof_stride-th launch
    int64_t prof_seen = 0;
    std::vector<cudaEvent_t> prof_ev;      // pairs
    size_t prof_used = 0;                  // events used
    int64_t prof_launches = 0;

    SeqState& state(int layer, int seq) { return st[size_t(layer) * cfg.max_seqs + seq]; }
    int64_t seq_index(int layer, int seq) const { return int64_t(layer) * cfg.max_seqs + seq; }
    char* u_ptr(int layer, int seq, int64_t blk) { return u_host + (seq_index(layer, seq) * u_cap + blk) * bb; }
    bool has_p() const { return p_host != nullptr || grow_p; }
    int p_segment_of(int64_t blk) const {
        return blk < pseg[0].nb ? 0 : 1 + int((blk - pseg[0].nb) / w_blocks);
    }
    int64_t w_off(int seq) const { return int64_t(seq) * w_blocks * bb; }                       // inside a layer
    char* w_layer(int layer) { return w_dev + int64_t(layer) * cfg.max_seqs * w_blocks * bb; }
    // extent of the memory behind base `id` of a launch (0 ring of one layer, 1 D-windows of one layer, 2 PP slots), for the
    // bounds-checked build; a self-test may declare one of them smaller than it is (selftest_bounds)
    int64_t selftest_bounds[kMaxBases] = {0, 0, 0, 0};
    int64_t region_bytes(int id) const {
        if (id >= 0 && id < kMaxBases && selftest_bounds[id] > 0) return selftest_bounds[id];
        if (id == 0) return rmap.total() * bb;
        if (id == kSegBaseWindow) return int64_t(cfg.max_seqs) * w_blocks * bb;
        if (id == 2) return int64_t(sizes[4]);
        return 0;
    }
    int64_t ring_of(int seq) const { return rmap.blocks(seq); }                                 // block slots of the sequence
    int64_t ring_off(int seq) const { return rmap.first_slot(seq) * bb; }                       // inside a layer
    char* ring_layer(int layer) { return res_dev + int64_t(layer) * rmap.total() * bb; }
    int64_t slot_bytes() const { return int64_t(cfg.max_seqs) * chunk_blocks * bb; }
};

namespace {

// Makes the handle's device current for the duration of a call and restores the caller's device afterwards.
class DeviceGuard {
public:
    explicit DeviceGuard(int device) {
        if (device < 0) return;                               // no device of its own: stay on the caller's
        if (cudaGetDevice(&prev_) != cudaSuccess) prev_ = -1;
        err_ = (prev_ == device) ? cudaSuccess : cudaSetDevice(device);
        changed_ = (prev_ != device) && err_ == cudaSuccess;
    }
    ~DeviceGuard() { if (changed_ && prev_ >= 0) cudaSetDevice(prev_); }
    cudaError_t error() const { return err_; }
    DeviceGuard(const DeviceGuard&) = delete;
    DeviceGuard& operator=(const DeviceGuard&) = delete;
private:
    int prev_ = -1;
    cudaError_t err_ = cudaSuccess;
    bool changed_ = false;
};

ipkv_status fail(ipkv* h, ipkv_status s, const std::string& msg) {
    if (h) h->err = msg;
    return s;
}
ipkv_status fail_cuda(ipkv* h, cudaError_t e, const char* what) {
    return fail(h, IPKV_ECUDA, std::string(what) + ": " + cudaGetErrorString(e));
}
#define CU(h, call)                                                  \
    do {                                                             \
        cudaError_t e__ = (call);                                    \
        if (e__ != cudaSuccess) return fail_cuda((h), e__, #call);   \
    } while (0)

// ---- pin-ahead growth of P ------------------------------------------------------------------------
size_t p_segment_bytes(const ipkv* h, int k) {
    return size_t(int64_t(h->cfg.n_layers) * h->cfg.max_seqs * h->pseg[size_t(k)].nb * h->bb);
}

// Allocates and page-locks segment k.  One cudaHostAlloc of the whole segment (the paper's call) holds the driver's
// lock for its full duration — measured here: 70-410 ms during which the decode thread's launches stall — so the
// memory is allocated and faulted in with plain host calls first, and then registered with the driver one layer's
// range at a time (a few MB, under a millisecond each; every copy the library issues lies inside one such range),
// paced by the decode steps themselves when the decode thread is running beside it: at most one range per step, the
// whole segment within half an eviction window.
bool pin_segment(ipkv* h, int k, bool beside_decode, char** base_out) {
    const size_t bytes = p_segment_bytes(h, k);
    const size_t layer_bytes = bytes / size_t(h->cfg.n_layers);
    void* p = nullptr;
    if (posix_memalign(&p, size_t(2) << 20, bytes) != 0) return false;
    // 2 MB pages where the kernel grants them: measured on the B200 host, faulting in drops from 0.36 to 0.12 ms/MB
    // and page-locking a 4 MB range from 1.4 ms to 0.3 ms (a refusal changes nothing but the speed)
    madvise(p, bytes, MADV_HUGEPAGE);
    std::memset(p, 0, bytes);                                       // fault every page in before the driver sees it
    const bool by_layer = layer_bytes % 4096 == 0;
    const size_t piece = by_layer ? layer_bytes : bytes;
    const uint64_t n_pieces = bytes / piece;
    const uint64_t steps_per_piece = std::max<uint64_t>(1, uint64_t(h->cfg.window_tokens) / 2 / n_pieces);
    size_t done = 0;
    uint64_t reg_us = 0, reg_max = 0;
    for (; done < bytes; done += piece) {
        const auto r0 = std::chrono::steady_clock::now();
        if (cudaHostRegister(static_cast<char*>(p) + done, piece, cudaHostRegisterDefault) != cudaSuccess) break;
        const uint64_t us = uint64_t(std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now() - r0).count());
        reg_us += us; reg_max = std::max(reg_max, us);
        if (beside_decode && done + piece < bytes) {
            // next range after `steps_per_piece` more decode steps; at once if a call is waiting for this segment,
            // and after 2 ms anyway (nobody is decoding)
            std::unique_lock<std::mutex> lk(h->pmu);
            const uint64_t target = h->p_tick + steps_per_piece;
            h->pcv.wait_for(lk, std::chrono::milliseconds(2), [&] { return h->p_quit || h->p_waiters > 0 || h->p_tick >= target; });
            if (h->p_quit) { done += piece; break; }
        }
    }
    {
        std::lock_guard<std::mutex> lk(h->pmu);
        h->p_register_us += reg_us; h->p_register_calls += done / piece; h->p_register_max_us = std::max(h->p_register_max_us, reg_max);
    }
    if (done < bytes) {
        cudaGetLastError();
        for (size_t u = 0; u < done; u += piece) cudaHostUnregister(static_cast<char*>(p) + u);
        std::free(p);
        return false;
    }
    *base_out = static_cast<char*>(p);
    return true;
}

void unpin_segment(ipkv* h, int k) {
    char* p = h->pseg[size_t(k)].base;
    if (!p) return;
    const size_t bytes = p_segment_bytes(h, k);
    const size_t layer_bytes = bytes / size_t(h->cfg.n_layers);
    const size_t piece = (layer_bytes % 4096 == 0) ? layer_bytes : bytes;
    for (size_t u = 0; u < bytes; u += piece) cudaHostUnregister(p + u);
    std::free(p);
    h->pseg[size_t(k)].base = nullptr;
}

// The pinning thread: page-locks the requested segments in order.
void pin_worker(ipkv* h) {
    cudaSetDevice(h->cfg.device);
    std::unique_lock<std::mutex> lk(h->pmu);
    for (;;) {
        h->pcv.wait(lk, [&] { return h->p_quit || (!h->p_failed && h->p_ready < h->p_requested); });
        if (h->p_quit) return;
        const int k = h->p_ready;
        const size_t bytes = p_segment_bytes(h, k);
        lk.unlock();
        const auto t0 = std::chrono::steady_clock::now();
        char* p = nullptr;
        const bool ok = pin_segment(h, k, true, &p);
        const auto t1 = std::chrono::steady_clock::now();
        lk.lock();
        if (!ok) {
            h->p_failed = true;
        } else {
            h->pseg[size_t(k)].base = p;
            h->p_ready = k + 1;
            h->p_pinned_bytes += bytes;
            h->p_pin_us += uint64_t(std::chrono::duration_cast<std::chrono::microseconds>(t1 - t0).count());
        }
        h->pcv.notify_all();
    }
}

// Ask for segments [0, upto] to be pinned (no wait).
void p_request(ipkv* h, int upto) {
    upto = std::min(upto, int(h->pseg.size()) - 1);
    std::lock_guard<std::mutex> lk(h->pmu);
    if (upto + 1 > h->p_requested) { h->p_requested = upto + 1; h->pcv.notify_all(); }
}

// Make sure segment k is usable; normally it was pinned a window ago and this returns at once.
ipkv_status p_ensure(ipkv* h, int k) {
    if (k < 0 || k >= int(h->pseg.size())) return fail(h, IPKV_ERANGE, "P block beyond the capacity of P");
    std::unique_lock<std::mutex> lk(h->pmu);
    if (k < h->p_ready) return IPKV_OK;
    if (k + 1 > h->p_requested) { h->p_requested = k + 1; h->pcv.notify_all(); }
    const auto t0 = std::chrono::steady_clock::now();
    h->p_waiters += 1;
    h->pcv.notify_all();
    h->pcv.wait(lk, [&] { return h->p_failed || k < h->p_ready; });
    h->p_waiters -= 1;
    h->stats.p_grow_waits += 1;
    h->stats.p_grow_wait_us += uint64_t(std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now() - t0).count());
    if (k >= h->p_ready) return fail(h, IPKV_ENOMEM, "could not pin the next segment of P");
    return IPKV_OK;
}

// Host address of P block `blk` of (layer, seq) and how many blocks from there are contiguous in host memory.
ipkv_status p_locate(ipkv* h, int layer, int seq, int64_t blk, char** ptr, int64_t* contiguous) {
    if (!h->grow_p) {
        *ptr = h->p_host + (h->seq_index(layer, seq) * h->p_cap + blk) * h->bb;
        *contiguous = h->p_cap - blk;
        return IPKV_OK;
    }
    const int k = h->p_segment_of(blk);
    ipkv_status rc = p_ensure(h, k);
    if (rc != IPKV_OK) return rc;
    const ipkv::PSegment& sg = h->pseg[size_t(k)];
    *ptr = sg.base + (h->seq_index(layer, seq) * sg.nb + (blk - sg.b0)) * h->bb;
    *contiguous = sg.b0 + sg.nb - blk;
    return IPKV_OK;
}

// Calls fn(host_ptr, first_block, n_blocks) for every host-contiguous piece of P blocks [lo, hi) of (layer, seq).
template <class F>
ipkv_status for_p_pieces(ipkv* h, int layer, int seq, int64_t lo, int64_t hi, F&& fn) {
    while (lo < hi) {
        char* ptr = nullptr;
        int64_t contiguous = 0;
        ipkv_status rc = p_locate(h, layer, seq, lo, &ptr, &contiguous);
        if (rc != IPKV_OK) return rc;
        const int64_t n = std::min(hi - lo, contiguous);
        rc = fn(ptr, lo, n);
        if (rc != IPKV_OK) return rc;
        lo += n;
    }
    return IPKV_OK;
}

// A batch was placed in P blocks up to `last_blk`: pin the segment after the one it landed in (one window ahead).
void p_note_placed(ipkv* h, int64_t last_blk) {
    if (h->grow_p) p_request(h, h->p_segment_of(last_blk) + 1);
}

ipkv_status validate(const ipkv_config* c, std::string* why) {
    auto bad = [&](const char* m) { *why = m; return IPKV_EINVAL; };
    if (!c) return bad("config is NULL");
    if (c->struct_size != sizeof(ipkv_config)) return bad("struct_size does not match this library's ipkv_config");
    if (c->n_layers <= 0 || c->max_seqs <= 0) return bad("n_layers and max_seqs must be positive");
    if (!shape_ok(c->kind, c->n_q_heads, c->n_kv_heads, c->dim_qk, c->dim_v, c->block_tokens, why)) return IPKV_EINVAL;
    if (c->window_tokens <= 0 || c->window_tokens % c->block_tokens != 0) return bad("window_tokens must be a positive multiple of block_tokens");
    if (c->chunk_tokens <= 0 || c->chunk_tokens % c->block_tokens != 0) return bad("chunk_tokens must be a positive multiple of block_tokens");
    if (c->n_slots < 2) return bad("n_slots must be at least 2");
    if (c->max_u_tokens_per_seq < 0 || c->max_p_tokens_per_seq < 0 || c->resident_tokens_per_seq < 0) return bad("negative capacity");
    if (c->resident_tokens_by_seq)
        for (int s = 0; s < c->max_seqs; ++s)
            if (c->resident_tokens_by_seq[s] < 0) return bad("negative capacity in resident_tokens_by_seq");
    if (c->share_den <= 0 || c->share_num < 0 || c->share_num > c->share_den) return bad("share must satisfy 0 <= num <= den, den > 0");
    if (!(c->softmax_scale >= 0.f) || std::isinf(c->softmax_scale)) return bad("softmax_scale must be finite and non-negative");
    if (c->flags & IPKV_FLAG_GROW_P) {
        if (c->flags & IPKV_FLAG_NO_HOST_P) return bad("IPKV_FLAG_GROW_P needs the host copy of P");
        if (c->p_host_pinned) return bad("IPKV_FLAG_GROW_P: the library pins P itself, p_host_pinned must be NULL");
        if (c->p_initial_tokens_per_seq < 0 || c->p_initial_tokens_per_seq > c->max_p_tokens_per_seq) return bad("p_initial_tokens_per_seq out of range");
        if (c->p_initial_tokens_per_seq % c->chunk_tokens != 0) return bad("p_initial_tokens_per_seq must be a multiple of chunk_tokens");
        if (c->chunk_tokens % c->window_tokens != 0) return bad("IPKV_FLAG_GROW_P: chunk_tokens must be a multiple of window_tokens");
    }
    return IPKV_OK;
}

void compute_sizes(const ipkv_config* c, int64_t* bb, int64_t* u_cap, int64_t* p_cap, RingMap* ring, size_t sizes[5]) {
    const BlockGeom g = make_geom(c->kind, c->n_kv_heads, c->dim_qk, c->dim_v, c->block_tokens);
    *bb = g.block_bytes();
    const int64_t bt = c->block_tokens;
    // +1 block: a run always starts on a block boundary, so an explicit partial eviction can waste one
    *u_cap = (c->max_u_tokens_per_seq + bt - 1) / bt + (c->max_u_tokens_per_seq > 0 ? 1 : 0);
    *p_cap = (c->max_p_tokens_per_seq + bt - 1) / bt + (c->max_p_tokens_per_seq > 0 ? 1 : 0);
    ring->init(c->max_seqs, c->resident_tokens_per_seq, c->resident_tokens_by_seq, bt);
    const int64_t seqs = int64_t(c->n_layers) * c->max_seqs;
    sizes[0] = (c->flags & IPKV_FLAG_NO_HOST_U) ? 0 : size_t(seqs * *u_cap * *bb);
    sizes[1] = (c->flags & IPKV_FLAG_NO_HOST_P) ? 0 : size_t(seqs * *p_cap * *bb);
    if (c->flags & IPKV_FLAG_GROW_P) sizes[1] = size_t(seqs * (c->p_initial_tokens_per_seq / bt) * *bb);   // what create pins
    sizes[2] = size_t(seqs * (c->window_tokens / bt) * *bb);
    sizes[3] = size_t(int64_t(c->n_layers) * ring->total() * *bb);
    sizes[4] = size_t(int64_t(c->n_slots) * c->max_seqs * (c->chunk_tokens / bt) * *bb);
}

ipkv_status check_ls(ipkv* h, int layer, int seq) {
    if (!h) return IPKV_EINVAL;
    if (layer < 0 || layer >= h->cfg.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (seq < 0 || seq >= h->cfg.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
    return IPKV_OK;
}

// Record a P run for the attention scheduler: consecutive whole blocks extend the previous run.
void note_p_run(SeqState& s, const Run& r, int64_t bt) {
    if (!s.p_runs.empty()) {
        PRun& last = s.p_runs.back();
        if (last.n_tokens % bt == 0 && last.first_block + last.n_tokens / bt == r.first_block) {
            last.n_tokens += r.n_tokens;
            return;
        }
    }
    s.p_runs.push_back(PRun{r.first_block, r.n_tokens});
}

ipkv_status ensure_staging(ipkv* h, size_t bytes) {
    if (h->staging_bytes >= bytes) return IPKV_OK;
    CU(h, cudaDeviceSynchronize());
    if (h->staging) cudaFree(h->staging);
    h->staging = nullptr; h->staging_bytes = 0;
    CU(h, cudaMalloc(&h->staging, bytes));
    h->staging_bytes = bytes;
    return IPKV_OK;
}

struct BounceJob { std::vector<void*> dst; std::vector<const void*> src; std::vector<size_t> bytes; };
void CUDART_CB bounce_to_unpinned(void* arg) {
    BounceJob* j = static_cast<BounceJob*>(arg);
    for (size_t i = 0; i < j->dst.size(); ++i) std::memcpy(j->dst[i], j->src[i], j->bytes[i]);
    delete j;
}

// Evict the windows of the listed sequences of one layer (Sec. 4.2): each is one whole batch, routed to U or P.
// The compute stream only takes a device-side snapshot of the batches (and refreshes the resident ring); the
// device-to-host write-back runs on the copy stream, so it rides the otherwise idle D2H direction and decode steps
// stay flat. Neighbouring sequences with the same destination are handled by one launch / one copy (a batch that
// advances in lockstep evicts every sequence of a layer to the same side). Host contents are complete once the
// copy stream has drained (sync_host()).
// Something is about to write device-side K/V of `layer` (all layers if negative): a standalone operation, or with
// `inside_launch` the next attention launch itself (fused append).
void note_kv_write(ipkv* h, int layer, bool inside_launch = false, bool window_only = false) {
    const uint64_t at = h->launch_seq + 1 + (inside_launch ? 1 : 0);
    for (int l = 0; l < int(h->kv_written_at.size()); ++l) {
        if (layer >= 0 && l != layer) continue;
        h->w_written_at[l] = std::max(h->w_written_at[l], at);
        if (!window_only) h->kv_written_at[l] = std::max(h->kv_written_at[l], at);
    }
}

// Bounds-checked build: the host computes the destinations of the packing and ring-refresh kernels; a destination that
// does not lie inside the part of the ring that belongs to (layer, seq) is an internal error and nothing is launched.
ipkv_status check_ring_range(ipkv* h, int layer, int seq, const char* dst, int64_t bytes) {
    if (!kChecked) return IPKV_OK;
    const char* lo = h->ring_layer(layer) + h->ring_off(seq);
    const char* hi = lo + h->ring_of(seq) * h->bb;
    if (dst < lo || dst + bytes > hi) return fail(h, IPKV_EINTERNAL, "bounds-checked build: a ring destination left its sequence's part of the ring");
    return IPKV_OK;
}

ipkv_status flush_layer(ipkv* h, int layer, const int* seqs_in, int n, cudaStream_t s) {
    note_kv_write(h, layer);
    const bool no_u = h->cfg.flags & IPKV_FLAG_NO_HOST_U, no_p = h->cfg.flags & IPKV_FLAG_NO_HOST_P;
    struct Job { int seq; Run r; int64_t nb; };
    std::vector<int> seqs(seqs_in, seqs_in + n);
    std::sort(seqs.begin(), seqs.end());
    // pass 1: capacity checks for every sequence before anything changes
    for (int seq : seqs) {
        SeqState& st = h->state(layer, seq);
        const int64_t fill = st.router.window_fill();
        if (fill == 0) continue;
        const int64_t nb = st.router.blocks_for(fill);
        if (st.router.peek_eviction_side() == REGION_U) {
            if (st.router.blocks_used(REGION_U) + nb > h->u_cap) return fail(h, IPKV_ERANGE, "eviction would exceed the capacity of U");
        } else {
            if (st.router.blocks_used(REGION_P) + nb > h->p_cap) return fail(h, IPKV_ERANGE, "eviction would exceed the capacity of P");
            if (no_p && st.router.blocks_used(REGION_P) + nb > h->ring_of(seq))
                return fail(h, IPKV_ERANGE, "eviction would push P blocks out of the resident ring, and no host copy of P exists");
        }
    }
    std::vector<Job> jobs;
    bool need_wb = false;
    for (int seq : seqs) {
        SeqState& st = h->state(layer, seq);
        if (st.router.window_fill() == 0) continue;
        const int64_t nb = st.router.blocks_for(st.router.window_fill());
        const Run r = st.router.evict();
        jobs.push_back(Job{seq, r, nb});
        h->stats.flushes += 1;
        h->stats.flushes_to_u += (r.region == REGION_U);
        need_wb |= (r.region == REGION_U) ? !no_u : !no_p;
        if (r.region == REGION_P) note_p_run(st, r, h->cfg.block_tokens);
    }
    if (jobs.empty()) return IPKV_OK;
    if (need_wb && h->wb_busy_set[layer]) CU(h, cudaStreamWaitEvent(s, h->wb_busy[layer], 0));   // previous write-back of this layer
    const int64_t win_bytes = h->w_blocks * h->bb;
    const int64_t layer_off = h->w_layer(layer) - h->w_dev;
    // groups of neighbouring sequences with the same destination: [g0, g1) in `jobs`
    std::vector<std::pair<size_t, size_t>> groups;
    for (size_t i = 0; i < jobs.size();) {
        size_t j = i + 1;
        while (j < jobs.size() && jobs[j].seq == jobs[j - 1].seq + 1 && jobs[j].r.region == jobs[i].r.region) ++j;
        groups.push_back({i, j});
        i = j;
    }
    // ---- compute stream: snapshots of the evicted windows, refresh of the resident ring ----
    CopySpans spans;
    int n_spans = 0;
    auto flush_spans = [&]() -> ipkv_status {
        if (n_spans > 0) { CU(h, launch_copy_spans(spans, n_spans, s)); n_spans = 0; }
        return IPKV_OK;
    };
    for (const auto& g : groups) {
        const Job& first = jobs[g.first];
        const int64_t n_seq_g = int64_t(g.second - g.first);
        const char* src = h->w_layer(layer) + h->w_off(first.seq);
        char* snap = h->wb_stage ? h->wb_stage + layer_off + h->w_off(first.seq) : nullptr;
        if (first.r.region == REGION_U) {
            if (!no_u) {
                CU(h, launch_tile_to_plain(h->geom, src, snap, n_seq_g * h->w_blocks, s));
                h->stats.pack_kernels += 1;
            }
        } else {
            if (!no_p) {
                CU(h, cudaMemcpyAsync(snap, src, size_t(n_seq_g * win_bytes), cudaMemcpyDeviceToDevice, s));
                h->stats.d2d_bytes += uint64_t(n_seq_g * win_bytes);
            }
            if (h->rmap.total() > 0)
                for (size_t k = g.first; k < g.second; ++k) {
                    const Job& j = jobs[k];
                    const int64_t ring = h->ring_of(j.seq);
                    if (ring == 0) continue;
                    const char* wsrc = h->w_layer(layer) + h->w_off(j.seq);
                    int64_t j0 = j.r.first_block, j1 = j.r.first_block + j.nb;
                    if (j1 - j0 > ring) { wsrc += (j1 - j0 - ring) * h->bb; j0 = j1 - ring; }   // only the newest fit
                    char* base = h->ring_layer(layer) + h->ring_off(j.seq);
                    while (j0 < j1) {
                        const int64_t pos = j0 % ring;
                        const int64_t cnt = std::min(j1 - j0, ring - pos);
                        { ipkv_status crc = check_ring_range(h, layer, j.seq, base + pos * h->bb, cnt * h->bb); if (crc != IPKV_OK) return crc; }
                        spans.src[n_spans] = wsrc; spans.dst[n_spans] = base + pos * h->bb; spans.bytes[n_spans] = cnt * h->bb;
                        h->stats.d2d_bytes += uint64_t(cnt * h->bb);
                        if (++n_spans == kCopySpansPerLaunch) { ipkv_status rc = flush_spans(); if (rc != IPKV_OK) return rc; }
                        wsrc += cnt * h->bb; j0 += cnt;
                    }
                }
        }
    }
    { ipkv_status rc = flush_spans(); if (rc != IPKV_OK) return rc; }
    if (!need_wb) return IPKV_OK;
    // ---- copy stream: write-back ----
    CU(h, cudaEventRecord(h->ev_wb, s));
    CU(h, cudaStreamWaitEvent(h->copy, h->ev_wb, 0));
    for (const auto& g : groups) {
        const Job& first = jobs[g.first];
        const int64_t n_seq_g = int64_t(g.second - g.first);
        const char* snap = h->wb_stage + layer_off + h->w_off(first.seq);
        if (first.r.region == REGION_U) {
            if (no_u) continue;
            // U is unpinned: the group lands in the pinned bounce buffer, then a host callback moves every batch
            // to its place in U (stream-ordered, so the bounce buffer is free again before the next copy)
            char* bounce = h->wb_bounce + h->w_off(first.seq);
            CU(h, cudaMemcpyAsync(bounce, snap, size_t(n_seq_g * win_bytes), cudaMemcpyDeviceToHost, h->copy));
            BounceJob* bj = new (std::nothrow) BounceJob();
            if (!bj) return fail(h, IPKV_ENOMEM, "out of host memory");
            for (size_t k = g.first; k < g.second; ++k) {
                bj->dst.push_back(h->u_ptr(layer, jobs[k].seq, jobs[k].r.first_block));
                bj->src.push_back(h->wb_bounce + h->w_off(jobs[k].seq));
                bj->bytes.push_back(size_t(jobs[k].nb * h->bb));
                h->stats.d2h_bytes += uint64_t(jobs[k].nb * h->bb);
            }
            CU(h, cudaLaunchHostFunc(h->copy, bounce_to_unpinned, bj));
        } else {
            if (no_p) continue;
            for (size_t k = g.first; k < g.second; ++k) {
                const Job& j = jobs[k];
                const char* snap_k = h->wb_stage + layer_off + h->w_off(j.seq);
                ipkv_status rc = for_p_pieces(h, layer, j.seq, j.r.first_block, j.r.first_block + j.nb,
                                              [&](char* dst, int64_t b, int64_t nblk) -> ipkv_status {
                    CU(h, cudaMemcpyAsync(dst, snap_k + (b - j.r.first_block) * h->bb, size_t(nblk * h->bb), cudaMemcpyDeviceToHost, h->copy));
                    h->stats.d2h_bytes += uint64_t(nblk * h->bb);
                    return IPKV_OK;
                });
                if (rc != IPKV_OK) return rc;
                p_note_placed(h, j.r.first_block + j.nb - 1);
            }
        }
    }
    CU(h, cudaEventRecord(h->wb_busy[layer], h->copy));
    h->wb_busy_set[layer] = 1;
    return IPKV_OK;
}

// Host-visible contents of U and P are complete after this.
ipkv_status sync_host(ipkv* h) {
    if (h->copy) CU(h, cudaStreamSynchronize(h->copy));
    return IPKV_OK;
}

// Upload a table image; returns its device address. Identical consecutive images are uploaded once.
ipkv_status upload_table(ipkv* h, const Plan& plan, cudaStream_t s, const char** dev_out) {
    const size_t bytes = align_up(plan.table_bytes(), 256);
    std::vector<char> img(bytes, 0);
    plan.serialize(img.data());
    if (h->last_table_valid && h->last_table_stream == s && h->last_table.size() == bytes &&
        std::memcmp(h->last_table.data(), img.data(), bytes) == 0) {
        *dev_out = h->table_dev + h->last_table_off;
        return IPKV_OK;
    }
    const size_t part_cap = h->table_cap / ipkv::kTableParts;
    if (bytes > part_cap) {
        // grow the rings (rare: very large batches)
        CU(h, cudaDeviceSynchronize());
        const size_t cap = align_up(bytes * ipkv::kTableParts * 2, 4096);
        if (h->table_pinned) cudaFreeHost(h->table_pinned);
        if (h->table_dev) cudaFree(h->table_dev);
        h->table_pinned = nullptr; h->table_dev = nullptr; h->table_cap = 0;
        CU(h, cudaMallocHost(&h->table_pinned, cap));
        CU(h, cudaMalloc(&h->table_dev, cap));
        h->table_cap = cap; h->table_head = 0; h->table_part = 0;
        for (int i = 0; i < ipkv::kTableParts; ++i) h->table_ev_set[i] = false;
        h->last_table_valid = false;
    }
    const size_t pc = h->table_cap / ipkv::kTableParts;
    size_t part_begin = size_t(h->table_part) * pc;
    if (h->table_head + bytes > part_begin + pc || (h->last_table_valid && h->last_table_stream != s)) {
        // leave this part: mark it with an event on the stream that used it, enter the next one when it is free
        if (h->last_table_valid) {
            CU(h, cudaEventRecord(h->table_ev[h->table_part], h->last_table_stream));
            h->table_ev_set[h->table_part] = true;
        }
        h->table_part = (h->table_part + 1) % ipkv::kTableParts;
        if (h->table_ev_set[h->table_part]) CU(h, cudaEventSynchronize(h->table_ev[h->table_part]));
        part_begin = size_t(h->table_part) * pc;
        h->table_head = part_begin;
    }
    const size_t off = h->table_head;
    std::memcpy(h->table_pinned + off, img.data(), bytes);
    CU(h, cudaMemcpyAsync(h->table_dev + off, h->table_pinned + off, bytes, cudaMemcpyHostToDevice, s));
    h->stats.h2d_bytes += bytes;
    h->table_head += bytes;
    h->last_table.swap(img);
    h->last_table_off = off; h->last_table_stream = s; h->last_table_valid = true;
    *dev_out = h->table_dev + off;
    return IPKV_OK;
}

ipkv_status ensure_scratch(ipkv* h, size_t bytes) {
    if (h->scratch_bytes >= bytes) return IPKV_OK;
    CU(h, cudaDeviceSynchronize());
    if (h->scratch) cudaFree(h->scratch);
    h->scratch = nullptr; h->scratch_bytes = 0;
    const size_t want = align_up(bytes + bytes / 4, 1 << 20);
    CU(h, cudaMalloc(&h->scratch, want));
    h->scratch_bytes = want;
    return IPKV_OK;
}

void fill_launch(AttnLaunch* a, int kind, int Hq, int Hkv, int dqk, int dv, int bt, float scale, const Plan& plan,
                 const char* table_dev, char* partials, const void* q, int n_rows, size_t extra_partials = 0) {
    a->kind = kind; a->n_q_heads = Hq; a->n_kv_heads = Hkv; a->dim_qk = dqk; a->dim_v = dv; a->bt = bt; a->scale = scale;
    a->q = q;
    const PartGeom pg = part_geom(kind, Hq, Hkv);
    size_t o = 0;
    a->segs = reinterpret_cast<const Seg*>(table_dev + o);
    o += align_up(plan.segs.size() * sizeof(Seg), 16);
    a->spans = reinterpret_cast<const Span*>(table_dev + o);
    o += align_up(plan.spans.size() * sizeof(Span), 16);
    a->cta_span_start = reinterpret_cast<const int32_t*>(table_dev + o);
    o += align_up(plan.cta_span_start.size() * sizeof(int32_t), 16);
    a->rg_span_start = reinterpret_cast<const int32_t*>(table_dev + o);
    o += align_up(plan.rg_span_start.size() * sizeof(int32_t), 16);
    a->cta_tiles = reinterpret_cast<const int32_t*>(table_dev + o);
    a->n_spans = int(plan.spans.size());
    a->n_ctas = plan.n_ctas();
    a->n_rows = n_rows;
    a->n_gh = pg.n_gh;
    int64_t tiles = 0;
    for (const Span& sp : plan.spans) tiles += sp.ntiles;
    a->parts_per_span = parts_per_span_for(kind, tiles, int64_t(plan.spans.size()), int64_t(plan.n_ctas()));
    static const int forced_parts = [] { const char* e = std::getenv("IPKV_PARTS_PER_SPAN"); return e ? std::atoi(e) : 0; }();
    if (kind != 1 && (forced_parts == 1 || forced_parts == 4)) a->parts_per_span = forced_parts;     // test hook
    const size_t rows = (plan.spans.size() + extra_partials) * size_t(a->parts_per_span) * pg.rows_per_group;
    a->part_rows = int64_t(rows);
    a->part_o = reinterpret_cast<float*>(partials);
    a->part_lse = reinterpret_cast<float*>(partials + align_up(rows * dv * sizeof(float), 256));
}

// One group of segments for all rows: attention + split reduce, folding into (out_o, out_lse) when `fold`.
ipkv_status run_group(ipkv* h, std::vector<std::vector<PlanSeg>>& rows, const char* const bases[kMaxBases],
                      const void* q, int kv_splits, const float* fold_o, const float* fold_lse, float* out_o, float* out_lse,
                      cudaStream_t s, int schedule_flags = 0, const void* append_k = nullptr, const void* append_v = nullptr,
                      int layer = -1, bool device_resident_only = false) {
    const ipkv_config& c = h->cfg;
    if (h->fail_next_launch) {
        h->fail_next_launch = false;
        return fail(h, IPKV_ECUDA, "attention launch refused (ipkv_selftest_fail_next_launch)");
    }
    const Plan* plan_ptr = nullptr;
    const PartGeom pg = part_geom(c.kind, c.n_q_heads, c.n_kv_heads);
    const int win_tail = window_tail(rows);
    // signature of everything the plan depends on (the token counts as the tables will hold them)
    std::vector<int64_t>& sig = h->plan_sig_scratch;
    sig.clear();
    sig.push_back(int64_t(rows.size())); sig.push_back(pg.n_gh); sig.push_back(kv_splits); sig.push_back(pg.ctas_per_sm);
    int64_t total_tokens = 0;
    for (const auto& row : rows) {
        sig.push_back(int64_t(row.size()));
        for (const PlanSeg& sg : row) {
            total_tokens += sg.n_tokens > 0 ? sg.n_tokens : 0;
            sig.push_back(sg.off);
            sig.push_back(sg.tail_param ? (sg.n_tokens + kTileTokens - 1) / kTileTokens * kTileTokens : sg.n_tokens);
            sig.push_back(int64_t(sg.base_id) | (sg.appended ? 1 << 8 : 0) | (sg.tail_param ? 1 << 9 : 0));
        }
    }
    const bool same_plan = h->last_table_valid && h->last_table_stream == s && sig == h->last_plan_sig;
    if (same_plan) {
        plan_ptr = &h->last_plan;
    } else {
        build_plan(rows, pg.n_gh, kv_splits, pg.ctas_per_sm, &h->last_plan);
        h->last_plan_sig = sig;
        plan_ptr = &h->last_plan;
    }
    const Plan& plan = *plan_ptr;
    // dynamic balancing (grouped-query kernel): every CTA may fill up to kStealSlots extra partials
    const size_t n_lists = rows.size() * size_t(pg.n_gh) * (1 + kStealListCap);
    const size_t steal_words = n_lists + plan.spans.size() + 2 * size_t(plan.n_ctas());
    // balancing pays once the chunks are long enough (plan.hpp)
    int64_t plan_tiles = 0;
    for (int32_t t : plan.cta_tiles) plan_tiles += t;
    const int64_t min_tiles_per_cta = min_tiles_per_cta_to_balance(int64_t(rows.size()), c.n_q_heads);
    const bool balance = !(schedule_flags & IPKV_ATTEND_STATIC_SCHEDULE) && c.kind == IPKV_GQA && plan.n_ctas() > 1 &&
                         steal_words <= size_t(ipkv::kStealWords) &&
                         ((schedule_flags & IPKV_ATTEND_BALANCE) || plan_tiles >= min_tiles_per_cta * plan.n_ctas());
    const size_t extra = balance ? size_t(plan.n_ctas()) * kStealSlots : 0;
    ipkv_status rc = ensure_scratch(h, partial_bytes(plan.spans.size() + extra, pg, c.dim_v));
    if (rc != IPKV_OK) return rc;
    const char* table = nullptr;
    if (same_plan) {
        table = h->table_dev + h->last_table_off;          // the tables of the previous launch, still in place
    } else {
        rc = upload_table(h, plan, s, &table);
        if (rc != IPKV_OK) { h->last_plan_sig.clear(); return rc; }
    }
    AttnLaunch a{};
    fill_launch(&a, c.kind, c.n_q_heads, c.n_kv_heads, c.dim_qk, c.dim_v, c.block_tokens, h->scale, plan, table, h->scratch, q,
                int(rows.size()), extra);
    if (balance) {
        const int set = int(h->steal_epoch & 1u), other = set ^ 1;
        int32_t* words = h->steal_dev + size_t(set) * ipkv::kStealWords;
        a.steal_lists = words;
        a.steal_next = words + n_lists;
        h->steal_dirty[set] = int(steal_words);
        a.steal_clear = h->steal_dev + size_t(other) * ipkv::kStealWords;     // used by the balanced launch after this one
        a.steal_clear_words = h->steal_dirty[other];
        h->steal_dirty[other] = 0;
        h->steal_epoch += 1;
    }
    for (int i = 0; i < kMaxBases; ++i) { a.bases[i] = bases[i]; a.base_bytes[i] = bases[i] ? h->region_bytes(i) : 0; }
    a.acc_o = fold_o;
    a.acc_lse = fold_lse;
    a.out_o = out_o; a.out_lse = out_lse;
    a.status = h->status_dev;
    a.append_k = append_k; a.append_v = append_v;
    a.win_tail = win_tail;
    if (a.n_spans > 0) {
        // may this launch fill its copy ring before the previous kernel has completed? (see ipkv::kv_written_at)
        if (!h->launch_stream_valid || h->launch_stream != s) {
            note_kv_write(h, -1);                   // another stream: nothing is known about what ran before
            h->launch_stream = s; h->launch_stream_valid = true;
        }
        static const bool early_allowed = std::getenv("IPKV_NO_EARLY_COPIES") == nullptr;
        a.early_tiles = 0;                                              // 1: ring tiles only, 2: window tiles too
        if (early_allowed && device_resident_only && layer >= 0 && h->launch_seq >= h->kv_written_at[layer])
            a.early_tiles = h->launch_seq >= h->w_written_at[layer] ? 2 : 1;
        if (append_k && layer >= 0) note_kv_write(h, layer, true, true);     // the kernel itself writes the new rows into the window
        h->stats.early_launches += a.early_tiles ? 1 : 0;
        h->launch_seq += 1;
        const bool sampled = h->prof_on && (h->prof_seen++ % h->prof_stride) == 0;
        const bool timed = sampled && !h->prof_reduce && h->prof_used + 2 <= h->prof_ev.size();
        if (timed) CU(h, cudaEventRecord(h->prof_ev[h->prof_used], s));
        CU(h, launch_attend(a, s));
        if (timed) { CU(h, cudaEventRecord(h->prof_ev[h->prof_used + 1], s)); h->prof_used += 2; }
        if (h->prof_on) h->prof_launches += 1;
        h->stats.attend_kernels += 1;
    }
    {
        const bool timed = h->prof_on && h->prof_reduce && ((h->prof_seen - 1) % h->prof_stride) == 0 && h->prof_used + 2 <= h->prof_ev.size();
        if (timed) CU(h, cudaEventRecord(h->prof_ev[h->prof_used], s));
        CU(h, launch_split_reduce(a, s));
        if (timed) { CU(h, cudaEventRecord(h->prof_ev[h->prof_used + 1], s)); h->prof_used += 2; }
        h->stats.reduce_kernels += 1;
    }
    h->stats.kv_bytes_attended += uint64_t(total_tokens) * uint64_t(h->bb / c.block_tokens);
    return IPKV_OK;
}

}  // namespace

// ---- C ABI --------------------------------------------------------------------------------------
extern "C" {

const char* ipkv_version(void) { return kChecked ? "ipkv 0.2 (sm_100a, bounds-checked build)" : "ipkv 0.2 (sm_100a)"; }

const char* ipkv_status_str(ipkv_status s) {
    switch (s) {
        case IPKV_OK: return "ok";
        case IPKV_EINVAL: return "invalid argument";
        case IPKV_ENOMEM: return "out of memory";
        case IPKV_ERANGE: return "capacity exceeded";
        case IPKV_ESTATE: return "illegal in this state";
        case IPKV_ECUDA: return "CUDA error";
        case IPKV_ETIMEOUT: return "device wait timed out";
        case IPKV_EINTERNAL: return "internal error";
    }
    return "unknown status";
}

const char* ipkv_last_error(const ipkv_t* h) { return h ? h->err.c_str() : "no handle"; }

ipkv_status ipkv_query_sizes(const ipkv_config* cfg, size_t out_bytes[5]) {
    std::string why;
    ipkv_status rc = validate(cfg, &why);
    if (rc != IPKV_OK || !out_bytes) return IPKV_EINVAL;
    int64_t bb, u_cap, p_cap;
    RingMap ring;
    compute_sizes(cfg, &bb, &u_cap, &p_cap, &ring, out_bytes);
    return IPKV_OK;
}

ipkv_status ipkv_destroy(ipkv_t* h) {
    if (!h) return IPKV_OK;
    DeviceGuard dev_guard(h->cfg.device);
    cudaDeviceSynchronize();
    if (h->p_thread.joinable()) {
        { std::lock_guard<std::mutex> lk(h->pmu); h->p_quit = true; }
        h->pcv.notify_all();
        h->p_thread.join();
    }
    for (size_t k = 0; k < h->pseg.size(); ++k) unpin_segment(h, int(k));
    if (h->own[0] && h->u_host) std::free(h->u_host);
    if (h->own[1] && h->p_host) cudaFreeHost(h->p_host);
    if (h->own[2] && h->w_dev) cudaFree(h->w_dev);
    if (h->own[3] && h->res_dev) cudaFree(h->res_dev);
    if (h->own[4] && h->pp_dev) cudaFree(h->pp_dev);
    if (h->staging) cudaFree(h->staging);
    if (h->scratch) cudaFree(h->scratch);
    if (h->table_pinned) cudaFreeHost(h->table_pinned);
    if (h->table_dev) cudaFree(h->table_dev);
    if (h->merge_stage) cudaFree(h->merge_stage);
    if (h->status_dev) cudaFree(h->status_dev);
    if (h->steal_dev) cudaFree(h->steal_dev);
    for (int i = 0; i < 2; ++i) {
        if (h->gather[i]) cudaFreeHost(h->gather[i]);
        if (h->gather_done[i]) cudaEventDestroy(h->gather_done[i]);
    }
    if (h->wb_stage) cudaFree(h->wb_stage);
    if (h->wb_bounce) cudaFreeHost(h->wb_bounce);
    for (auto e : h->wb_busy) if (e) cudaEventDestroy(e);
    if (h->ev_wb) cudaEventDestroy(h->ev_wb);
    if (h->ev_copy) cudaEventDestroy(h->ev_copy);
    if (h->copy) cudaStreamDestroy(h->copy);
    for (int i = 0; i < ipkv::kTableParts; ++i) if (h->table_ev[i]) cudaEventDestroy(h->table_ev[i]);
    for (auto e : h->prof_ev) cudaEventDestroy(e);
    for (auto e : h->slot_ready) cudaEventDestroy(e);
    for (auto e : h->slot_free) cudaEventDestroy(e);
    if (h->ev_main) cudaEventDestroy(h->ev_main);
    if (h->ev_p_host) cudaEventDestroy(h->ev_p_host);
    if (h->side) cudaStreamDestroy(h->side);
    delete h;
    return IPKV_OK;
}

ipkv_status ipkv_create(const ipkv_config* cfg, ipkv_t** out) {
    if (!out) return IPKV_EINVAL;
    *out = nullptr;
    std::string why;
    ipkv_status rc = validate(cfg, &why);
    if (rc != IPKV_OK) return rc;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) return IPKV_ECUDA;
    DeviceGuard dev_guard(cfg->device);
    if (dev_guard.error() != cudaSuccess) return IPKV_ECUDA;
    ipkv* h = new (std::nothrow) ipkv();
    if (!h) return IPKV_ENOMEM;
    h->cfg = *cfg;
    std::memset(&h->stats, 0, sizeof h->stats);
    h->geom = make_geom(cfg->kind, cfg->n_kv_heads, cfg->dim_qk, cfg->dim_v, cfg->block_tokens);
    h->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt(float(cfg->dim_qk));
    compute_sizes(cfg, &h->bb, &h->u_cap, &h->p_cap, &h->rmap, h->sizes);
    h->cfg.resident_tokens_by_seq = nullptr;        // the capacities were copied: the caller's array need not outlive the call
    h->w_blocks = cfg->window_tokens / cfg->block_tokens;
    h->chunk_blocks = cfg->chunk_tokens / cfg->block_tokens;

    auto bail = [&](ipkv_status s) { ipkv_destroy(h); return s; };
    struct Prov { void* p; size_t n; } prov[5] = {{cfg->u_host, cfg->u_bytes}, {cfg->p_host_pinned, cfg->p_bytes},
                                                  {cfg->w_dev, cfg->w_bytes}, {cfg->resident_dev, cfg->resident_bytes},
                                                  {cfg->pp_dev, cfg->pp_bytes}};
    char** dst[5] = {&h->u_host, &h->p_host, &h->w_dev, &h->res_dev, &h->pp_dev};
    h->grow_p = (cfg->flags & IPKV_FLAG_GROW_P) != 0;
    if (h->grow_p) {
        const int64_t nb0 = cfg->p_initial_tokens_per_seq / cfg->block_tokens;
        h->pseg.push_back(ipkv::PSegment{nullptr, 0, nb0});
        for (int64_t b = nb0; b < h->p_cap; b += h->w_blocks)
            h->pseg.push_back(ipkv::PSegment{nullptr, b, h->w_blocks});   // the last one may reach past p_cap: capacity checks use p_cap
        if (nb0 > 0) {                            // the prefill share: pinned here, "during model loading and warm-up"
            char* p0 = nullptr;
            const auto t0 = std::chrono::steady_clock::now();
            if (!pin_segment(h, 0, false, &p0)) return bail(IPKV_ENOMEM);
            h->pseg[0].base = p0;
            h->p_pinned_bytes = h->sizes[1];
            h->p_pin_us = uint64_t(std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now() - t0).count());
        }
        h->p_ready = h->p_requested = 1;
        h->p_thread = std::thread(pin_worker, h);
        p_request(h, 1);                          // the first decode batch's segment, one window ahead
    }
    for (int i = 0; i < 5; ++i) {
        if (h->sizes[i] == 0 || (i == 1 && h->grow_p)) continue;
        if (prov[i].p) {
            if (prov[i].n < h->sizes[i]) return bail(IPKV_ENOMEM);
            *dst[i] = static_cast<char*>(prov[i].p);
        } else {
            void* p = nullptr;
            if (i == 0) { p = std::malloc(h->sizes[i]); if (!p) return bail(IPKV_ENOMEM); }
            else if (i == 1) { if (cudaMallocHost(&p, h->sizes[i]) != cudaSuccess) return bail(IPKV_ENOMEM); }
            else { if (cudaMalloc(&p, h->sizes[i]) != cudaSuccess) return bail(IPKV_ENOMEM); }
            *dst[i] = static_cast<char*>(p);
            h->own[i] = true;
        }
        if (i >= 2 && cudaMemset(*dst[i], 0, h->sizes[i]) != cudaSuccess) return bail(IPKV_ECUDA);
    }
    h->st.resize(size_t(cfg->n_layers) * cfg->max_seqs);
    h->kv_written_at.assign(size_t(cfg->n_layers), 0);
    h->w_written_at.assign(size_t(cfg->n_layers), 0);
    for (auto& s : h->st) s.router.init(cfg->block_tokens, cfg->window_tokens, cfg->share_num, cfg->share_den);

    if (cudaMalloc(&h->status_dev, 256) != cudaSuccess) return bail(IPKV_ENOMEM);
    if (cudaMemset(h->status_dev, 0, 256) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaMalloc(&h->steal_dev, 2 * size_t(ipkv::kStealWords) * sizeof(int32_t)) != cudaSuccess) return bail(IPKV_ENOMEM);
    if (cudaMemset(h->steal_dev, 0, 2 * size_t(ipkv::kStealWords) * sizeof(int32_t)) != cudaSuccess) return bail(IPKV_ECUDA);
    h->table_cap = 1 << 20;
    if (cudaMallocHost(&h->table_pinned, h->table_cap) != cudaSuccess) return bail(IPKV_ENOMEM);
    if (cudaMalloc(&h->table_dev, h->table_cap) != cudaSuccess) return bail(IPKV_ENOMEM);
    for (int i = 0; i < ipkv::kTableParts; ++i)
        if (cudaEventCreateWithFlags(&h->table_ev[i], cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaStreamCreateWithFlags(&h->copy, cudaStreamNonBlocking) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaEventCreateWithFlags(&h->ev_wb, cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaEventCreateWithFlags(&h->ev_copy, cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    h->wb_busy.resize(cfg->n_layers); h->wb_busy_set.assign(cfg->n_layers, 0);
    for (int i = 0; i < cfg->n_layers; ++i)
        if (cudaEventCreateWithFlags(&h->wb_busy[i], cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    if (h->sizes[0] > 0 || h->sizes[1] > 0 || h->grow_p) {      // some host copy is kept: snapshots of the windows for the write-back
        if (cudaMalloc(&h->wb_stage, h->sizes[2]) != cudaSuccess) return bail(IPKV_ENOMEM);
        if (h->sizes[0] > 0 && cudaMallocHost(&h->wb_bounce, size_t(int64_t(cfg->max_seqs) * h->w_blocks * h->bb)) != cudaSuccess) return bail(IPKV_ENOMEM);
    }
    h->slot_ready.resize(cfg->n_slots); h->slot_free.resize(cfg->n_slots); h->slot_free_set.assign(cfg->n_slots, 0);
    for (int i = 0; i < cfg->n_slots; ++i) {
        if (cudaEventCreateWithFlags(&h->slot_ready[i], cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
        if (cudaEventCreateWithFlags(&h->slot_free[i], cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    }
    if (cudaEventCreateWithFlags(&h->ev_main, cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaEventCreateWithFlags(&h->ev_p_host, cudaEventDisableTiming) != cudaSuccess) return bail(IPKV_ECUDA);
    if (cudaDeviceSynchronize() != cudaSuccess) return bail(IPKV_ECUDA);
    *out = h;
    return IPKV_OK;
}

ipkv_status ipkv_set_share(ipkv_t* h, int32_t num) {
    if (!h) return IPKV_EINVAL;
    if (num < 0 || num > h->cfg.share_den) return fail(h, IPKV_EINVAL, "share numerator out of range");
    h->cfg.share_num = num;
    for (auto& s : h->st) s.router.set_share(num);
    return IPKV_OK;
}

ipkv_status ipkv_reset(ipkv_t* h, int32_t seq) {
    if (!h) return IPKV_EINVAL;
    if (seq < -1 || seq >= h->cfg.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
    for (int l = 0; l < h->cfg.n_layers; ++l)
        for (int s = 0; s < h->cfg.max_seqs; ++s)
            if (seq < 0 || s == seq) { h->state(l, s).router.clear(); h->state(l, s).p_runs.clear(); }
    h->last_table_valid = false;
    return IPKV_OK;
}

ipkv_status ipkv_append_bulk(ipkv_t* h, int32_t layer, int32_t seq, const void* k_dev, const void* v_dev,
                             int64_t n_tokens, int32_t num0, int32_t den0, void* stream) {
    ipkv_status rc = check_ls(h, layer, seq);
    if (rc != IPKV_OK) return rc;
    const ipkv_config& c = h->cfg;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (n_tokens < 0 || den0 <= 0 || num0 < 0 || num0 > den0) return fail(h, IPKV_EINVAL, "bad token count or prefill share");
    if (n_tokens > 0 && (!k_dev || (c.kind == IPKV_GQA && !v_dev))) return fail(h, IPKV_EINVAL, "K/V pointer is NULL");
    SeqState& st = h->state(layer, seq);
    if (st.router.length() != 0) return fail(h, IPKV_ESTATE, "bulk append is only legal on an empty sequence");
    note_kv_write(h, layer);
    const int64_t bt = c.block_tokens;
    const int64_t n_cpu = st.router.prefill_cpu_tokens(n_tokens, num0, den0);
    const int64_t n_gpu = n_tokens - n_cpu;
    const bool no_u = c.flags & IPKV_FLAG_NO_HOST_U, no_p = c.flags & IPKV_FLAG_NO_HOST_P;
    if (st.router.blocks_for(n_cpu) > h->u_cap) return fail(h, IPKV_ERANGE, "prefill exceeds the capacity of U");
    if (st.router.blocks_for(n_gpu) > h->p_cap) return fail(h, IPKV_ERANGE, "prefill exceeds the capacity of P");
    if (no_p && st.router.blocks_for(n_gpu) > h->ring_of(seq)) return fail(h, IPKV_ERANGE, "prefill exceeds the resident ring and no host copy of P exists");
    DeviceGuard dev_guard(c.device);
    CU(h, dev_guard.error());
    Run placed[2];
    const int n_runs = st.router.bulk(n_tokens, num0, den0, placed);
    bool wrote_p_host = false;
    const int64_t k_row = int64_t(c.n_kv_heads) * c.dim_qk * 2, v_row = int64_t(c.n_kv_heads) * c.dim_v * 2;
    const size_t stage_cap = size_t(std::max<int64_t>(h->bb, (int64_t(32) << 20) / h->bb * h->bb));
    for (int i = 0; i < n_runs; ++i) {
        const Run& r = placed[i];
        const int64_t nb = st.router.blocks_for(r.n_tokens);
        const bool to_u = r.region == REGION_U;
        if (!to_u) note_p_run(st, r, bt);
        if (to_u && no_u) continue;
        const int64_t ring = h->ring_of(seq);
        const int64_t first_resident = to_u ? nb : std::max<int64_t>(0, nb - ring);   // relative block index
        int64_t j = 0;
        while (j < nb) {
            const bool resident = !to_u && j >= first_resident;
            int64_t j_end;
            char* dst;
            if (resident) {
                const int64_t pos = (r.first_block + j) % ring;
                j_end = std::min(nb, j + (ring - pos));
                dst = h->ring_layer(layer) + h->ring_off(seq) + pos * h->bb;
                rc = check_ring_range(h, layer, seq, dst, (j_end - j) * h->bb);
                if (rc != IPKV_OK) return rc;
            } else {
                if (!to_u && no_p) { j = first_resident; continue; }
                rc = ensure_staging(h, stage_cap);
                if (rc != IPKV_OK) return rc;
                j_end = std::min<int64_t>(to_u ? nb : first_resident, j + int64_t(stage_cap / h->bb));
                dst = h->staging;
            }
            const int64_t tok0 = j * bt, tok1 = std::min(r.n_tokens, j_end * bt);
            const char* ks = static_cast<const char*>(k_dev) + (r.first_token + tok0) * k_row;
            const char* vs = v_dev ? static_cast<const char*>(v_dev) + (r.first_token + tok0) * v_row : nullptr;
            CU(h, launch_pack(h->geom, to_u ? 0 : 1, ks, vs, tok1 - tok0, dst, 0, s));
            h->stats.pack_kernels += 1;
            if (to_u) {
                CU(h, cudaMemcpyAsync(h->u_ptr(layer, seq, r.first_block + j), dst, size_t((j_end - j) * h->bb), cudaMemcpyDeviceToHost, s));
                h->stats.d2h_bytes += uint64_t((j_end - j) * h->bb);
            } else if (!no_p) {
                const int64_t b_lo = r.first_block + j;
                rc = for_p_pieces(h, layer, seq, b_lo, r.first_block + j_end, [&](char* host, int64_t b, int64_t nblk) -> ipkv_status {
                    CU(h, cudaMemcpyAsync(host, dst + (b - b_lo) * h->bb, size_t(nblk * h->bb), cudaMemcpyDeviceToHost, s));
                    h->stats.d2h_bytes += uint64_t(nblk * h->bb);
                    return IPKV_OK;
                });
                if (rc != IPKV_OK) return rc;
                p_note_placed(h, r.first_block + j_end - 1);
                wrote_p_host = true;
            }
            j = j_end;
        }
    }
    if (wrote_p_host) {                        // the streamed attention path reads these bytes on another stream
        CU(h, cudaEventRecord(h->ev_p_host, s));
        h->ev_p_host_set = true;
    }
    return IPKV_OK;
}

ipkv_status ipkv_flush(ipkv_t* h, int32_t layer, int32_t seq, void* stream) {
    if (!h) return IPKV_EINVAL;
    if (layer < -1 || layer >= h->cfg.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (seq < -1 || seq >= h->cfg.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    for (int l = 0; l < h->cfg.n_layers; ++l) {
        if (layer >= 0 && l != layer) continue;
        std::vector<int> seqs;
        for (int s = 0; s < h->cfg.max_seqs; ++s)
            if (seq < 0 || s == seq) seqs.push_back(s);
        ipkv_status rc = flush_layer(h, l, seqs.data(), int(seqs.size()), static_cast<cudaStream_t>(stream));
        if (rc != IPKV_OK) return rc;
    }
    return IPKV_OK;
}

namespace {

// The routing half of a decode append (Sec. 4.2) and, unless `defer_copy`, the copy of the new rows into the windows.
// With `defer_copy` the caller's attention launch writes the rows itself (fused append).
ipkv_status append_tokens(ipkv* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* k_dev, const void* v_dev,
                          cudaStream_t s, bool defer_copy) {
    const ipkv_config& c = h->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (n_seq < 0 || (n_seq > 0 && (!seq_ids || !k_dev || (c.kind == IPKV_GQA && !v_dev)))) return fail(h, IPKV_EINVAL, "bad arguments");
    for (int i = 0; i < n_seq; ++i) {
        if (seq_ids[i] < 0 || seq_ids[i] >= c.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
        for (int j = 0; j < i; ++j) if (seq_ids[j] == seq_ids[i]) return fail(h, IPKV_EINVAL, "duplicate sequence id");
    }
    if (h->grow_p && layer == 0) {                  // one decode step further: the pinning thread paces itself by these
        std::lock_guard<std::mutex> lk(h->pmu);
        h->p_tick += 1;
        h->pcv.notify_all();
    }
    // evict full windows first, so that the newest token is always GPU-side
    {
        std::vector<int> full;
        for (int i = 0; i < n_seq; ++i)
            if (h->state(layer, seq_ids[i]).router.window_full()) full.push_back(seq_ids[i]);
        if (!full.empty()) {
            ipkv_status rc = flush_layer(h, layer, full.data(), int(full.size()), s);
            if (rc != IPKV_OK) return rc;
        }
    }
    const int64_t k_row = int64_t(c.n_kv_heads) * c.dim_qk * 2, v_row = int64_t(c.n_kv_heads) * c.dim_v * 2;
    for (int base = 0; base < n_seq; base += kAppendRowsPerLaunch) {
        const int n = std::min(kAppendRowsPerLaunch, n_seq - base);
        AppendRows rows;
        for (int i = 0; i < n; ++i) {
            SeqState& st = h->state(layer, seq_ids[base + i]);
            rows.dst_off[i] = h->w_off(seq_ids[base + i]);
            rows.slot[i] = int32_t(st.router.stage());
        }
        if (defer_copy) continue;
        note_kv_write(h, layer, false, true);
        const char* ks = static_cast<const char*>(k_dev) + base * k_row;
        const char* vs = v_dev ? static_cast<const char*>(v_dev) + base * v_row : nullptr;
        CU(h, launch_append(h->geom, ks, vs, c.dim_v, h->w_layer(layer), rows, n, s, h->region_bytes(kSegBaseWindow), h->status_dev));
        h->stats.append_kernels += 1;
    }
    return IPKV_OK;
}

// The rows of tokens that append_tokens has already staged (defer_copy) go into their window slots with the append
// kernel after all: used when the attention launch that was to write them did not happen.
ipkv_status write_staged_rows(ipkv* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* k_dev, const void* v_dev,
                              cudaStream_t s) {
    const ipkv_config& c = h->cfg;
    const int64_t k_row = int64_t(c.n_kv_heads) * c.dim_qk * 2, v_row = int64_t(c.n_kv_heads) * c.dim_v * 2;
    for (int base = 0; base < n_seq; base += kAppendRowsPerLaunch) {
        const int n = std::min(kAppendRowsPerLaunch, n_seq - base);
        AppendRows rows;
        for (int i = 0; i < n; ++i) {
            rows.dst_off[i] = h->w_off(seq_ids[base + i]);
            rows.slot[i] = int32_t(h->state(layer, seq_ids[base + i]).router.window_fill() - 1);
        }
        note_kv_write(h, layer, false, true);
        const char* ks = static_cast<const char*>(k_dev) + base * k_row;
        const char* vs = v_dev ? static_cast<const char*>(v_dev) + base * v_row : nullptr;
        CU(h, launch_append(h->geom, ks, vs, c.dim_v, h->w_layer(layer), rows, n, s, h->region_bytes(kSegBaseWindow), h->status_dev));
        h->stats.append_kernels += 1;
    }
    return IPKV_OK;
}

}  // namespace

ipkv_status ipkv_append(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq,
                        const void* k_dev, const void* v_dev, void* stream) {
    if (!h) return IPKV_EINVAL;
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    return append_tokens(h, layer, seq_ids, n_seq, k_dev, v_dev, static_cast<cudaStream_t>(stream), false);
}

ipkv_status ipkv_attend_gpu(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq,
                            const void* q_dev, const ipkv_attend_opts* opts,
                            float* o_part_dev, float* lse_part_dev, void* stream) {
    if (!h) return IPKV_EINVAL;
    const ipkv_config& c = h->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (n_seq <= 0 || !seq_ids || !q_dev || !o_part_dev || !lse_part_dev) return fail(h, IPKV_EINVAL, "bad arguments");
    if (n_seq > c.max_seqs) return fail(h, IPKV_EINVAL, "more rows than max_seqs");
    for (int i = 0; i < n_seq; ++i)
        if (seq_ids[i] < 0 || seq_ids[i] >= c.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int kv_splits = opts ? opts->kv_splits : 0;
    if (kv_splits < 0) return fail(h, IPKV_EINVAL, "kv_splits must be >= 0");
    const int static_schedule = opts ? opts->flags & (IPKV_ATTEND_STATIC_SCHEDULE | IPKV_ATTEND_BALANCE) : 0;
    cudaStream_t side = (opts && opts->side_stream) ? static_cast<cudaStream_t>(opts->side_stream) : h->side;
    DeviceGuard dev_guard(c.device);
    CU(h, dev_guard.error());
    h->stats.attend_calls += 1;
    const int64_t bt = c.block_tokens;

    const float* fold_o = opts ? opts->fold_o_dev : nullptr;
    const float* fold_lse = opts ? opts->fold_lse_dev : nullptr;
    if ((fold_o == nullptr) != (fold_lse == nullptr)) return fail(h, IPKV_EINVAL, "fold_o_dev and fold_lse_dev must be given together");

    // append first, if asked to: routing now; the rows themselves are written by the attention kernel where it can
    // (grouped-query kernel, blocks of at least one tile), by the append kernel otherwise
    const void* app_k = opts ? opts->append_k_dev : nullptr;
    const void* app_v = opts ? opts->append_v_dev : nullptr;
    bool fused_append = false;
    if (app_k) {
        fused_append = c.kind == IPKV_GQA && bt >= kTileTokens;
        ipkv_status arc = append_tokens(h, layer, seq_ids, n_seq, app_k, app_v, s, fused_append);
        if (arc != IPKV_OK) return arc;
        if (fused_append) h->stats.fused_appends += 1;
    }

    // group 0: everything already on the device (resident ring + D-window)
    std::vector<std::vector<PlanSeg>> rows(n_seq);
    int64_t max_stream_chunks = 0;
    for (int i = 0; i < n_seq; ++i) {
        const int seq = seq_ids[i];
        SeqState& st = h->state(layer, seq);
        const int64_t used = st.router.blocks_used(REGION_P);
        const int64_t ring = h->ring_of(seq);
        const int64_t nr = std::max<int64_t>(0, used - ring);      // blocks [0, nr) are host-only
        if (nr > 0 && (c.flags & IPKV_FLAG_NO_HOST_P)) return fail(h, IPKV_EINTERNAL, "host-only P blocks without a host copy");
        max_stream_chunks = std::max(max_stream_chunks, (nr + h->chunk_blocks - 1) / h->chunk_blocks);
        for (const PRun& r : st.p_runs) {
            const int64_t nb = (r.n_tokens + bt - 1) / bt;
            int64_t j = std::max(r.first_block, nr);
            const int64_t end = r.first_block + nb;
            while (j < end) {
                const int64_t pos = j % ring;
                const int64_t n = std::min(end - j, ring - pos);
                const int64_t tok = std::min(r.n_tokens - (j - r.first_block) * bt, n * bt);
                rows[i].push_back(PlanSeg{0, h->ring_off(seq) + pos * h->bb, tok});
                j += n;
            }
        }
        if (st.router.window_fill() > 0) rows[i].push_back(PlanSeg{1, h->w_off(seq), st.router.window_fill(), fused_append});
    }
    const char* bases[kMaxBases] = {h->rmap.total() ? h->ring_layer(layer) : nullptr, h->w_layer(layer), h->pp_dev, nullptr};
    ipkv_status rc = run_group(h, rows, bases, q_dev, kv_splits, fold_o, fold_lse, o_part_dev, lse_part_dev, s, static_schedule,
                               fused_append ? app_k : nullptr, fused_append ? app_v : nullptr, layer, true);
    if (rc != IPKV_OK) {
        // The routing state already counts the new tokens.  If the launch that was to write their rows did not happen, the
        // append kernel writes them, so that the windows hold what the routing says they hold; the attention itself failed.
        if (fused_append) {
            const std::string why = h->err;
            write_staged_rows(h, layer, seq_ids, n_seq, app_k, app_v, s);
            h->err = why;
        }
        return rc;
    }
    if (max_stream_chunks == 0) return IPKV_OK;

    // groups 1..: host-only P chunks, streamed through the PP slots in overwrite-reuse order (Sec. 4.2)
    // P's host bytes were written by a prefill copy on a compute stream or by write-backs on the copy stream. The side
    // stream waits for exactly those, not for everything queued on `s`: the copies of this layer's chunks then run
    // while the previous layer's kernels are still going.
    if (h->ev_p_host_set) CU(h, cudaStreamWaitEvent(side, h->ev_p_host, 0));
    CU(h, cudaEventRecord(h->ev_copy, h->copy));
    CU(h, cudaStreamWaitEvent(side, h->ev_copy, 0));
    const int64_t chunk_bytes = h->chunk_blocks * h->bb;
    // A chunk that lies in grown segments holds chunk_blocks / w_blocks whole eviction batches. Each batch is one
    // contiguous [seq][w_blocks] range of host memory per layer, so it travels as ONE copy for all sequences (the
    // paper's load unit: a whole batch, Sec. 4.2) and the slot is laid out [batch][seq][w_blocks]; the per-sequence
    // form is kept for calls that list under half of the sequences, and for segment 0.
    const int64_t seg0_blocks = h->grow_p ? h->pseg[0].nb : INT64_MAX;
    const bool whole_batches = h->grow_p && int64_t(n_seq) * 2 >= c.max_seqs;
    const int64_t batch_bytes = int64_t(c.max_seqs) * h->w_blocks * h->bb;      // one batch of every sequence, one layer
    for (int64_t ch = 0; ch < max_stream_chunks; ++ch) {
        const int slot = int(ch % c.n_slots);
        if (h->slot_free_set[slot]) CU(h, cudaStreamWaitEvent(side, h->slot_free[slot], 0));
        const int64_t lo = ch * h->chunk_blocks;
        const bool batched = whole_batches && lo >= seg0_blocks;
        if (batched) {
            int64_t hi_all = lo;                                       // blocks some listed sequence still needs from the host
            for (int i = 0; i < n_seq; ++i) {
                const int64_t nr = std::max<int64_t>(0, h->state(layer, seq_ids[i]).router.blocks_used(REGION_P) - h->ring_of(seq_ids[i]));
                hi_all = std::max(hi_all, std::min(nr, lo + h->chunk_blocks));
            }
            for (int64_t b = lo; b < hi_all; b += h->w_blocks) {
                char* src = nullptr;
                int64_t contiguous = 0;
                rc = p_locate(h, layer, 0, b, &src, &contiguous);       // sequence 0's blocks open the batch
                if (rc != IPKV_OK) return rc;
                CU(h, cudaMemcpyAsync(h->pp_dev + slot * h->slot_bytes() + ((b - lo) / h->w_blocks) * batch_bytes, src, size_t(batch_bytes),
                                      cudaMemcpyHostToDevice, side));
                h->stats.h2d_bytes += uint64_t(batch_bytes);
            }
        }
        for (int i = 0; i < n_seq; ++i) {
            rows[i].clear();
            const int seq = seq_ids[i];
            SeqState& st = h->state(layer, seq);
            const int64_t nr = std::max<int64_t>(0, st.router.blocks_used(REGION_P) - h->ring_of(seq));
            const int64_t hi = std::min(nr, lo + h->chunk_blocks);
            if (lo >= hi) continue;
            const int64_t row_base = slot * h->slot_bytes() + int64_t(i) * chunk_bytes;
            // slot offset of block j (lo <= j < hi) of this row
            auto slot_off = [&](int64_t j) -> int64_t {
                if (!batched) return row_base + (j - lo) * h->bb;
                const int64_t batch = (j - lo) / h->w_blocks, within = (j - lo) % h->w_blocks;
                return slot * h->slot_bytes() + batch * batch_bytes + (int64_t(seq) * h->w_blocks + within) * h->bb;
            };
            if (!batched) {
                rc = for_p_pieces(h, layer, seq, lo, hi, [&](char* src, int64_t b, int64_t nblk) -> ipkv_status {
                    CU(h, cudaMemcpyAsync(h->pp_dev + slot_off(b), src, size_t(nblk * h->bb), cudaMemcpyHostToDevice, side));
                    h->stats.h2d_bytes += uint64_t(nblk * h->bb);
                    return IPKV_OK;
                });
                if (rc != IPKV_OK) return rc;
            }
            for (const PRun& r : st.p_runs) {
                const int64_t nb = (r.n_tokens + bt - 1) / bt;
                int64_t a = std::max(lo, r.first_block);
                const int64_t b = std::min(hi, r.first_block + nb);
                while (a < b) {
                    // blocks [a, e) are contiguous in the slot: the whole range, or up to the end of the batch
                    const int64_t e = batched ? std::min(b, lo + ((a - lo) / h->w_blocks + 1) * h->w_blocks) : b;
                    const int64_t tok = std::min(r.n_tokens - (a - r.first_block) * bt, (e - a) * bt);
                    rows[i].push_back(PlanSeg{2, slot_off(a), tok});
                    a = e;
                }
            }
        }
        CU(h, cudaEventRecord(h->slot_ready[slot], side));
        CU(h, cudaStreamWaitEvent(s, h->slot_ready[slot], 0));
        rc = run_group(h, rows, bases, q_dev, kv_splits, o_part_dev, lse_part_dev, o_part_dev, lse_part_dev, s, static_schedule);
        if (rc != IPKV_OK) return rc;
        CU(h, cudaEventRecord(h->slot_free[slot], s));
        h->slot_free_set[slot] = 1;
    }
    return IPKV_OK;
}

ipkv_status ipkv_attend_gpu_sparse(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* q_dev,
                                   const int64_t* p_blocks, const int32_t* row_block_start, int32_t include_window,
                                   const ipkv_attend_opts* opts, float* o_part_dev, float* lse_part_dev, void* stream) {
    if (!h) return IPKV_EINVAL;
    const ipkv_config& c = h->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (n_seq <= 0 || !seq_ids || !q_dev || !o_part_dev || !lse_part_dev || !row_block_start) return fail(h, IPKV_EINVAL, "bad arguments");
    if (n_seq > c.max_seqs) return fail(h, IPKV_EINVAL, "more rows than max_seqs");
    if (row_block_start[0] != 0 || (row_block_start[n_seq] > 0 && !p_blocks)) return fail(h, IPKV_EINVAL, "bad block lists");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int kv_splits = opts ? opts->kv_splits : 0;
    if (kv_splits < 0) return fail(h, IPKV_EINVAL, "kv_splits must be >= 0");
    const int static_schedule = opts ? opts->flags & (IPKV_ATTEND_STATIC_SCHEDULE | IPKV_ATTEND_BALANCE) : 0;
    cudaStream_t side = (opts && opts->side_stream) ? static_cast<cudaStream_t>(opts->side_stream) : h->side;
    const float* fold_o = opts ? opts->fold_o_dev : nullptr;
    const float* fold_lse = opts ? opts->fold_lse_dev : nullptr;
    if ((fold_o == nullptr) != (fold_lse == nullptr)) return fail(h, IPKV_EINVAL, "fold_o_dev and fold_lse_dev must be given together");
    DeviceGuard dev_guard(c.device);
    CU(h, dev_guard.error());
    h->stats.attend_calls += 1;
    const int64_t bt = c.block_tokens;

    // tokens held by P block j of a sequence (blocks are full except the last one of a placed run)
    auto block_tokens = [&](const SeqState& st, int64_t j) -> int64_t {
        for (const PRun& r : st.p_runs) {
            const int64_t nb = (r.n_tokens + bt - 1) / bt;
            if (j >= r.first_block && j < r.first_block + nb) return std::min<int64_t>(bt, r.n_tokens - (j - r.first_block) * bt);
        }
        return 0;
    };
    struct HostPick { int row; int64_t block; int64_t tokens; };
    std::vector<HostPick> host_picks;                       // selected blocks that are not device-resident, row-major
    std::vector<std::vector<PlanSeg>> rows(n_seq);
    for (int i = 0; i < n_seq; ++i) {
        const int seq = seq_ids[i];
        if (seq < 0 || seq >= c.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
        SeqState& st = h->state(layer, seq);
        const int64_t used = st.router.blocks_used(REGION_P);
        const int64_t ring = h->ring_of(seq);
        const int64_t nr = std::max<int64_t>(0, used - ring);
        if (row_block_start[i + 1] < row_block_start[i]) return fail(h, IPKV_EINVAL, "bad block lists");
        int64_t prev = -1;
        for (int k = row_block_start[i]; k < row_block_start[i + 1]; ++k) {
            const int64_t j = p_blocks[k];
            if (j <= prev || j >= used) return fail(h, IPKV_EINVAL, "block ordinals must be strictly increasing and inside region P");
            prev = j;
            const int64_t tok = block_tokens(st, j);
            if (tok <= 0) return fail(h, IPKV_EINTERNAL, "selected block holds no tokens");
            if (j < nr) { host_picks.push_back(HostPick{i, j, tok}); continue; }
            // resident: extend the previous segment when this block directly follows it in the ring and that one is full
            const int64_t off = h->ring_off(seq) + (j % ring) * h->bb;
            if (!rows[i].empty() && rows[i].back().base_id == 0 && rows[i].back().n_tokens % bt == 0 &&
                rows[i].back().off + (rows[i].back().n_tokens / bt) * h->bb == off)
                rows[i].back().n_tokens += tok;
            else
                rows[i].push_back(PlanSeg{0, off, tok});
        }
        if (include_window && st.router.window_fill() > 0) rows[i].push_back(PlanSeg{1, h->w_off(seq), st.router.window_fill()});
    }
    const char* bases[kMaxBases] = {h->rmap.total() ? h->ring_layer(layer) : nullptr, h->w_layer(layer), h->pp_dev, nullptr};
    ipkv_status rc = run_group(h, rows, bases, q_dev, kv_splits, fold_o, fold_lse, o_part_dev, lse_part_dev, s, static_schedule);
    if (rc != IPKV_OK) return rc;
    if (host_picks.empty()) return IPKV_OK;
    if (c.flags & IPKV_FLAG_NO_HOST_P) return fail(h, IPKV_EINTERNAL, "host-only P blocks without a host copy");

    // host-only picks: gather -> one DMA per slot -> attend, pipelined over two pinned gather buffers (Sec. 4.4)
    const int64_t slot_blocks = int64_t(c.max_seqs) * h->chunk_blocks;        // blocks one PP slot holds
    for (int b = 0; b < 2; ++b) {
        if (!h->gather[b]) CU(h, cudaMallocHost(&h->gather[b], size_t(slot_blocks * h->bb)));
        if (!h->gather_done[b]) CU(h, cudaEventCreateWithFlags(&h->gather_done[b], cudaEventDisableTiming));
    }
    CU(h, cudaEventRecord(h->ev_main, s));
    CU(h, cudaStreamWaitEvent(side, h->ev_main, 0));
    CU(h, cudaStreamSynchronize(h->copy));                 // the host reads P here: write-backs must have landed
    CU(h, cudaStreamSynchronize(s));                       // ... including prefill copies queued on the compute stream
    size_t next = 0;
    for (int64_t round = 0; next < host_picks.size(); ++round) {
        const int gb = int(round & 1), slot = int(round % c.n_slots);
        if (h->gather_busy[gb]) CU(h, cudaEventSynchronize(h->gather_done[gb]));
        for (int i = 0; i < n_seq; ++i) rows[i].clear();
        int64_t filled = 0;
        while (next < host_picks.size() && filled < slot_blocks) {
            const HostPick& pk = host_picks[next];
            char* blk_host = nullptr;
            int64_t contiguous = 0;
            ipkv_status lrc = p_locate(h, layer, seq_ids[pk.row], pk.block, &blk_host, &contiguous);
            if (lrc != IPKV_OK) return lrc;
            std::memcpy(h->gather[gb] + filled * h->bb, blk_host, size_t(h->bb));   // one memcpy per block
            const int64_t off = slot * h->slot_bytes() + filled * h->bb;
            auto& rr = rows[pk.row];
            if (!rr.empty() && rr.back().n_tokens % bt == 0 && rr.back().off + (rr.back().n_tokens / bt) * h->bb == off)
                rr.back().n_tokens += pk.tokens;
            else
                rr.push_back(PlanSeg{2, off, pk.tokens});
            ++filled; ++next;
        }
        if (h->slot_free_set[slot]) CU(h, cudaStreamWaitEvent(side, h->slot_free[slot], 0));
        CU(h, cudaMemcpyAsync(h->pp_dev + slot * h->slot_bytes(), h->gather[gb], size_t(filled * h->bb), cudaMemcpyHostToDevice, side));
        h->stats.h2d_bytes += uint64_t(filled * h->bb);
        CU(h, cudaEventRecord(h->gather_done[gb], side));
        h->gather_busy[gb] = true;
        CU(h, cudaEventRecord(h->slot_ready[slot], side));
        CU(h, cudaStreamWaitEvent(s, h->slot_ready[slot], 0));
        rc = run_group(h, rows, bases, q_dev, kv_splits, o_part_dev, lse_part_dev, o_part_dev, lse_part_dev, s, static_schedule);
        if (rc != IPKV_OK) return rc;
        CU(h, cudaEventRecord(h->slot_free[slot], s));
        h->slot_free_set[slot] = 1;
    }
    return IPKV_OK;
}

ipkv_status ipkv_attend_cpu(ipkv_t* h, int32_t layer, const int32_t* seq_ids, int32_t n_seq, const void* q_host,
                            float* o_part_host, float* lse_part_host, int32_t n_threads) {
    if (!h) return IPKV_EINVAL;
    const ipkv_config& c = h->cfg;
    if (layer < 0 || layer >= c.n_layers) return fail(h, IPKV_EINVAL, "layer out of range");
    if (n_seq <= 0 || !seq_ids || !q_host || !o_part_host || !lse_part_host) return fail(h, IPKV_EINVAL, "bad arguments");
    if (!h->u_host) return fail(h, IPKV_ESTATE, "U contents are not kept (IPKV_FLAG_NO_HOST_U): nothing for the CPU engine to read");
    DeviceGuard dev_guard(c.device);
    CU(h, dev_guard.error());
    { ipkv_status rc = sync_host(h); if (rc != IPKV_OK) return rc; }       // write-backs still in flight on the copy stream
    std::vector<CpuRun> runs;
    std::vector<int32_t> start(1, 0);
    for (int i = 0; i < n_seq; ++i) {
        if (seq_ids[i] < 0 || seq_ids[i] >= c.max_seqs) return fail(h, IPKV_EINVAL, "sequence id out of range");
        for (const Run& r : h->state(layer, seq_ids[i]).router.runs())
            if (r.region == REGION_U) runs.push_back(CpuRun{h->u_ptr(layer, seq_ids[i], r.first_block), r.n_tokens});
        start.push_back(int32_t(runs.size()));
    }
    CpuShape sh{c.n_q_heads, c.n_kv_heads, c.dim_qk, c.dim_v, h->geom.dim_v_stored, c.block_tokens, h->scale};
    if (cpu_attend_batch(sh, n_seq, static_cast<const uint16_t*>(q_host), runs.data(), start.data(), o_part_host, lse_part_host,
                         n_threads) != 0)
        return fail(h, IPKV_EINVAL, "shape not supported by the CPU engine");
    return IPKV_OK;
}

ipkv_status ipkv_merge(ipkv_t* h, int32_t n_rows, int32_t dim_v, int32_t n_parts,
                       const float* const* o_parts, const float* const* lse_parts,
                       void* o_out_dev, int32_t o_out_is_bf16, float* lse_out_dev, void* stream) {
    if (n_rows < 0 || dim_v <= 0 || dim_v % 4 != 0 || n_parts < 1 || n_parts > kMaxMergeParts || !o_parts || !lse_parts || !o_out_dev)
        return fail(h, IPKV_EINVAL, "bad merge arguments");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    DeviceGuard dev_guard(h ? h->cfg.device : -1);      // no handle: stay on the caller's device
    if (h) CU(h, dev_guard.error());
    MergeLaunch m{};
    m.n_parts = n_parts; m.n_rows = n_rows; m.dim_v = dim_v;
    m.out_o = o_out_dev; m.out_is_bf16 = o_out_is_bf16; m.out_lse = lse_out_dev;
    const size_t o_bytes = size_t(n_rows) * dim_v * sizeof(float), l_bytes = size_t(n_rows) * sizeof(float);
    const size_t per_part = align_up(o_bytes, 256) + align_up(l_bytes, 256);
    int n_host = 0;
    for (int i = 0; i < n_parts; ++i) {
        if (!o_parts[i] || !lse_parts[i]) return fail(h, IPKV_EINVAL, "NULL partial");
        cudaPointerAttributes at{};
        const cudaError_t e = cudaPointerGetAttributes(&at, o_parts[i]);
        const bool on_dev = (e == cudaSuccess) && (at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged);
        if (e != cudaSuccess) cudaGetLastError();
        if (on_dev) { m.o[i] = o_parts[i]; m.lse[i] = lse_parts[i]; continue; }
        // Pinned host memory is read by the kernel where it is: a partial is a few hundred KB, and a copy of it would wait
        // its turn on the copy engine behind whatever chunk copies are streaming (measured: 0.58 ms per join in the streamed
        // two-engine step, against tens of microseconds).  Pageable memory is staged.
        if (e == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer) {
            cudaPointerAttributes al{};
            const cudaError_t e2 = cudaPointerGetAttributes(&al, lse_parts[i]);
            if (e2 != cudaSuccess) cudaGetLastError();
            if (e2 == cudaSuccess && al.type == cudaMemoryTypeHost && al.devicePointer) {
                m.o[i] = static_cast<const float*>(at.devicePointer);
                m.lse[i] = static_cast<const float*>(al.devicePointer);
                continue;
            }
        }
        if (!h) return fail(h, IPKV_EINVAL, "host partials need a handle for staging");
        const size_t need = per_part * kMaxMergeParts;
        if (h->merge_stage_bytes < need) {
            CU(h, cudaDeviceSynchronize());
            if (h->merge_stage) cudaFree(h->merge_stage);
            h->merge_stage = nullptr; h->merge_stage_bytes = 0;
            CU(h, cudaMalloc(&h->merge_stage, need));
            h->merge_stage_bytes = need;
        }
        char* dst = h->merge_stage + size_t(n_host) * per_part;
        CU(h, cudaMemcpyAsync(dst, o_parts[i], o_bytes, cudaMemcpyHostToDevice, s));
        CU(h, cudaMemcpyAsync(dst + align_up(o_bytes, 256), lse_parts[i], l_bytes, cudaMemcpyHostToDevice, s));
        h->stats.h2d_bytes += o_bytes + l_bytes;
        m.o[i] = reinterpret_cast<const float*>(dst);
        m.lse[i] = reinterpret_cast<const float*>(dst + align_up(o_bytes, 256));
        ++n_host;
    }
    CU(h, launch_merge(m, s));
    if (h) h->stats.merge_kernels += 1;
    return IPKV_OK;
}

ipkv_status ipkv_views(ipkv_t* h, int32_t layer, int32_t seq, ipkv_extent* out, int32_t cap, int32_t* n_out) {
    ipkv_status rc = check_ls(h, layer, seq);
    if (rc != IPKV_OK) return rc;
    if (!n_out || (cap > 0 && !out)) return fail(h, IPKV_EINVAL, "bad arguments");
    SeqState& st = h->state(layer, seq);
    const auto& runs = st.router.runs();
    const int64_t bt = h->cfg.block_tokens;
    // with a grown P a run that crosses a segment boundary is reported as one extent per contiguous piece
    auto p_pieces = [&](const Run& r) -> int {
        if (!h->grow_p || r.region != REGION_P || r.n_tokens == 0) return 1;
        const int64_t last = r.first_block + (r.n_tokens + bt - 1) / bt - 1;
        return h->p_segment_of(last) - h->p_segment_of(r.first_block) + 1;
    };
    int total = st.router.window_fill() > 0 ? 1 : 0;
    for (const Run& r : runs) total += p_pieces(r);
    *n_out = total;
    if (cap < total) return cap == 0 ? IPKV_OK : fail(h, IPKV_ERANGE, "extent array too small");
    const int64_t used_p = st.router.blocks_used(REGION_P);
    const int64_t ring = h->ring_of(seq);
    const int64_t nr = std::max<int64_t>(0, used_p - ring);
    int k = 0;
    for (const Run& whole : runs) {
        const int64_t whole_nb = (whole.n_tokens + bt - 1) / bt;
        int64_t done_blocks = 0;
        for (int piece = 0, n_pieces = p_pieces(whole); piece < n_pieces; ++piece) {
            Run r = whole;
            if (n_pieces > 1) {
                r.first_block = whole.first_block + done_blocks;
                const ipkv::PSegment& sg = h->pseg[size_t(h->p_segment_of(r.first_block))];
                const int64_t nblk = std::min(whole_nb - done_blocks, sg.b0 + sg.nb - r.first_block);
                r.first_token = whole.first_token + done_blocks * bt;
                r.n_tokens = std::min(whole.n_tokens - done_blocks * bt, nblk * bt);
                done_blocks += nblk;
            }
            ipkv_extent& e = out[k++];
            e.region = r.region; e.first_token = r.first_token; e.n_tokens = r.n_tokens; e.region_block = r.first_block;
            e.block_bytes = h->bb; e.host_ptr = nullptr; e.dev_ptr = nullptr;
            const int64_t nb = (r.n_tokens + bt - 1) / bt;
            if (r.region == REGION_U) {
                e.layout = IPKV_LAYOUT_PLAIN;
                if (h->u_host) e.host_ptr = h->u_ptr(layer, seq, r.first_block);
            } else {
                e.layout = IPKV_LAYOUT_TILE;
                if (h->has_p() && r.n_tokens > 0) {
                    char* host = nullptr;
                    int64_t contiguous = 0;
                    rc = p_locate(h, layer, seq, r.first_block, &host, &contiguous);
                    if (rc != IPKV_OK) return rc;
                    e.host_ptr = host;
                }
                if (ring > 0 && r.first_block >= nr && (r.first_block % ring) + nb <= ring)
                    e.dev_ptr = h->ring_layer(layer) + h->ring_off(seq) + (r.first_block % ring) * h->bb;
            }
        }
    }
    if (st.router.window_fill() > 0) {
        ipkv_extent& e = out[k++];
        e.region = IPKV_REGION_W; e.layout = IPKV_LAYOUT_TILE; e.first_token = st.router.window_first();
        e.n_tokens = st.router.window_fill(); e.region_block = 0; e.block_bytes = h->bb;
        e.host_ptr = nullptr; e.dev_ptr = h->w_layer(layer) + h->w_off(seq);
    }
    return IPKV_OK;
}

ipkv_status ipkv_locate(ipkv_t* h, int32_t layer, int32_t seq, int64_t token,
                        int32_t* region, int64_t* region_block, int32_t* offset_in_block) {
    ipkv_status rc = check_ls(h, layer, seq);
    if (rc != IPKV_OK) return rc;
    if (!region || !region_block || !offset_in_block) return fail(h, IPKV_EINVAL, "NULL output");
    if (!h->state(layer, seq).router.locate(token, region, region_block, offset_in_block))
        return fail(h, IPKV_ERANGE, "token index out of range");
    return IPKV_OK;
}

ipkv_status ipkv_counts(ipkv_t* h, int32_t layer, int32_t seq, int64_t counts[6]) {
    ipkv_status rc = check_ls(h, layer, seq);
    if (rc != IPKV_OK) return rc;
    if (!counts) return fail(h, IPKV_EINVAL, "NULL output");
    SeqState& st = h->state(layer, seq);
    counts[0] = st.router.tokens_in(REGION_U);
    counts[1] = st.router.tokens_in(REGION_P);
    counts[2] = st.router.tokens_in(REGION_W);
    const int64_t nr = std::max<int64_t>(0, st.router.blocks_used(REGION_P) - h->ring_of(seq));
    int64_t res = 0;
    const int64_t bt = h->cfg.block_tokens;
    for (const PRun& r : st.p_runs) {
        const int64_t nb = (r.n_tokens + bt - 1) / bt;
        const int64_t j = std::max(r.first_block, nr);
        if (j < r.first_block + nb) res += r.n_tokens - (j - r.first_block) * bt;
    }
    counts[3] = res;
    counts[4] = st.router.evictions();
    counts[5] = st.router.evictions_cpu();
    return IPKV_OK;
}

ipkv_status ipkv_read_token(ipkv_t* h, int32_t layer, int32_t seq, int64_t token, void* k_out, void* v_out) {
    ipkv_status rc = check_ls(h, layer, seq);
    if (rc != IPKV_OK) return rc;
    if (!k_out) return fail(h, IPKV_EINVAL, "NULL output");
    int32_t region, off;
    int64_t blk;
    SeqState& st = h->state(layer, seq);
    if (!st.router.locate(token, &region, &blk, &off)) return fail(h, IPKV_ERANGE, "token index out of range");
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    CU(h, cudaDeviceSynchronize());
    std::vector<char> buf(size_t(h->bb));
    bool tile = true;
    const int64_t bt = h->cfg.block_tokens;
    if (region == REGION_U) {
        if (!h->u_host) return fail(h, IPKV_ESTATE, "U contents are not kept (IPKV_FLAG_NO_HOST_U)");
        std::memcpy(buf.data(), h->u_ptr(layer, seq, blk), size_t(h->bb));
        tile = false;
    } else if (region == REGION_P) {
        if (h->has_p()) {
            char* blk_host = nullptr;
            int64_t contiguous = 0;
            rc = p_locate(h, layer, seq, blk, &blk_host, &contiguous);
            if (rc != IPKV_OK) return rc;
            std::memcpy(buf.data(), blk_host, size_t(h->bb));
        } else {
            CU(h, cudaMemcpy(buf.data(), h->ring_layer(layer) + h->ring_off(seq) + (blk % h->ring_of(seq)) * h->bb, size_t(h->bb), cudaMemcpyDeviceToHost));
        }
    } else {
        const int64_t wb = off / bt;
        off = int32_t(off - wb * bt);
        CU(h, cudaMemcpy(buf.data(), h->w_layer(layer) + h->w_off(seq) + wb * h->bb, size_t(h->bb), cudaMemcpyDeviceToHost));
    }
    const BlockGeom& g = h->geom;
    for (int head = 0; head < g.n_kv_heads; ++head) {
        const char* hp = buf.data() + int64_t(head) * g.head_bytes();
        for (int ch = 0; ch < g.dim_qk / 8; ++ch) {
            const int64_t o = tile ? tile_chunk_offset(g.bt, off, ch) : plain_chunk_offset(g.dim_qk, off, ch);
            std::memcpy(static_cast<char*>(k_out) + (int64_t(head) * g.dim_qk + ch * 8) * 2, hp + o, 16);
        }
        if (v_out && g.dim_v_stored > 0)
            for (int ch = 0; ch < g.dim_v_stored / 8; ++ch) {
                const int64_t o = g.k_plane_bytes() + (tile ? tile_chunk_offset(g.bt, off, ch) : plain_chunk_offset(g.dim_v_stored, off, ch));
                std::memcpy(static_cast<char*>(v_out) + (int64_t(head) * g.dim_v_stored + ch * 8) * 2, hp + o, 16);
            }
    }
    return IPKV_OK;
}

ipkv_status ipkv_get_stats(ipkv_t* h, ipkv_stats* out) {
    if (!h || !out) return IPKV_EINVAL;
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    CU(h, cudaDeviceSynchronize());
    CU(h, cudaMemcpy(&h->stats.device_status, h->status_dev, sizeof(uint32_t), cudaMemcpyDeviceToHost));
    if (h->grow_p) {
        std::lock_guard<std::mutex> lk(h->pmu);
        h->stats.p_segments = uint64_t(h->p_ready) - (h->pseg[0].nb == 0 ? 1 : 0);
        h->stats.p_pinned_bytes = h->p_pinned_bytes;
        h->stats.p_pin_us = h->p_pin_us;
        h->stats.p_register_us = h->p_register_us;
        h->stats.p_register_calls = h->p_register_calls;
        h->stats.p_register_max_us = h->p_register_max_us;
    }
    *out = h->stats;
    if (h->stats.device_status) {
        // reported once: the word is cleared so that the calls after this one are judged on their own
        CU(h, cudaMemset(h->status_dev, 0, sizeof(uint32_t)));
        if (h->stats.device_status & kStatusBadIndex)
            return fail(h, IPKV_EINTERNAL, "bounds-checked build: an index left its region; the access was not made" +
                                               describe_device_status(h->stats.device_status));
        return fail(h, IPKV_ETIMEOUT, "a kernel's bounded wait gave up; results of that call are invalid" +
                                          describe_device_status(h->stats.device_status));
    }
    return IPKV_OK;
}

ipkv_status ipkv_selftest_expire_wait(ipkv_t* h, uint32_t limit_us, void* stream) {
    if (!h || limit_us == 0 || limit_us > 1000000u) return IPKV_EINVAL;
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    CU(h, launch_expire_wait(h->status_dev, uint64_t(limit_us) * 1000ull, static_cast<cudaStream_t>(stream)));
    return IPKV_OK;
}

ipkv_status ipkv_selftest_declare_bounds(ipkv_t* h, int32_t base_id, int64_t bytes) {
    if (!h || base_id < 0 || base_id >= kMaxBases || bytes < 0) return IPKV_EINVAL;
    if (!kChecked) return fail(h, IPKV_ESTATE, "not a bounds-checked build (libipkv_checked.so)");
    h->selftest_bounds[base_id] = bytes;
    return IPKV_OK;
}

ipkv_status ipkv_selftest_fail_next_launch(ipkv_t* h) {
    if (!h) return IPKV_EINVAL;
    h->fail_next_launch = true;
    return IPKV_OK;
}

ipkv_status ipkv_profile_enable(ipkv_t* h, int32_t on) {
    if (!h) return IPKV_EINVAL;
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    if (on && h->prof_ev.empty()) {
        h->prof_ev.resize(2 * 8192);
        for (auto& e : h->prof_ev) e = nullptr;
        for (auto& e : h->prof_ev) CU(h, cudaEventCreate(&e));
    }
    h->prof_on = on != 0;
    h->prof_reduce = (on & 3) == 2;
    h->prof_stride = (on >> 8) > 0 ? (on >> 8) : 1;
    h->prof_seen = 0;
    return IPKV_OK;
}

ipkv_status ipkv_profile_read(ipkv_t* h, double* attend_kernel_ms, int64_t* n_timed, int64_t* n_launches) {
    if (!h || !attend_kernel_ms || !n_timed || !n_launches) return IPKV_EINVAL;
    DeviceGuard dev_guard(h->cfg.device);
    CU(h, dev_guard.error());
    CU(h, cudaDeviceSynchronize());
    double total = 0.0;
    for (size_t i = 0; i + 1 < h->prof_used; i += 2) {
        float ms = 0.f;
        CU(h, cudaEventElapsedTime(&ms, h->prof_ev[i], h->prof_ev[i + 1]));
        total += ms;
    }
    *attend_kernel_ms = total;
    *n_timed = int64_t(h->prof_used / 2);
    *n_launches = h->prof_launches;
    h->prof_used = 0; h->prof_launches = 0;
    return IPKV_OK;
}

// ---- roofline share policy (host only) ----------------------------------------------------------
struct ipkv_policy {
    SharePolicy impl;
    ipkv_policy(const RooflineParams& m, int w, int d) : impl(m, w, d) {}
};

static bool roofline_ok(const ipkv_roofline* m) {
    return m && m->A > 0.0 && m->B > 0.0 && std::isfinite(m->A) && std::isfinite(m->B) && std::isfinite(m->C_cpu) &&
           std::isfinite(m->C_gpu) && m->C_cpu >= 0.0 && m->C_gpu >= 0.0;
}

double ipkv_roofline_share(const ipkv_roofline* m, double L) {
    if (!roofline_ok(m)) return NAN;
    return balanced_share(RooflineParams{m->A, m->B, m->C_cpu, m->C_gpu}, L);
}

double ipkv_roofline_step_time(const ipkv_roofline* m, double r, double L, double t_merge, double* t_cpu_out, double* t_gpu_out) {
    if (!roofline_ok(m) || !(r >= 0.0 && r <= 1.0) || !(L >= 0.0)) return NAN;
    const RooflineParams rp{m->A, m->B, m->C_cpu, m->C_gpu};
    if (t_cpu_out) *t_cpu_out = engine_time_cpu(rp, r, L);
    if (t_gpu_out) *t_gpu_out = engine_time_gpu(rp, r, L);
    return step_time(rp, r, L, t_merge);
}

ipkv_status ipkv_policy_create(const ipkv_roofline* m, int32_t window_steps, int32_t share_den, ipkv_policy_t** out) {
    if (!out) return IPKV_EINVAL;
    *out = nullptr;
    if (!roofline_ok(m) || window_steps <= 0 || share_den <= 0) return IPKV_EINVAL;
    ipkv_policy* p = new (std::nothrow) ipkv_policy(RooflineParams{m->A, m->B, m->C_cpu, m->C_gpu}, window_steps, share_den);
    if (!p) return IPKV_ENOMEM;
    *out = p;
    return IPKV_OK;
}

ipkv_status ipkv_policy_destroy(ipkv_policy_t* p) { delete p; return IPKV_OK; }

ipkv_status ipkv_policy_observe(ipkv_policy_t* p, double cpu_seconds, double cpu_tokens) {
    if (!p || !(cpu_seconds >= 0.0) || !(cpu_tokens >= 0.0) || !std::isfinite(cpu_seconds) || !std::isfinite(cpu_tokens)) return IPKV_EINVAL;
    p->impl.observe(cpu_seconds, cpu_tokens);
    return IPKV_OK;
}

ipkv_status ipkv_policy_update(ipkv_policy_t* p, int32_t* share_num_out, ipkv_roofline* model_out) {
    if (!p || !share_num_out) return IPKV_EINVAL;
    *share_num_out = p->impl.update();
    if (model_out) {
        const RooflineParams& m = p->impl.model();
        model_out->A = m.A; model_out->B = m.B; model_out->C_cpu = m.C_cpu; model_out->C_gpu = m.C_gpu;
    }
    return IPKV_OK;
}

ipkv_status ipkv_policy_prefill_share(const ipkv_policy_t* p, double L0, int32_t* share_num_out) {
    if (!p || !share_num_out || !(L0 >= 0.0)) return IPKV_EINVAL;
    *share_num_out = p->impl.prefill_numerator(L0);
    return IPKV_OK;
}

// ---- stateless entry points ---------------------------------------------------------------------

int64_t ipkv_block_bytes(const ipkv_attn_shape* sh) {
    if (!sh || !shape_ok(sh->kind, sh->n_q_heads, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens, nullptr)) return -1;
    return make_geom(sh->kind, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens).block_bytes();
}

ipkv_status ipkv_attend_scratch_bytes(const ipkv_attn_shape* sh, int32_t n_rows, int32_t n_runs,
                                      int64_t total_tokens, int32_t kv_splits, size_t* out_bytes) {
    if (!sh || !out_bytes || n_rows < 0 || n_runs < 0 || total_tokens < 0 || kv_splits < 0) return IPKV_EINVAL;
    if (!shape_ok(sh->kind, sh->n_q_heads, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens, nullptr)) return IPKV_EINVAL;
    (void)total_tokens;
    const PartGeom pg = part_geom(sh->kind, sh->n_q_heads, sh->n_kv_heads);
    const int64_t spans = max_spans_bound(n_rows, n_runs, pg.n_gh, kv_splits, pg.ctas_per_sm);
    const size_t table = align_up(size_t(n_runs) * sizeof(Seg), 16) + align_up(size_t(spans) * sizeof(Span), 16) +
                         align_up(size_t(kSmCount * pg.ctas_per_sm + 1) * sizeof(int32_t), 16) +
                         align_up((size_t(n_rows) * pg.n_gh + 1) * sizeof(int32_t), 16) +
                         align_up(size_t(kSmCount * pg.ctas_per_sm) * sizeof(int32_t), 16);
    *out_bytes = align_up(table, 256) + 256 + partial_bytes(size_t(spans), pg, sh->dim_v);
    return IPKV_OK;
}

ipkv_status ipkv_attend_runs(const ipkv_attn_shape* sh, int32_t n_rows,
                             const ipkv_run* runs, const int32_t* row_run_start,
                             const void* q_dev, int32_t kv_splits,
                             void* scratch_dev, size_t scratch_bytes,
                             float* o_part_dev, float* lse_part_dev, uint32_t* status_dev, void* stream) {
    if (!sh || n_rows <= 0 || !row_run_start || !q_dev || !scratch_dev || !o_part_dev || !lse_part_dev || kv_splits < 0) return IPKV_EINVAL;
    if (!shape_ok(sh->kind, sh->n_q_heads, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens, nullptr)) return IPKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(scratch_dev) & 255u) != 0) return IPKV_EINVAL;
    const int n_runs = row_run_start[n_rows];
    if (n_runs < 0 || (n_runs > 0 && !runs)) return IPKV_EINVAL;
    std::vector<std::vector<PlanSeg>> rows(n_rows);
    for (int r = 0; r < n_rows; ++r) {
        if (row_run_start[r] > row_run_start[r + 1] || row_run_start[r] < 0) return IPKV_EINVAL;
        for (int k = row_run_start[r]; k < row_run_start[r + 1]; ++k) {
            if (runs[k].n_tokens < 0 || (runs[k].n_tokens > 0 && !runs[k].blocks_dev)) return IPKV_EINVAL;
            if (reinterpret_cast<uintptr_t>(runs[k].blocks_dev) & 15u) return IPKV_EINVAL;
            rows[r].push_back(PlanSeg{0, int64_t(reinterpret_cast<intptr_t>(runs[k].blocks_dev)), runs[k].n_tokens});
        }
    }
    Plan plan;
    const PartGeom pg = part_geom(sh->kind, sh->n_q_heads, sh->n_kv_heads);
    build_plan(rows, pg.n_gh, kv_splits, pg.ctas_per_sm, &plan);
    const size_t table = align_up(plan.table_bytes(), 256);
    if (table + 256 + partial_bytes(plan.spans.size(), pg, sh->dim_v) > scratch_bytes) return IPKV_ENOMEM;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    std::vector<char> img(table, 0);
    plan.serialize(img.data());
    // Outside a capture the tables go up as one copy from this pageable image (the runtime stages it before returning, so
    // `img` may go out of scope).  A captured copy would be replayed from the image's address long after it is gone, so
    // under capture the tables travel as kernel parameters instead, which a graph keeps by value.
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &capturing) != cudaSuccess) return IPKV_ECUDA;
    if (capturing == cudaStreamCaptureStatusNone) {
        if (cudaMemcpyAsync(scratch_dev, img.data(), table, cudaMemcpyHostToDevice, s) != cudaSuccess) return IPKV_ECUDA;
    } else if (launch_upload_by_value(scratch_dev, img.data(), table, s) != cudaSuccess) {
        return IPKV_ECUDA;
    }
    AttnLaunch a{};
    const float scale = sh->softmax_scale > 0.f ? sh->softmax_scale : 1.0f / std::sqrt(float(sh->dim_qk));
    fill_launch(&a, sh->kind, sh->n_q_heads, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens, scale, plan,
                static_cast<const char*>(scratch_dev), static_cast<char*>(scratch_dev) + table + 256, q_dev, n_rows);
    a.bases[0] = nullptr;
    a.plain_launch = capturing == cudaStreamCaptureStatusNone ? 0 : 1;
    a.out_o = o_part_dev; a.out_lse = lse_part_dev;
    a.status = status_dev ? status_dev : reinterpret_cast<uint32_t*>(static_cast<char*>(scratch_dev) + table);
    if (a.n_spans > 0 && launch_attend(a, s) != cudaSuccess) return IPKV_ECUDA;
    if (launch_split_reduce(a, s) != cudaSuccess) return IPKV_ECUDA;
    return IPKV_OK;
}

ipkv_status ipkv_pack_blocks(const ipkv_attn_shape* sh, int32_t layout, const void* k_dev, const void* v_dev,
                             int64_t n_tokens, void* dst_dev, void* stream) {
    if (!sh || n_tokens < 0 || (n_tokens > 0 && (!k_dev || !dst_dev))) return IPKV_EINVAL;
    if (!shape_ok(sh->kind, sh->n_q_heads, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens, nullptr)) return IPKV_EINVAL;
    if (sh->kind == IPKV_GQA && n_tokens > 0 && !v_dev) return IPKV_EINVAL;
    if (layout != IPKV_LAYOUT_PLAIN && layout != IPKV_LAYOUT_TILE) return IPKV_EINVAL;
    const BlockGeom g = make_geom(sh->kind, sh->n_kv_heads, sh->dim_qk, sh->dim_v, sh->block_tokens);
    if (launch_pack(g, layout == IPKV_LAYOUT_TILE, k_dev, v_dev, n_tokens, dst_dev, 0, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return IPKV_ECUDA;
    return IPKV_OK;
}

}  // extern "C"
