// Internal state of a context and the helpers its translation units share.  Not part of the ABI.
#pragma once

#include <algorithm>
#include <atomic>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <deque>
#include <map>
#include <mutex>
#include <condition_variable>
#include <string>
#include <thread>
#include <unordered_map>
#include <vector>

#include "ps_internal.h"
#include "ps_kvswap.h"

namespace psrt {


constexpr int kSlots = 4;
constexpr int64_t kHostAlign = 4096;


inline int64_t round_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }

struct Req {
    int32_t n_tokens = 0;
    std::vector<int32_t> table;
    int32_t state = PS_REQ_RESIDENT;
    // Host image: one segment per offload issued for the request.  A segment covers logical blocks [lo, hi)
    // in the layer-major layout [L][hi - lo][K,V][slab].  On-demand offloading makes one segment; proactive
    // offloading (ps_offload_progress) adds segments as the request grows, ps_swap_out adds the last.
    struct Seg {
        int32_t lo, hi;
        int64_t off, bytes;
        uint64_t ticket;  // s_d2h ticket after the segment's last copy
    };
    std::vector<Seg> segs;
    int32_t host_issued = 0;          // blocks covered by segs
    std::vector<int32_t> layer_done;  // blocks issued per layer while SWAPPING_IN
    uint64_t out_ticket = 0;          // s_d2h ticket after the last segment
    bool gated = false;               // RESIDENT but reload copies not yet seen complete
    uint64_t in_ticket = 0;           // s_scatter ticket after the last scatter
};

struct Tracker {  // completion tickets on one stream
    cudaStream_t s = nullptr;
    std::deque<std::pair<uint64_t, cudaEvent_t>> pending;
    uint64_t next = 1, done = 0;
    // via_worker: tickets are numbered by the caller but their events are recorded by the offload worker when it
    // reaches them in its queue; `pending` is then shared between the two threads (under mu), `next` and `done`
    // stay with the caller's thread
    bool via_worker = false;
    std::mutex mu;
};

// One unit of offload work handed to the worker: a staging slot's worth of an image (gather + copy), and / or
// a completion ticket to record on the D2H stream behind everything issued before it.
struct OutChunk {
    const int32_t* d_table = nullptr;
    int32_t n_blk = 0;
    int64_t s0 = 0, cnt = 0;     // slabs [s0, s0 + cnt) of the segment's image; cnt = 0: ticket only
    char* host_dst = nullptr;
    uint64_t ticket = 0;         // != 0: record this ticket's event after the chunk's copy
};

struct Arena {  // pinned (mapped) + device ring of chunks for descriptor uploads on ONE stream
    char* h = nullptr;   // host view of the pinned buffer
    char* hd = nullptr;  // device view of the same pinned buffer (source of the upload kernel)
    char* d = nullptr;
    size_t chunk = 0;
    int nchunks = 0, cur = 0;
    size_t used = 0;
    cudaStream_t s = nullptr;
    std::vector<cudaEvent_t> fence;
    std::vector<char> fenced;
};

struct HostPool {
    int64_t cap = 0;
    std::map<int64_t, int64_t> free_;  // offset -> bytes
    void init(int64_t c) {
        cap = c;
        free_.clear();
        if (c > 0) free_[0] = c;
    }
    int64_t alloc(int64_t bytes) {
        bytes = round_up(std::max<int64_t>(bytes, 1), kHostAlign);
        for (auto it = free_.begin(); it != free_.end(); ++it) {
            if (it->second >= bytes) {
                const int64_t off = it->first, rest = it->second - bytes;
                free_.erase(it);
                if (rest > 0) free_[off + bytes] = rest;
                return off;
            }
        }
        return -1;
    }
    void release(int64_t off, int64_t bytes) {
        bytes = round_up(std::max<int64_t>(bytes, 1), kHostAlign);
        auto it = free_.emplace(off, bytes).first;
        auto nx = std::next(it);
        if (nx != free_.end() && it->first + it->second == nx->first) {
            it->second += nx->second;
            free_.erase(nx);
        }
        if (it != free_.begin()) {
            auto pv = std::prev(it);
            if (pv->first + pv->second == it->first) {
                pv->second += it->second;
                free_.erase(it);
            }
        }
    }
};

enum ProfKind { kProfAttn = 0, kProfMerge, kProfGather, kProfScatter, kProfD2H, kProfH2D, kProfKinds };

struct ProfSpan {
    int kind;
    int tag;  // layer, or -1
    cudaEvent_t e0, e1;
};

struct PlanEntry {
    int64_t req;
    int32_t lo, hi;
};

struct BatchMeta {  // cached device metadata of the last prepared decode batch
    std::vector<int64_t> reqs;
    std::vector<char> gated, active;
    uint64_t epoch = 0;
    bool valid = false;
    ps::AttnBatch dev{};
    int32_t n_items = 0, n_ungated_items = 0, n_parts = 0;
    int32_t n_gated_rows = 0;
    bool any_multi = false, lane_multi[2] = {false, false};
    bool two_lanes = false;
    int tail_mode = 0;
    int64_t kv_bytes_per_layer = 0;
};


}  // namespace psrt

using namespace psrt;

struct ps_ctx {
    ps_config cfg{};
    bool bk = false, profile = false;
    int G = 1;
    int64_t slab_bytes = 0, layer_block_bytes = 0, block_bytes = 0;
    int32_t slab_vec = 0;
    std::string err = "";

    // pool
    std::vector<int32_t> free_stack;
    std::unordered_map<int64_t, Req> reqs;
    std::deque<int64_t> out_fifo, in_fifo;
    uint64_t table_epoch = 1;

    // device resources
    std::vector<void*> kpools, vpools;
    void** d_kpools = nullptr;
    void** d_vpools = nullptr;
    char* host_pool = nullptr;
    bool own_host_pool = false;
    HostPool hpool;
    cudaStream_t compute = nullptr, s_gather = nullptr, s_d2h = nullptr, s_h2d = nullptr, s_scatter = nullptr,
                 s_lane = nullptr;
    char* stage_out = nullptr;
    char* stage_in = nullptr;
    int64_t slot_bytes = 0;
    cudaEvent_t e_gathered[kSlots]{}, e_drained[kSlots]{}, e_loaded[kSlots]{}, e_scattered[kSlots]{};
    bool out_used[kSlots]{}, in_used[kSlots]{};
    uint64_t out_next = 0, in_next = 0;
    int in_slot = -1;        // reload staging: the slot being filled and the bytes used in it (pieces are packed)
    int64_t in_fill = 0;
    std::vector<cudaEvent_t> ev_in;      // completion events of layer chunks, indexed by the chunk's first layer
    std::vector<int32_t> ev_of_layer;    // per layer: first layer of the chunk that last reloaded into it
    int64_t chunk_min_bytes = 0;         // layers are grouped into one chunk until a chunk carries this many bytes
    int64_t max_pitch = 0;               // largest row pitch of a strided copy
    cudaEvent_t e_mark = nullptr, e_mark2 = nullptr, e_fork = nullptr, e_join = nullptr;
    int32_t* status = nullptr;  // mapped pinned word written by kernels on a bad block id
    int32_t* d_status = nullptr;
    Tracker t_d2h, t_scatter, t_compute;
    Arena a_gather, a_meta, a_ids, a_scatter;
    std::vector<int32_t> scatter_ids_cache;  // ids of the last reload-plan upload and where they sit in a_scatter
    size_t scatter_ids_off = 0;
    std::vector<int32_t> ids_cache;  // ids of the last ps_copy_blocks upload and where they sit in a_ids
    size_t ids_cache_off = 0;
    std::vector<cudaEvent_t> ev_pool, ev_pool_timing;
    std::deque<std::pair<uint64_t, std::pair<int64_t, int64_t>>> img_release;  // in_ticket -> (off, bytes)
    std::deque<std::pair<uint64_t, std::pair<int64_t, int64_t>>> host_release;  // t_d2h ticket -> (off, bytes)
    std::deque<std::pair<uint64_t, int64_t>> reload_inflight;  // s_scatter ticket -> reload bytes issued before it
    std::vector<int64_t> gated_reqs;
    // split-KV scratch: sets 0 and 1 are used alternately by the launches on the compute stream (consecutive
    // launches of a step may overlap), set 2 by the launches on the reload lane
    float* partials[3] = {nullptr, nullptr, nullptr};
    int32_t* d_sched[3] = {nullptr, nullptr, nullptr};     // chunk counters of the tensor-core kernel: {next, done} per lane
    int32_t* d_row_done[3] = {nullptr, nullptr, nullptr};  // its split-KV arrival counters: max_batch x num_kv_heads
    int scratch_set = 0;
    std::vector<ps::AttnTensorMaps> tmaps;  // per layer; empty = the kernel copies row by row
    int32_t max_parts = 0;
    int attn_kernel = 1;
    int32_t num_sms = 1;
    BatchMeta meta;
    char* io_q = nullptr;    // ps_step_host: device copies of the queries and of the outputs (allocated on first use)
    char* io_out = nullptr;

    // offload worker (Section 4.3 "Asynchronous Offloading": a separate thread copies the blocks): hands the
    // copy engine at most kOutInflight staging slots at a time, so that other device-to-host copies of the
    // process queue behind that much and not behind a whole offload
    bool out_paced = false;
    int device = 0;
    std::thread out_thread;
    std::mutex out_mu;
    std::condition_variable out_cv;
    std::deque<OutChunk> out_pending;
    bool out_stop = false;
    std::atomic<bool> out_failed{false};
    std::string out_error;

    // measurement
    std::atomic<int64_t> launches{0};
    std::vector<ProfSpan> spans;
    double prof_ms[kProfKinds]{};
    int64_t prof_n[kProfKinds]{};
    int64_t prof_bytes[kProfKinds]{};
    bool tracing = false;
    cudaEvent_t trace_base = nullptr;
    std::vector<ps_trace_span> trace;

    int32_t fail(int32_t code, const std::string& msg) {
        err = msg;
        return code;
    }
    int32_t fail_cuda(cudaError_t e, const char* what) {
        err = std::string(what) + ": " + cudaGetErrorString(e);
        return PS_ERR_CUDA;
    }
};


#define CK(call)                                                 \
    do {                                                         \
        cudaError_t e__ = (call);                                \
        if (e__ != cudaSuccess) return ctx->fail_cuda(e__, #call); \
    } while (0)

namespace psrt {

std::string& create_error();  // text of the most recent ps_create / ps_link_probe failure

// events, completion trackers, descriptor arenas (ps_runtime.cu)
cudaError_t get_event(ps_ctx* ctx, bool timing, cudaEvent_t* out);
int32_t tracker_mark(ps_ctx* ctx, Tracker& t, uint64_t* ticket);
int32_t tracker_poll(ps_ctx* ctx, Tracker& t);
int32_t tracker_drain(ps_ctx* ctx, Tracker& t, bool bounded, std::chrono::steady_clock::time_point deadline);
int32_t arena_init(ps_ctx* ctx, Arena& a, size_t chunk, int nchunks, cudaStream_t s);
int32_t arena_next_chunk(ps_ctx* ctx, Arena& a, bool record_fence = true);
int32_t arena_alloc(ps_ctx* ctx, Arena& a, size_t bytes, size_t* off);
void arena_free(Arena& a);
void resolve_profile(ps_ctx* ctx);

struct ProfScope {
    ps_ctx* ctx;
    int kind;
    cudaStream_t s;
    cudaEvent_t e0 = nullptr;
    bool on = false;
    int tag;
    ProfScope(ps_ctx* c, int k, cudaStream_t st, int64_t bytes, int tg = -1, bool enabled = true)
        : ctx(c), kind(k), s(st), tag(tg) {
        if (!enabled) return;  // the offload worker's thread keeps out of the profiling state
        ctx->prof_bytes[kind] += bytes;
        ctx->prof_n[kind] += 1;
        if (ctx->profile && !ctx->bk && get_event(ctx, true, &e0) == cudaSuccess) {
            on = cudaEventRecord(e0, s) == cudaSuccess;
        }
    }
    ~ProfScope() {
        if (!on) return;
        cudaEvent_t e1;
        if (get_event(ctx, true, &e1) != cudaSuccess) return;
        cudaEventRecord(e1, s);
        ctx->spans.push_back({kind, tag, e0, e1});
    }
};


// pool helpers and completion (ps_runtime.cu)
inline int32_t blocks_for(const ps_ctx* ctx, int32_t n_tokens) {
    return (n_tokens + ctx->cfg.block_size - 1) / ctx->cfg.block_size;
}
void push_table(ps_ctx* ctx, std::vector<int32_t>& table);
int32_t check_status_word(ps_ctx* ctx);
// reap_offloads = false: only the side tasks (host images of landed reloads, reload gates, parked ranges);
// finished offloads give their blocks back in ps_poll / ps_step / ps_sync alone, which report how many, so a
// caller can follow the free-block count exactly.
int32_t do_poll(ps_ctx* ctx, int32_t* n_reaped, bool reap_offloads = true);

// offload worker (ps_swap.cu)
constexpr int kOutInflight = 2;
void out_worker_main(ps_ctx* ctx);
cudaError_t issue_out_chunk(ps_ctx* ctx, const OutChunk& c, int slot, bool profiled);

// swap-out and swap-in issue (ps_swap.cu)
int32_t offload_segment(ps_ctx* ctx, Req& r, int32_t lo, int32_t hi);
int32_t order_scatter_after_compute(ps_ctx* ctx);
int32_t upload_plan_ids(ps_ctx* ctx, const std::vector<PlanEntry>& plan, const int32_t** d_ids);
int32_t issue_reload_group(ps_ctx* ctx, int32_t l0, int32_t g, const std::vector<PlanEntry>& plan, const int32_t* d_ids);
int32_t note_layer_issued(ps_ctx* ctx, int64_t id, Req& r, int32_t layer, int32_t hi);
int32_t missing_of(const Req& r);

// copy-budget consumption and the attention batch (ps_step.cu)
std::vector<PlanEntry> make_plan(ps_ctx* ctx, int64_t copy_budget_bytes, const ps_copy_rule* rule);
int32_t prepare_batch(ps_ctx* ctx, const int64_t* reqs, int32_t B, const std::vector<char>& active,
                      const std::vector<char>& gated, bool want_lanes, int tail_mode);
int32_t launch_layer_attn(ps_ctx* ctx, int32_t layer, const void* q, void* out, float* lse, cudaEvent_t wait_event,
                          bool follows_own, int32_t* n_launched);

}  // namespace psrt
