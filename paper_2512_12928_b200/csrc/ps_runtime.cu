// Host runtime of the KV swap library: block pool, request states, host-image pool, copy streams,
// per-layer reload events, copy-budget consumption and the step loop.  See include/ps_kvswap.h for
// the contract of every entry point.
//
// Streams (Appendix B: a copy stream per direction, independent of the compute stream; one
// completion event per layer chunk):
//   compute  : the caller's stream; attention runs here.
//   s_lane   : attention of the requests whose reload lands in this step, layer by layer behind that
//              layer's reload event (tensor-core kernel; other kernels make the whole launch wait instead).
//   s_gather : gather kernels of swap-out.           s_d2h : staging -> pinned host copies.
//   s_h2d    : pinned host -> staging copies.        s_scatter : scatter kernels of swap-in.
// Each direction owns kSlots staging slots; two events per slot hand a slot back and forth between
// the kernel stream and the copy-engine stream, so the copy engine never waits for a kernel launch
// and a kernel never reads a slot the engine is still filling.
#include <algorithm>
#include <chrono>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <deque>
#include <map>
#include <string>
#include <thread>
#include <unordered_map>
#include <vector>

#include "ps_internal.h"
#include "ps_kvswap.h"

namespace {

constexpr int kSlots = 4;
constexpr int64_t kHostAlign = 4096;

std::string g_create_error = "";

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
    bool two_lanes = false, contended = false;
    int64_t kv_bytes_per_layer = 0;
};

}  // namespace

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
    std::vector<cudaEvent_t> ev_in;  // per layer
    cudaEvent_t e_mark = nullptr, e_mark2 = nullptr, e_fork = nullptr, e_join = nullptr;
    int32_t* status = nullptr;  // mapped pinned word written by kernels on a bad block id
    int32_t* d_status = nullptr;
    Tracker t_d2h, t_scatter, t_compute;
    Arena a_gather, a_meta, a_ids;
    std::vector<int32_t> ids_cache;  // ids of the last ps_copy_blocks upload and where they sit in a_ids
    size_t ids_cache_off = 0;
    std::vector<cudaEvent_t> ev_pool, ev_pool_timing;
    std::deque<std::pair<uint64_t, std::pair<int64_t, int64_t>>> img_release;  // in_ticket -> (off, bytes)
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

    // measurement
    int64_t launches = 0;
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

namespace {

// ---- events -------------------------------------------------------------------------------------

cudaError_t get_event(ps_ctx* ctx, bool timing, cudaEvent_t* out) {
    auto& pool = timing ? ctx->ev_pool_timing : ctx->ev_pool;
    if (!pool.empty()) {
        *out = pool.back();
        pool.pop_back();
        return cudaSuccess;
    }
    return cudaEventCreateWithFlags(out, timing ? cudaEventDefault : cudaEventDisableTiming);
}

int32_t tracker_mark(ps_ctx* ctx, Tracker& t, uint64_t* ticket) {
    *ticket = t.next++;
    if (ctx->bk) {
        t.done = *ticket;
        return PS_OK;
    }
    cudaEvent_t ev;
    CK(get_event(ctx, false, &ev));
    CK(cudaEventRecord(ev, t.s));
    t.pending.emplace_back(*ticket, ev);
    return PS_OK;
}

int32_t tracker_poll(ps_ctx* ctx, Tracker& t) {
    while (!t.pending.empty()) {
        cudaError_t e = cudaEventQuery(t.pending.front().second);
        if (e == cudaErrorNotReady) break;
        if (e != cudaSuccess) return ctx->fail_cuda(e, "cudaEventQuery");
        t.done = t.pending.front().first;
        ctx->ev_pool.push_back(t.pending.front().second);
        t.pending.pop_front();
    }
    return PS_OK;
}

// Waits until every ticket of the tracker is complete or the deadline passes.
int32_t tracker_drain(ps_ctx* ctx, Tracker& t, bool bounded, std::chrono::steady_clock::time_point deadline) {
    while (!t.pending.empty()) {
        if (!bounded) {
            CK(cudaEventSynchronize(t.pending.back().second));
        }
        int32_t rc = tracker_poll(ctx, t);
        if (rc != PS_OK) return rc;
        if (t.pending.empty()) break;
        if (bounded && std::chrono::steady_clock::now() > deadline) return ctx->fail(PS_ERR_TIMEOUT, "ps_sync timed out");
        std::this_thread::sleep_for(std::chrono::microseconds(50));
    }
    return PS_OK;
}

// ---- descriptor arenas ----------------------------------------------------------------------------

int32_t arena_init(ps_ctx* ctx, Arena& a, size_t chunk, int nchunks, cudaStream_t s) {
    a.chunk = (size_t)round_up((int64_t)chunk, 256);
    a.nchunks = nchunks;
    a.s = s;
    a.cur = 0;
    a.used = 0;
    CK(cudaHostAlloc((void**)&a.h, a.chunk * nchunks, cudaHostAllocMapped));
    CK(cudaHostGetDevicePointer((void**)&a.hd, a.h, 0));
    CK(cudaMalloc((void**)&a.d, a.chunk * nchunks));
    a.fence.resize(nchunks);
    a.fenced.assign(nchunks, 0);
    for (int i = 0; i < nchunks; ++i) CK(cudaEventCreateWithFlags(&a.fence[i], cudaEventDisableTiming));
    return PS_OK;
}

int32_t arena_next_chunk(ps_ctx* ctx, Arena& a, bool record_fence = true) {
    if (record_fence) {
        CK(cudaEventRecord(a.fence[a.cur], a.s));
        a.fenced[a.cur] = 1;
    }
    a.cur = (a.cur + 1) % a.nchunks;
    a.used = 0;
    if (a.fenced[a.cur]) {
        CK(cudaEventSynchronize(a.fence[a.cur]));  // uploads from this chunk were enqueued nchunks-1 chunks ago
        a.fenced[a.cur] = 0;
    }
    return PS_OK;
}

// Reserves `bytes` in the current chunk (moving on when it is full); *off is the byte offset in both buffers.
int32_t arena_alloc(ps_ctx* ctx, Arena& a, size_t bytes, size_t* off) {
    bytes = (size_t)round_up((int64_t)bytes, 256);
    if (bytes > a.chunk) return ctx->fail(PS_ERR_INVALID, "descriptor larger than an arena chunk");
    if (a.used + bytes > a.chunk) {
        int32_t rc = arena_next_chunk(ctx, a);
        if (rc != PS_OK) return rc;
    }
    *off = (size_t)a.cur * a.chunk + a.used;
    a.used += bytes;
    return PS_OK;
}

void arena_free(Arena& a) {
    if (a.h) cudaFreeHost(a.h);
    if (a.d) cudaFree(a.d);
    for (auto e : a.fence) cudaEventDestroy(e);
    a = Arena{};
}

// ---- profiling ------------------------------------------------------------------------------------

struct ProfScope {
    ps_ctx* ctx;
    int kind;
    cudaStream_t s;
    cudaEvent_t e0 = nullptr;
    bool on = false;
    int tag;
    ProfScope(ps_ctx* c, int k, cudaStream_t st, int64_t bytes, int tg = -1) : ctx(c), kind(k), s(st), tag(tg) {
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

void resolve_profile(ps_ctx* ctx) {
    size_t keep = 0;
    for (size_t i = 0; i < ctx->spans.size(); ++i) {
        ProfSpan& sp = ctx->spans[i];
        float ms = 0.f;
        if (cudaEventQuery(sp.e1) == cudaSuccess && cudaEventElapsedTime(&ms, sp.e0, sp.e1) == cudaSuccess) {
            ctx->prof_ms[sp.kind] += ms;
            if (ctx->tracing && ctx->trace_base) {
                float t0 = 0.f;
                if (cudaEventElapsedTime(&t0, ctx->trace_base, sp.e0) == cudaSuccess)
                    ctx->trace.push_back({sp.kind, sp.tag, t0 * 1e3f, (t0 + ms) * 1e3f});
            }
            ctx->ev_pool_timing.push_back(sp.e0);
            ctx->ev_pool_timing.push_back(sp.e1);
        } else {
            ctx->spans[keep++] = sp;
        }
    }
    ctx->spans.resize(keep);
    cudaGetLastError();
}

// ---- pool helpers -----------------------------------------------------------------------------------

inline int32_t blocks_for(const ps_ctx* ctx, int32_t n_tokens) {
    return (n_tokens + ctx->cfg.block_size - 1) / ctx->cfg.block_size;
}

void push_table(ps_ctx* ctx, std::vector<int32_t>& table) {
    for (int32_t id : table) ctx->free_stack.push_back(id);  // table order: the last entry ends on top
    table.clear();
    ctx->table_epoch++;
}

int32_t check_status_word(ps_ctx* ctx) {
    if (ctx->status && *(volatile int32_t*)ctx->status != 0) {
        const int v = *(volatile int32_t*)ctx->status;
        *(volatile int32_t*)ctx->status = 0;
        return ctx->fail(PS_ERR_BOUNDS, v == 2 ? "attention kernel met a block id outside the pool"
                                               : "copy kernel met a block id outside the pool");
    }
    return PS_OK;
}

int32_t do_poll(ps_ctx* ctx, int32_t* n_reaped) {
    int32_t reaped = 0;
    int32_t rc = tracker_poll(ctx, ctx->t_d2h);
    if (rc != PS_OK) return rc;
    while (!ctx->out_fifo.empty()) {
        Req& r = ctx->reqs[ctx->out_fifo.front()];
        if (r.out_ticket > ctx->t_d2h.done) break;  // offloads complete in issue order
        push_table(ctx, r.table);
        r.state = PS_REQ_HOST;
        ctx->out_fifo.pop_front();
        ++reaped;
    }
    rc = tracker_poll(ctx, ctx->t_scatter);
    if (rc != PS_OK) return rc;
    while (!ctx->img_release.empty() && ctx->img_release.front().first <= ctx->t_scatter.done) {
        ctx->hpool.release(ctx->img_release.front().second.first, ctx->img_release.front().second.second);
        ctx->img_release.pop_front();
    }
    size_t keep = 0;
    for (size_t i = 0; i < ctx->gated_reqs.size(); ++i) {
        auto it = ctx->reqs.find(ctx->gated_reqs[i]);
        if (it == ctx->reqs.end() || !it->second.gated) continue;
        if (it->second.in_ticket <= ctx->t_scatter.done)
            it->second.gated = false;
        else
            ctx->gated_reqs[keep++] = ctx->gated_reqs[i];
    }
    ctx->gated_reqs.resize(keep);
    rc = tracker_poll(ctx, ctx->t_compute);
    if (rc != PS_OK) return rc;
    if (n_reaped) *n_reaped = reaped;
    return check_status_word(ctx);
}

// ---- swap-in issue ------------------------------------------------------------------------------------

// Orders the scatter stream after everything already enqueued on the compute stream: a fresh block
// may have been released by a request whose last attention launch is still running.
int32_t order_scatter_after_compute(ps_ctx* ctx) {
    if (ctx->bk) return PS_OK;
    CK(cudaEventRecord(ctx->e_mark, ctx->compute));
    CK(cudaStreamWaitEvent(ctx->s_scatter, ctx->e_mark, 0));
    return PS_OK;
}

// Issues the reload of one layer for a list of (request, block range); records ev_in[layer].
int32_t issue_reload_layer(ps_ctx* ctx, int32_t layer, const std::vector<PlanEntry>& plan) {
    if (ctx->bk || plan.empty()) return PS_OK;
    const int64_t Bl = ctx->layer_block_bytes;
    const int64_t cap = ctx->slot_bytes / Bl;  // pairs per slot
    size_t i = 0;
    int32_t lo = plan[0].lo;
    std::vector<int32_t> ids;
    while (i < plan.size()) {
        const int slot = (int)(ctx->in_next++ % kSlots);
        char* sp = ctx->stage_in + (int64_t)slot * ctx->slot_bytes;
        if (ctx->in_used[slot]) CK(cudaStreamWaitEvent(ctx->s_h2d, ctx->e_scattered[slot], 0));
        int64_t used = 0;
        ids.clear();
        while (i < plan.size() && used < cap) {
            Req& r = ctx->reqs[plan[i].req];
            const int64_t take = std::min<int64_t>(plan[i].hi - lo, cap - used);
            // one contiguous host range per (segment, layer): a run of blocks is cut at segment borders
            for (int64_t j = lo, done = 0; done < take;) {
                const Req::Seg* sg = nullptr;
                for (const Req::Seg& c : r.segs)
                    if (j >= c.lo && j < c.hi) sg = &c;
                if (sg == nullptr) return ctx->fail(PS_ERR_STATE, "reload: block outside the host image");
                const int64_t piece = std::min<int64_t>(take - done, sg->hi - j);
                const char* src = ctx->host_pool + sg->off + ((int64_t)layer * (sg->hi - sg->lo) + (j - sg->lo)) * Bl;
                ProfScope prof(ctx, kProfH2D, ctx->s_h2d, piece * Bl, layer);
                CK(cudaMemcpyAsync(sp + (used + done) * Bl, src, (size_t)(piece * Bl), cudaMemcpyHostToDevice, ctx->s_h2d));
                j += piece;
                done += piece;
            }
            for (int64_t j = lo; j < lo + take; ++j) ids.push_back(r.table[(size_t)j]);
            used += take;
            lo += (int32_t)take;
            if (lo >= plan[i].hi) {
                ++i;
                if (i < plan.size()) lo = plan[i].lo;
            }
        }
        CK(cudaEventRecord(ctx->e_loaded[slot], ctx->s_h2d));
        CK(cudaStreamWaitEvent(ctx->s_scatter, ctx->e_loaded[slot], 0));
        for (size_t c0 = 0; c0 < ids.size(); c0 += ps::kMaxParamIds) {
            const int32_t n = (int32_t)std::min<size_t>(ps::kMaxParamIds, ids.size() - c0);
            ProfScope prof(ctx, kProfScatter, ctx->s_scatter, (int64_t)n * Bl, layer);
            CK(ps::launch_scatter_layer_ids(ctx->kpools[layer], ctx->vpools[layer], ids.data() + c0, n,
                                            sp + (int64_t)c0 * Bl, ctx->slab_vec, ctx->cfg.num_gpu_blocks,
                                            ctx->d_status, ctx->s_scatter));
            ctx->launches++;
        }
        CK(cudaEventRecord(ctx->e_scattered[slot], ctx->s_scatter));
        ctx->in_used[slot] = true;
    }
    CK(cudaEventRecord(ctx->ev_in[layer], ctx->s_scatter));
    return PS_OK;
}

// Book-keeping after blocks [.., hi) of `layer` have been issued for a request.
int32_t note_layer_issued(ps_ctx* ctx, int64_t id, Req& r, int32_t layer, int32_t hi) {
    r.layer_done[layer] = hi;
    const int32_t n = (int32_t)r.table.size();
    for (int32_t d : r.layer_done)
        if (d != n) return PS_OK;
    // every layer issued: the request is resident; attention over it stays gated on the reload events
    r.state = PS_REQ_RESIDENT;
    r.layer_done.clear();
    for (auto it = ctx->in_fifo.begin(); it != ctx->in_fifo.end(); ++it)
        if (*it == id) {
            ctx->in_fifo.erase(it);
            break;
        }
    int32_t rc = tracker_mark(ctx, ctx->t_scatter, &r.in_ticket);
    if (rc != PS_OK) return rc;
    for (const Req::Seg& sg : r.segs) {
        if (ctx->bk)
            ctx->hpool.release(sg.off, sg.bytes);
        else
            ctx->img_release.push_back({r.in_ticket, {sg.off, sg.bytes}});
    }
    r.segs.clear();
    r.host_issued = 0;
    if (!ctx->bk) {
        r.gated = true;
        ctx->gated_reqs.push_back(id);
    }
    ctx->table_epoch++;
    return PS_OK;
}

int32_t missing_of(const Req& r) {
    if (r.state != PS_REQ_SWAPPING_IN) return 0;
    int32_t mn = (int32_t)r.table.size();
    for (int32_t d : r.layer_done) mn = std::min(mn, d);
    return (int32_t)r.table.size() - mn;
}

// Copy-budget consumption (Alg. 1, ConsumeCopyBudget, reduced to the byte budget): FIFO, whole request if it
// fits, otherwise the residual.
std::vector<PlanEntry> make_plan(ps_ctx* ctx, int64_t copy_budget_bytes) {
    std::vector<PlanEntry> plan;
    const bool unlimited = copy_budget_bytes < 0;
    int64_t left = unlimited ? 0 : copy_budget_bytes / ctx->block_bytes;
    for (int64_t id : ctx->in_fifo) {
        Req& r = ctx->reqs[id];
        const int32_t miss = missing_of(r);
        if (miss == 0) continue;
        const int32_t lo = (int32_t)r.table.size() - miss;
        const int64_t take = unlimited ? miss : std::min<int64_t>(miss, left);
        if (take == 0) break;
        plan.push_back({id, lo, lo + (int32_t)take});
        if (!unlimited) {
            left -= take;
            if (left == 0) break;
        }
    }
    return plan;
}

// ---- attention batch ------------------------------------------------------------------------------------

int32_t choose_split(const ps_ctx* ctx, int64_t total_tokens) {
    if (ctx->cfg.kv_split_tokens > 0) return ctx->cfg.kv_split_tokens;
    const int64_t target_items = std::max<int64_t>(1, 4096 / ctx->cfg.num_kv_heads);
    int64_t split = (total_tokens + target_items - 1) / target_items;
    split = round_up(std::max<int64_t>(split, 1), 64);
    return (int32_t)std::min<int64_t>(std::max<int64_t>(split, 256), 1 << 20);
}

// Builds (or reuses) the device metadata for a decode batch.  Row b of the metadata is position b of
// the caller's request array (q / out rows are addressed by that position); rows with active[b] == 0
// get no work item.  gated[b] != 0 marks rows whose reload is still landing: their attention waits on
// the layer's reload event.  With want_lanes they get a work list of their own (lane 1), launched on
// the reload-lane stream behind the event, so that the launches of the other rows never wait.
int32_t prepare_batch(ps_ctx* ctx, const int64_t* reqs, int32_t B, const std::vector<char>& active,
                      const std::vector<char>& gated, bool want_lanes, bool contended) {
    BatchMeta& m = ctx->meta;
    // two work lists (lanes) only for the tensor-core kernel and only when some row is gated
    bool two_lanes = false;
    if (want_lanes && ctx->attn_kernel == PS_ATTN_MMA)
        for (int32_t b = 0; b < B; ++b) two_lanes |= active[b] && gated[b];
    if (m.valid && m.epoch == ctx->table_epoch && (int32_t)m.reqs.size() == B && m.two_lanes == two_lanes &&
        m.contended == contended &&
        std::equal(m.reqs.begin(), m.reqs.end(), reqs) && m.gated == gated && m.active == active)
        return PS_OK;

    int32_t stride = 1;
    int64_t total_tokens = 0;
    for (int32_t b = 0; b < B; ++b) {
        if (!active[b]) continue;
        const Req& r = ctx->reqs[reqs[b]];
        stride = std::max<int32_t>(stride, (int32_t)r.table.size());
        total_tokens += r.n_tokens;
    }
    std::vector<int32_t> row_first(B, 0), row_parts(B, 0), ctx_len(B, 0);
    std::vector<ps::AttnItem> items;
    std::vector<int32_t> cta_begin[2];
    int32_t parts = 0, n_ungated = 0, n_gated_rows = 0;
    bool any_multi = false, lane_multi[2] = {false, false};
    const bool mma = ctx->attn_kernel == PS_ATTN_MMA;
    const int32_t split = mma ? 0 : choose_split(ctx, total_tokens);
    for (int pass = 0; pass < (two_lanes ? 2 : 1); ++pass) {  // lane 0: rows that need no wait (or all rows); lane 1: gated rows
        if (!mma) {
            // SIMT kernel: one CTA per (item, KV head); items are fixed-size token ranges of a row
            for (int32_t b = 0; b < B; ++b) {
                if (!active[b] || (two_lanes && (gated[b] ? 1 : 0) != pass)) continue;
                const Req& r = ctx->reqs[reqs[b]];
                const int32_t n = std::max(1, (r.n_tokens + split - 1) / split);
                row_first[b] = parts;
                row_parts[b] = n;
                ctx_len[b] = r.n_tokens;
                any_multi |= n > 1;
                lane_multi[pass] |= n > 1;
                for (int32_t k = 0; k < n; ++k) {
                    ps::AttnItem it{};
                    it.b = b;
                    it.t_begin = k * split;
                    it.t_end = std::min(r.n_tokens, (k + 1) * split);
                    it.part = parts + k;
                    it.n_parts = n;
                    items.push_back(it);
                }
                parts += n;
                if (gated[b]) ++n_gated_rows;
            }
        } else {
            // Tensor-core kernel: the lane's 16-token tiles form one sequence, cut into equal static shares,
            // one per CTA: every CTA streams the same number of bytes whatever the context-length mix, and
            // only the rows cut by share borders need combining.  When reload traffic runs beside the step
            // (scatter kernels and the reload lane take SM time unevenly) the last 5 % of the tiles become
            // chunks that the CTAs take dynamically; without contention such a tail only costs (more parts
            // to combine, a last round of chunks that does not fill the machine): 172 against 189 us per
            // 1 GiB launch.  An item is the part of a row that falls into one share or chunk.
            constexpr int kTile = ps::kMmaTileTokens;
            constexpr int64_t kMinTilesPerCta = 8;
            constexpr int64_t kDynMinChunk = 16;
            constexpr int64_t kDynChunksPerCta = 6;
            int64_t total_tiles = 0;
            int32_t lane_rows = 0;
            for (int32_t b = 0; b < B; ++b)
                if (active[b] && !(two_lanes && (gated[b] ? 1 : 0) != pass)) {
                    total_tiles += (ctx->reqs[reqs[b]].n_tokens + kTile - 1) / kTile;
                    ++lane_rows;
                }
            int64_t n_cta = 0;
            if (lane_rows > 0)
                n_cta = std::min<int64_t>(std::max<int64_t>((total_tiles + kMinTilesPerCta - 1) / kMinTilesPerCta, 1),
                                          ctx->num_sms);
            int64_t dyn_tiles = 0, chunk = 0;
            if (contended && n_cta > 0 && total_tiles >= 32 * n_cta) {
                dyn_tiles = total_tiles * 5 / 100;
                chunk = std::max<int64_t>(kDynMinChunk, (dyn_tiles + kDynChunksPerCta * n_cta - 1) / (kDynChunksPerCta * n_cta));
            }
            const int64_t static_tiles = total_tiles - dyn_tiles;
            const int64_t per = n_cta > 0 ? std::max<int64_t>((static_tiles + n_cta - 1) / n_cta, 1) : 1;
            // walk the rows; `pos` is the position in the lane's tile sequence
            int64_t pos = 0, filled = 0;       // filled: tiles in the current share or chunk
            bool in_dyn = false;
            if (n_cta > 0) cta_begin[pass].push_back((int32_t)items.size());
            auto close_static = [&]() {        // pad the share list and mark where the dynamic chunks start
                while ((int64_t)cta_begin[pass].size() < n_cta + 1) cta_begin[pass].push_back((int32_t)items.size());
                in_dyn = true;
                filled = 0;
            };
            for (int32_t b = 0; b < B; ++b) {
                if (!active[b] || (two_lanes && (gated[b] ? 1 : 0) != pass)) continue;
                const Req& r = ctx->reqs[reqs[b]];
                const int64_t tiles_b = (r.n_tokens + kTile - 1) / kTile;
                const size_t first_item = items.size();
                ctx_len[b] = r.n_tokens;
                row_first[b] = parts;
                if (tiles_b == 0) {  // empty context: one item without tiles writes the zero row
                    ps::AttnItem it{};
                    it.b = b;
                    items.push_back(it);
                }
                for (int64_t lo = 0; lo < tiles_b;) {
                    if (!in_dyn && pos >= static_tiles) close_static();
                    int64_t room;
                    if (!in_dyn) {
                        if (filled == per && (int64_t)cta_begin[pass].size() < n_cta) {
                            cta_begin[pass].push_back((int32_t)items.size());
                            filled = 0;
                        }
                        room = std::min(per - filled, static_tiles - pos);
                    } else {
                        if (filled == chunk) filled = 0;
                        room = chunk - filled;
                    }
                    const int64_t take = std::min(tiles_b - lo, std::max<int64_t>(room, 1));
                    ps::AttnItem it{};
                    it.b = b;
                    it.t_begin = (int32_t)(lo * kTile);
                    it.t_end = (int32_t)std::min<int64_t>(r.n_tokens, (lo + take) * kTile);
                    items.push_back(it);
                    lo += take;
                    pos += take;
                    // a dynamic chunk never spans two rows: every item of the tail is its own chunk
                    filled = in_dyn ? chunk : filled + take;
                    if (in_dyn && take < chunk && lo < tiles_b) filled = chunk;
                }
                const int32_t n = (int32_t)(items.size() - first_item);
                for (size_t k = first_item; k < items.size(); ++k) {
                    items[k].part = parts + (int32_t)(k - first_item);
                    items[k].n_parts = n;
                }
                row_parts[b] = n;
                parts += n;
                any_multi |= n > 1;
                lane_multi[pass] |= n > 1;
                if (gated[b]) ++n_gated_rows;
            }
            if (n_cta > 0 && !in_dyn) close_static();
        }
        if (pass == 0) n_ungated = (int32_t)items.size();
    }
    if (parts > ctx->max_parts) return ctx->fail(PS_ERR_INVALID, "split-KV scratch too small for this batch");

    const size_t sz_tables = (size_t)round_up((int64_t)B * stride * 4, 256);
    const size_t sz_vec = (size_t)round_up((int64_t)B * 4, 256);
    const size_t sz_items = (size_t)round_up((int64_t)std::max<size_t>(items.size(), 1) * sizeof(ps::AttnItem), 256);
    const size_t sz_cta = (size_t)round_up((int64_t)(cta_begin[0].size() + cta_begin[1].size() + 2) * 4, 256);
    const size_t total = sz_tables + 4 * sz_vec + sz_items + sz_cta;
    if (total > ctx->a_meta.chunk) return ctx->fail(PS_ERR_INVALID, "decode batch metadata exceeds its buffer");
    // a fresh chunk: the chunk of the cached batch stays intact until this point
    int32_t rc = arena_next_chunk(ctx, ctx->a_meta, /*record_fence=*/false);
    if (rc != PS_OK) return rc;
    size_t off = 0;
    rc = arena_alloc(ctx, ctx->a_meta, total, &off);
    if (rc != PS_OK) return rc;
    char* h = ctx->a_meta.h + off;
    char* d = ctx->a_meta.d + off;
    int32_t* ht = (int32_t*)h;
    memset(ht, 0, sz_tables);
    for (int32_t b = 0; b < B; ++b) {
        if (!active[b]) continue;
        const Req& r = ctx->reqs[reqs[b]];
        if (!r.table.empty()) memcpy(ht + (size_t)b * stride, r.table.data(), r.table.size() * 4);
    }
    memcpy(h + sz_tables, ctx_len.data(), (size_t)B * 4);
    memcpy(h + sz_tables + sz_vec, row_first.data(), (size_t)B * 4);
    memcpy(h + sz_tables + 2 * sz_vec, row_parts.data(), (size_t)B * 4);
    {
        int32_t* lane = (int32_t*)(h + sz_tables + 3 * sz_vec);
        for (int32_t b = 0; b < B; ++b) lane[b] = two_lanes && gated[b] ? 1 : 0;
    }
    if (!items.empty()) memcpy(h + sz_tables + 4 * sz_vec, items.data(), items.size() * sizeof(ps::AttnItem));
    {
        int32_t* cb = (int32_t*)(h + sz_tables + 4 * sz_vec + sz_items);
        if (!cta_begin[0].empty()) memcpy(cb, cta_begin[0].data(), cta_begin[0].size() * 4);
        if (!cta_begin[1].empty()) memcpy(cb + cta_begin[0].size(), cta_begin[1].data(), cta_begin[1].size() * 4);
    }
    CK(ps::launch_upload(d, ctx->a_meta.hd + off, total, ctx->compute));
    ctx->launches++;
    // the pinned side of this chunk may be rewritten once this upload has run
    CK(cudaEventRecord(ctx->a_meta.fence[ctx->a_meta.cur], ctx->compute));
    ctx->a_meta.fenced[ctx->a_meta.cur] = 1;

    m.reqs.assign(reqs, reqs + B);
    m.gated = gated;
    m.active = active;
    m.two_lanes = two_lanes;
    m.contended = contended;
    m.epoch = ctx->table_epoch;
    m.valid = true;
    m.dev.block_tables = (const int32_t*)d;
    m.dev.ctx_len = (const int32_t*)(d + sz_tables);
    m.dev.row_first_part = (const int32_t*)(d + sz_tables + sz_vec);
    m.dev.row_parts = (const int32_t*)(d + sz_tables + 2 * sz_vec);
    m.dev.row_lane = (const int32_t*)(d + sz_tables + 3 * sz_vec);
    m.dev.items = (const ps::AttnItem*)(d + sz_tables + 4 * sz_vec);
    {
        const int32_t* cb = (const int32_t*)(d + sz_tables + 4 * sz_vec + sz_items);
        m.dev.cta_begin[0] = cb;
        m.dev.cta_begin[1] = cb + cta_begin[0].size();
        m.dev.n_cta[0] = cta_begin[0].empty() ? 0 : (int32_t)cta_begin[0].size() - 1;
        m.dev.n_cta[1] = cta_begin[1].empty() ? 0 : (int32_t)cta_begin[1].size() - 1;
        m.dev.lane_items[0] = 0;
        m.dev.lane_items[1] = n_ungated;
        m.dev.lane_items[2] = (int32_t)items.size();
    }
    m.dev.table_stride = stride;
    m.dev.batch = B;
    m.n_items = (int32_t)items.size();
    m.n_ungated_items = n_ungated;
    m.n_parts = parts;
    m.n_gated_rows = n_gated_rows;
    m.any_multi = any_multi;
    m.lane_multi[0] = lane_multi[0];
    m.lane_multi[1] = lane_multi[1];
    m.kv_bytes_per_layer = total_tokens * 2 * ctx->cfg.num_kv_heads * ctx->cfg.head_dim * 2;
    return PS_OK;
}

// Launches one layer of attention for the prepared batch.  wait_event: the layer's reload event when rows
// of the batch are still being reloaded (Appendix B: the computation synchronises on a layer chunk's event
// only before it executes that chunk); nullptr = no wait.  With two work lists the rows that need no wait
// run on the compute stream and the gated rows on the reload lane behind the event; with one list the
// whole launch waits.  follows_own: the previous kernel on the compute stream is this function's launch
// for the previous layer of the same step (independent data); full-grid tensor-core launches then overlap
// head to tail.
int32_t launch_layer_attn(ps_ctx* ctx, int32_t layer, const void* q, void* out, float* lse, cudaEvent_t wait_event,
                          bool follows_own, int32_t* n_launched) {
    BatchMeta& m = ctx->meta;
    if (m.n_items == 0) return PS_OK;
    ps::AttnShape sh{ctx->cfg.num_kv_heads, ctx->cfg.num_q_heads, ctx->cfg.head_dim, ctx->cfg.block_size,
                     ctx->cfg.num_gpu_blocks};
    const bool mma = ctx->attn_kernel == PS_ATTN_MMA;
    const ps::AttnTensorMaps* maps = ctx->tmaps.empty() ? nullptr : &ctx->tmaps[(size_t)layer];
    const bool lanes = m.two_lanes && m.n_items > m.n_ungated_items;
    if (wait_event && !lanes) CK(cudaStreamWaitEvent(ctx->compute, wait_event, 0));
    if (m.n_ungated_items > 0) {
        const bool overlap = follows_own && mma && !ctx->profile && m.dev.n_cta[0] == ctx->num_sms;
        const int set = ctx->scratch_set;
        ctx->scratch_set ^= 1;
        const int64_t bytes = m.kv_bytes_per_layer * m.n_ungated_items / m.n_items;
        {
            ProfScope prof(ctx, kProfAttn, ctx->compute, bytes, wait_event && !lanes ? 1000 + layer : layer);
            CK(ps::launch_decode_attn(ctx->attn_kernel, sh, ctx->kpools[layer], ctx->vpools[layer], maps, q, out, lse, m.dev,
                                      0, ctx->partials[set], ctx->d_sched[set], ctx->d_row_done[set], ctx->d_status,
                                      overlap, ctx->compute));
            ctx->launches++;
            ++*n_launched;
        }
        // the tensor-core kernel combines split rows itself; the CUDA-core kernel needs the merge pass
        if (!mma && m.any_multi) {
            ProfScope prof(ctx, kProfMerge, ctx->compute, 0, layer);
            CK(ps::launch_attn_merge(sh, out, lse, m.dev, ctx->partials[set], -1, ctx->compute));
            ctx->launches++;
            ++*n_launched;
        }
    }
    if (lanes) {
        if (wait_event) CK(cudaStreamWaitEvent(ctx->s_lane, wait_event, 0));
        const int64_t bytes = m.kv_bytes_per_layer * (m.n_items - m.n_ungated_items) / m.n_items;
        ProfScope prof(ctx, kProfAttn, ctx->s_lane, bytes, 1000 + layer);
        CK(ps::launch_decode_attn(ctx->attn_kernel, sh, ctx->kpools[layer], ctx->vpools[layer], maps, q, out, lse, m.dev, 1,
                                  ctx->partials[2], ctx->d_sched[2], ctx->d_row_done[2], ctx->d_status, false, ctx->s_lane));
        ctx->launches++;
        ++*n_launched;
    }
    return PS_OK;
}

void destroy_ctx(ps_ctx* ctx) {
    if (!ctx->bk) {
        for (cudaStream_t s : {ctx->s_gather, ctx->s_d2h, ctx->s_h2d, ctx->s_scatter, ctx->s_lane})
            if (s) cudaStreamDestroy(s);
        for (int i = 0; i < kSlots; ++i)
            for (cudaEvent_t e : {ctx->e_gathered[i], ctx->e_drained[i], ctx->e_loaded[i], ctx->e_scattered[i]})
                if (e) cudaEventDestroy(e);
        for (cudaEvent_t e : ctx->ev_in) cudaEventDestroy(e);
        for (cudaEvent_t e : {ctx->e_mark, ctx->e_mark2, ctx->e_fork, ctx->e_join, ctx->trace_base})
            if (e) cudaEventDestroy(e);
        for (auto& t : {&ctx->t_d2h, &ctx->t_scatter, &ctx->t_compute})
            for (auto& p : t->pending) cudaEventDestroy(p.second);
        for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
        for (cudaEvent_t e : ctx->ev_pool_timing) cudaEventDestroy(e);
        for (auto& sp : ctx->spans) {
            cudaEventDestroy(sp.e0);
            cudaEventDestroy(sp.e1);
        }
        arena_free(ctx->a_gather);
        arena_free(ctx->a_meta);
        arena_free(ctx->a_ids);
        if (ctx->stage_out) cudaFree(ctx->stage_out);
        if (ctx->stage_in) cudaFree(ctx->stage_in);
        if (ctx->d_kpools) cudaFree(ctx->d_kpools);
        if (ctx->d_vpools) cudaFree(ctx->d_vpools);
        for (int i = 0; i < 3; ++i) {
            if (ctx->partials[i]) cudaFree(ctx->partials[i]);
            if (ctx->d_sched[i]) cudaFree(ctx->d_sched[i]);
            if (ctx->d_row_done[i]) cudaFree(ctx->d_row_done[i]);
        }
        if (ctx->status) cudaFreeHost(ctx->status);
        if (ctx->own_host_pool && ctx->host_pool) cudaFreeHost(ctx->host_pool);
        cudaGetLastError();
    }
    delete ctx;
}

int32_t create_fail(ps_ctx* ctx, int32_t code) {
    g_create_error = ctx->err;
    destroy_ctx(ctx);
    return code;
}

}  // namespace

// =====================================================================================================
// C ABI
// =====================================================================================================

extern "C" {

const char* ps_last_error(const ps_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

int32_t ps_create(const ps_config* cfg, void* const* k_pools, void* const* v_pools, void* host_pool,
                  void* compute_stream, ps_ctx** out) {
    if (!cfg || !out) {
        g_create_error = "null argument";
        return PS_ERR_INVALID;
    }
    *out = nullptr;
    ps_ctx* ctx = new ps_ctx();
    ctx->cfg = *cfg;
    ctx->cfg.initial_free_order = nullptr;
    ctx->bk = (cfg->flags & PS_FLAG_BOOKKEEPING_ONLY) != 0;
    ctx->profile = (cfg->flags & PS_FLAG_PROFILE) != 0;
    const bool shape_ok = cfg->num_layers > 0 && cfg->num_kv_heads > 0 && cfg->num_q_heads > 0 &&
                          cfg->num_q_heads % cfg->num_kv_heads == 0 && cfg->block_size > 0 &&
                          cfg->num_gpu_blocks > 0 && cfg->max_blocks_per_req > 0 && cfg->max_batch >= 0 &&
                          cfg->host_pool_bytes >= 0 && cfg->head_dim > 0 && cfg->head_dim % 8 == 0;
    if (!shape_ok) {
        ctx->err = "invalid shape in ps_config";
        return create_fail(ctx, PS_ERR_INVALID);
    }
    ctx->G = cfg->num_q_heads / cfg->num_kv_heads;
    if (!ctx->bk) {
        const bool g_ok = ctx->G == 1 || ctx->G == 2 || ctx->G == 4 || ctx->G == 8;
        if (!g_ok || (cfg->head_dim != 64 && cfg->head_dim != 128)) {
            ctx->err = "unsupported attention shape: head_dim must be 64 or 128, Hq/Hkv in {1,2,4,8}";
            return create_fail(ctx, PS_ERR_INVALID);
        }
        if (!k_pools || !v_pools) {
            ctx->err = "k_pools / v_pools are required";
            return create_fail(ctx, PS_ERR_INVALID);
        }
    }
    ctx->slab_bytes = (int64_t)cfg->block_size * cfg->num_kv_heads * cfg->head_dim * 2;
    ctx->slab_vec = (int32_t)(ctx->slab_bytes / 16);
    ctx->layer_block_bytes = 2 * ctx->slab_bytes;
    ctx->block_bytes = ctx->layer_block_bytes * cfg->num_layers;

    // free stack: initial_free_order[0] is handed out first, so it sits on top (the vector's back)
    {
        const int32_t M = cfg->num_gpu_blocks;
        std::vector<char> seen((size_t)M, 0);
        ctx->free_stack.resize((size_t)M);
        for (int32_t i = 0; i < M; ++i) {
            const int32_t id = cfg->initial_free_order ? cfg->initial_free_order[i] : i;
            if (id < 0 || id >= M || seen[(size_t)id]) {
                ctx->err = "initial_free_order is not a permutation of 0..num_gpu_blocks-1";
                return create_fail(ctx, PS_ERR_INVALID);
            }
            seen[(size_t)id] = 1;
            ctx->free_stack[(size_t)(M - 1 - i)] = id;
        }
    }
    ctx->hpool.init(cfg->host_pool_bytes);
    if (ctx->bk) {
        *out = ctx;
        return PS_OK;
    }

#define CKC(call)                                                        \
    do {                                                                 \
        cudaError_t e__ = (call);                                        \
        if (e__ != cudaSuccess) {                                        \
            ctx->fail_cuda(e__, #call);                                  \
            return create_fail(ctx, PS_ERR_CUDA);                        \
        }                                                                \
    } while (0)
#define CKR(call)                                       \
    do {                                                \
        int32_t rc__ = (call);                          \
        if (rc__ != PS_OK) return create_fail(ctx, rc__); \
    } while (0)

    const int L = cfg->num_layers;
    ctx->kpools.assign(k_pools, k_pools + L);
    ctx->vpools.assign(v_pools, v_pools + L);
    ctx->compute = (cudaStream_t)compute_stream;
    CKC(ps::attn_init());
    CKC(cudaMalloc((void**)&ctx->d_kpools, sizeof(void*) * L));
    CKC(cudaMalloc((void**)&ctx->d_vpools, sizeof(void*) * L));
    CKC(cudaMemcpy(ctx->d_kpools, ctx->kpools.data(), sizeof(void*) * L, cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->d_vpools, ctx->vpools.data(), sizeof(void*) * L, cudaMemcpyHostToDevice));

    if (host_pool) {
        ctx->host_pool = (char*)host_pool;
    } else if (cfg->host_pool_bytes > 0) {
        cudaError_t e = cudaHostAlloc((void**)&ctx->host_pool, (size_t)cfg->host_pool_bytes, cudaHostAllocDefault);
        if (e != cudaSuccess) {
            ctx->fail_cuda(e, "cudaHostAlloc(host_pool_bytes)");
            cudaGetLastError();
            return create_fail(ctx, PS_ERR_HOST_NOMEM);
        }
        ctx->own_host_pool = true;
    }

    int prio_lo = 0, prio_hi = 0;
    CKC(cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi));
    // copy-side kernels are tiny and on the reload's critical path: let them overtake attention CTAs
    CKC(cudaStreamCreateWithPriority(&ctx->s_gather, cudaStreamNonBlocking, prio_hi));
    CKC(cudaStreamCreateWithPriority(&ctx->s_d2h, cudaStreamNonBlocking, prio_hi));
    CKC(cudaStreamCreateWithPriority(&ctx->s_h2d, cudaStreamNonBlocking, prio_hi));
    CKC(cudaStreamCreateWithPriority(&ctx->s_scatter, cudaStreamNonBlocking, prio_hi));
    // the reload lane: attention of the requests whose reload lands in this step, behind the per-layer events;
    // its few CTAs should get an SM as soon as one frees up
    CKC(cudaStreamCreateWithPriority(&ctx->s_lane, cudaStreamNonBlocking, prio_hi));
    ctx->t_d2h.s = ctx->s_d2h;
    ctx->t_scatter.s = ctx->s_scatter;
    ctx->t_compute.s = ctx->compute;

    int64_t staging = cfg->staging_bytes > 0 ? cfg->staging_bytes : (256LL << 20);
    ctx->slot_bytes = std::max<int64_t>(staging / kSlots / ctx->layer_block_bytes, 1) * ctx->layer_block_bytes;
    CKC(cudaMalloc((void**)&ctx->stage_out, (size_t)(ctx->slot_bytes * kSlots)));
    CKC(cudaMalloc((void**)&ctx->stage_in, (size_t)(ctx->slot_bytes * kSlots)));
    for (int i = 0; i < kSlots; ++i) {
        CKC(cudaEventCreateWithFlags(&ctx->e_gathered[i], cudaEventDisableTiming));
        CKC(cudaEventCreateWithFlags(&ctx->e_drained[i], cudaEventDisableTiming));
        CKC(cudaEventCreateWithFlags(&ctx->e_loaded[i], cudaEventDisableTiming));
        CKC(cudaEventCreateWithFlags(&ctx->e_scattered[i], cudaEventDisableTiming));
    }
    ctx->ev_in.resize((size_t)L);
    for (int l = 0; l < L; ++l) CKC(cudaEventCreateWithFlags(&ctx->ev_in[(size_t)l], cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&ctx->e_mark, cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&ctx->e_mark2, cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&ctx->e_fork, cudaEventDisableTiming));
    CKC(cudaEventCreateWithFlags(&ctx->e_join, cudaEventDisableTiming));
    CKC(cudaHostAlloc((void**)&ctx->status, 64, cudaHostAllocMapped));
    memset(ctx->status, 0, 64);
    CKC(cudaHostGetDevicePointer((void**)&ctx->d_status, ctx->status, 0));

    // descriptor arenas: a table per swap-out; one decode batch per chunk (scatter ids travel as
    // kernel parameters).  Uploads are done by a kernel reading the mapped pinned side, so the copy
    // engines carry bulk KV traffic only.
    const size_t desc_chunk = std::max<size_t>((size_t)cfg->max_blocks_per_req * 4 * 8, 1 << 20);
    CKR(arena_init(ctx, ctx->a_gather, desc_chunk, 4, ctx->s_gather));
    CKR(arena_init(ctx, ctx->a_ids, (size_t)cfg->num_gpu_blocks * 4, 4, ctx->compute));  // ps_copy_blocks

    // split-KV scratch
    ctx->attn_kernel = PS_ATTN_SIMT;
    {
        ps::AttnShape sh{cfg->num_kv_heads, cfg->num_q_heads, cfg->head_dim, cfg->block_size, cfg->num_gpu_blocks};
        if ((cfg->attn_kernel == PS_ATTN_MMA || cfg->attn_kernel == PS_ATTN_MMA_ROWS) && !ps::attn_mma_supported(sh)) {
            ctx->err = "the tensor-core attention kernel does not support this shape";
            return create_fail(ctx, PS_ERR_INVALID);
        }
        if (cfg->attn_kernel == PS_ATTN_MMA || cfg->attn_kernel == PS_ATTN_MMA_ROWS ||
            (cfg->attn_kernel == PS_ATTN_AUTO && ps::attn_mma_supported(sh)))
            ctx->attn_kernel = PS_ATTN_MMA;
        if (ctx->attn_kernel == PS_ATTN_MMA && cfg->attn_kernel != PS_ATTN_MMA_ROWS) {
            // tiles by tensor-map box copies when the driver accepts the maps, else row by row
            ctx->tmaps.resize((size_t)L);
            for (int l = 0; l < L; ++l)
                if (ps::attn_make_tensor_maps(sh, ctx->kpools[(size_t)l], ctx->vpools[(size_t)l], &ctx->tmaps[(size_t)l]) !=
                    cudaSuccess) {
                    ctx->tmaps.clear();
                    cudaGetLastError();
                    break;
                }
        }
        const int64_t max_batch = std::max(cfg->max_batch, 1);
        int64_t max_parts;
        if (cfg->kv_split_tokens > 0) {
            const int64_t max_ctx = (int64_t)cfg->max_blocks_per_req * cfg->block_size;
            max_parts = max_batch * ((max_ctx + cfg->kv_split_tokens - 1) / cfg->kv_split_tokens);
        } else {
            max_parts = std::max<int64_t>(1, 4096 / cfg->num_kv_heads) + max_batch;
        }
        {
            int dev = 0, sms = 0;
            CKC(cudaGetDevice(&dev));
            CKC(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
            ctx->num_sms = std::max(sms, 1);
        }
        // the tensor-core kernel cuts a lane into at most num_sms shares: rows + shares parts per lane
        // (static shares + at most ~6 dynamic chunks per CTA, plus one chunk boundary per row)
        max_parts = std::max<int64_t>(max_parts, 3 * max_batch + 2 * 8 * (int64_t)ctx->num_sms + 16);
        ctx->max_parts = (int32_t)std::min<int64_t>(max_parts, 1 << 22);
        const size_t done_bytes = (size_t)max_batch * cfg->num_kv_heads * sizeof(int32_t);
        for (int i = 0; i < 3; ++i) {
            CKC(cudaMalloc((void**)&ctx->partials[i], ps::attn_partial_bytes(sh, ctx->max_parts)));
            CKC(cudaMalloc((void**)&ctx->d_sched[i], 4 * sizeof(int32_t)));
            CKC(cudaMemset(ctx->d_sched[i], 0, 4 * sizeof(int32_t)));
            CKC(cudaMalloc((void**)&ctx->d_row_done[i], done_bytes));
            CKC(cudaMemset(ctx->d_row_done[i], 0, done_bytes));
        }
        const size_t meta_chunk = (size_t)max_batch * cfg->max_blocks_per_req * 4 + (size_t)max_batch * 16 +
                                  (size_t)ctx->max_parts * sizeof(ps::AttnItem) + (size_t)ctx->num_sms * 8 + 8192;
        CKR(arena_init(ctx, ctx->a_meta, meta_chunk, 3, ctx->compute));
    }
#undef CKC
#undef CKR
    *out = ctx;
    return PS_OK;
}

int32_t ps_destroy(ps_ctx* ctx) {
    if (!ctx) return PS_ERR_INVALID;
    if (!ctx->bk) {
        ps_sync(ctx, 10000);
    }
    destroy_ctx(ctx);
    return PS_OK;
}

int32_t ps_kv_alloc(ps_ctx* ctx, int64_t req, int32_t n_tokens_total) {
    if (!ctx || n_tokens_total < 0) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    int32_t have = 0;
    if (it != ctx->reqs.end()) {
        if (it->second.state != PS_REQ_RESIDENT) return ctx->fail(PS_ERR_STATE, "ps_kv_alloc: request is not resident");
        if (n_tokens_total < it->second.n_tokens) return ctx->fail(PS_ERR_INVALID, "ps_kv_alloc: cannot shrink");
        have = (int32_t)it->second.table.size();
    }
    const int32_t want = blocks_for(ctx, n_tokens_total);
    if (want > ctx->cfg.max_blocks_per_req) return ctx->fail(PS_ERR_INVALID, "ps_kv_alloc: exceeds max_blocks_per_req");
    const int32_t need = want - have;
    if (need > (int32_t)ctx->free_stack.size()) return ctx->fail(PS_ERR_NOMEM, "ps_kv_alloc: not enough free blocks");
    Req& r = ctx->reqs[req];
    for (int32_t i = 0; i < need; ++i) {
        r.table.push_back(ctx->free_stack.back());
        ctx->free_stack.pop_back();
    }
    r.n_tokens = n_tokens_total;
    ctx->table_epoch++;
    return PS_OK;
}

int32_t ps_kv_free(ps_ctx* ctx, int64_t req) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_kv_free: unknown request");
    Req& r = it->second;
    if (r.state == PS_REQ_SWAPPING_OUT || r.state == PS_REQ_SWAPPING_IN)
        return ctx->fail(PS_ERR_BUSY, "ps_kv_free: transfer in flight");
    if (r.state == PS_REQ_RESIDENT) {
        if (r.gated) {
            int32_t rc = do_poll(ctx, nullptr);
            if (rc != PS_OK) return rc;
            if (r.gated) return ctx->fail(PS_ERR_BUSY, "ps_kv_free: reload copies still in flight");
        }
        if (!r.segs.empty()) {  // proactive copies: their transfers must have ended before the image goes
            int32_t rc = do_poll(ctx, nullptr);
            if (rc != PS_OK) return rc;
            if (r.segs.back().ticket > ctx->t_d2h.done)
                return ctx->fail(PS_ERR_BUSY, "ps_kv_free: proactive offload still in flight");
        }
        push_table(ctx, r.table);
    }
    for (const Req::Seg& sg : r.segs) ctx->hpool.release(sg.off, sg.bytes);
    ctx->reqs.erase(it);
    ctx->table_epoch++;
    return PS_OK;
}

int32_t ps_block_table(ps_ctx* ctx, int64_t req, int32_t* out_ids, int32_t cap, int32_t* n_blocks, int32_t* state,
                       int32_t* n_tokens) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_block_table: unknown request");
    const Req& r = it->second;
    if (n_blocks) *n_blocks = (int32_t)r.table.size();
    if (state) *state = r.state;
    if (n_tokens) *n_tokens = r.n_tokens;
    if (out_ids) {
        const int32_t n = std::min<int32_t>(cap, (int32_t)r.table.size());
        if (n > 0) memcpy(out_ids, r.table.data(), (size_t)n * 4);
    }
    return PS_OK;
}

int32_t ps_num_free_blocks(ps_ctx* ctx, int32_t* out) {
    if (!ctx || !out) return PS_ERR_INVALID;
    *out = (int32_t)ctx->free_stack.size();
    return PS_OK;
}

// Starts the offload of logical blocks [lo, hi) of a request as a new image segment: gather through the
// table into staging slots, slot by slot to the host.  Ordered after everything already enqueued on the
// compute stream (and after the scatters of a reload that is still landing).
static int32_t offload_segment(ps_ctx* ctx, Req& r, int32_t lo, int32_t hi) {
    const int64_t n_blk = hi - lo;
    const int64_t bytes = n_blk * ctx->block_bytes;
    int64_t off = ctx->hpool.alloc(bytes);
    if (off < 0) {  // images of reloads that have landed since the last poll may still be held
        int32_t rc = do_poll(ctx, nullptr);
        if (rc != PS_OK) return rc;
        off = ctx->hpool.alloc(bytes);
    }
    if (off < 0) return ctx->fail(PS_ERR_HOST_NOMEM, "host pool cannot hold the image");

    if (!ctx->bk && n_blk > 0) {
        cudaError_t e = cudaEventRecord(ctx->e_mark2, ctx->compute);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_gather, ctx->e_mark2, 0);
        if (e == cudaSuccess && r.gated) {
            e = cudaEventRecord(ctx->e_mark2, ctx->s_scatter);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_gather, ctx->e_mark2, 0);
        }
        size_t toff = 0;
        int32_t rc = e == cudaSuccess ? arena_alloc(ctx, ctx->a_gather, (size_t)n_blk * 4, &toff) : PS_ERR_CUDA;
        if (e != cudaSuccess) ctx->fail_cuda(e, "ordering the gather stream");
        if (rc != PS_OK) {
            ctx->hpool.release(off, bytes);
            return rc;
        }
        memcpy(ctx->a_gather.h + toff, r.table.data() + lo, (size_t)n_blk * 4);
        auto bail = [&](cudaError_t ce, const char* what) {
            ctx->hpool.release(off, bytes);
            return ctx->fail_cuda(ce, what);
        };
        e = ps::launch_upload(ctx->a_gather.d + toff, ctx->a_gather.hd + toff, (size_t)round_up(n_blk * 4, 16),
                              ctx->s_gather);
        ctx->launches++;
        if (e != cudaSuccess) return bail(e, "table upload");
        const int64_t total_slabs = 2 * n_blk * ctx->cfg.num_layers;
        const int64_t slot_slabs = ctx->slot_bytes / ctx->slab_bytes;
        for (int64_t s0 = 0; s0 < total_slabs; s0 += slot_slabs) {
            const int64_t cnt = std::min(slot_slabs, total_slabs - s0);
            const int slot = (int)(ctx->out_next++ % kSlots);
            char* sp = ctx->stage_out + (int64_t)slot * ctx->slot_bytes;
            if (ctx->out_used[slot]) {
                e = cudaStreamWaitEvent(ctx->s_gather, ctx->e_drained[slot], 0);
                if (e != cudaSuccess) return bail(e, "slot wait");
            }
            {
                ProfScope prof(ctx, kProfGather, ctx->s_gather, cnt * ctx->slab_bytes);
                e = ps::launch_gather_image((const void* const*)ctx->d_kpools, (const void* const*)ctx->d_vpools,
                                            (const int32_t*)(ctx->a_gather.d + toff), (int32_t)n_blk, s0, cnt, sp,
                                            ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status, ctx->s_gather);
                ctx->launches++;
            }
            if (e == cudaSuccess) e = cudaEventRecord(ctx->e_gathered[slot], ctx->s_gather);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_d2h, ctx->e_gathered[slot], 0);
            if (e != cudaSuccess) return bail(e, "gather launch");
            {
                ProfScope prof(ctx, kProfD2H, ctx->s_d2h, cnt * ctx->slab_bytes);
                e = cudaMemcpyAsync(ctx->host_pool + off + s0 * ctx->slab_bytes, sp, (size_t)(cnt * ctx->slab_bytes),
                                    cudaMemcpyDeviceToHost, ctx->s_d2h);
            }
            if (e == cudaSuccess) e = cudaEventRecord(ctx->e_drained[slot], ctx->s_d2h);
            if (e != cudaSuccess) return bail(e, "device-to-host copy");
            ctx->out_used[slot] = true;
        }
    }
    Req::Seg sg{lo, hi, off, bytes, 0};
    int32_t rc = tracker_mark(ctx, ctx->t_d2h, &sg.ticket);
    if (rc != PS_OK) return rc;
    r.segs.push_back(sg);
    r.host_issued = hi;
    return PS_OK;
}

int32_t ps_swap_out(ps_ctx* ctx, int64_t req) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_swap_out: unknown request");
    Req& r = it->second;
    if (r.state != PS_REQ_RESIDENT) return ctx->fail(PS_ERR_STATE, "ps_swap_out: request is not resident");
    const int32_t n_blk = (int32_t)r.table.size();
    // what proactive offloading has not covered yet (everything, without it) goes out now
    if (r.host_issued < n_blk || r.segs.empty()) {
        int32_t rc = offload_segment(ctx, r, r.host_issued, n_blk);
        if (rc != PS_OK) return rc;
    }
    r.out_ticket = r.segs.back().ticket;  // copies complete in issue order
    r.state = PS_REQ_SWAPPING_OUT;
    ctx->out_fifo.push_back(req);
    ctx->table_epoch++;
    return PS_OK;
}

int32_t ps_offload_progress(ps_ctx* ctx, int64_t req, int32_t n_off, int32_t* issued_blocks) {
    if (!ctx) return PS_ERR_INVALID;
    if (issued_blocks) *issued_blocks = 0;
    if (n_off <= 0) return ctx->fail(PS_ERR_INVALID, "ps_offload_progress: n_off must be positive");
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_offload_progress: unknown request");
    Req& r = it->second;
    if (r.state != PS_REQ_RESIDENT) return ctx->fail(PS_ERR_STATE, "ps_offload_progress: request is not resident");
    const int32_t full = r.n_tokens / ctx->cfg.block_size;  // blocks that will not change any more
    const int32_t groups = (full - r.host_issued) / n_off;
    if (groups <= 0) return PS_OK;
    const int32_t lo = r.host_issued, hi = lo + groups * n_off;
    int32_t rc = offload_segment(ctx, r, lo, hi);
    if (rc != PS_OK) return rc;
    if (issued_blocks) *issued_blocks = hi - lo;
    return PS_OK;
}

int32_t ps_host_blocks(ps_ctx* ctx, int64_t req, int32_t* issued, int32_t* on_host) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_host_blocks: unknown request");
    const Req& r = it->second;
    int32_t done = 0;
    for (const Req::Seg& sg : r.segs)
        if (sg.ticket <= ctx->t_d2h.done) done = sg.hi;
    if (issued) *issued = r.host_issued;
    if (on_host) *on_host = done;
    return PS_OK;
}

int32_t ps_host_image(ps_ctx* ctx, int64_t req, void** ptr, int64_t* bytes) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_host_image: unknown request");
    const Req& r = it->second;
    if (r.segs.empty()) return ctx->fail(PS_ERR_STATE, "ps_host_image: request has no host image");
    if (r.segs.size() != 1)
        return ctx->fail(PS_ERR_STATE, "ps_host_image: the image has several segments, use ps_host_segment");
    if (ptr) *ptr = ctx->host_pool ? (void*)(ctx->host_pool + r.segs[0].off) : nullptr;
    if (bytes) *bytes = r.segs[0].bytes;
    return PS_OK;
}

int32_t ps_host_segment(ps_ctx* ctx, int64_t req, int32_t index, void** ptr, int64_t* bytes, int32_t* blk_lo,
                        int32_t* blk_hi, int32_t* n_segments) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_host_segment: unknown request");
    const Req& r = it->second;
    if (n_segments) *n_segments = (int32_t)r.segs.size();
    if (index < 0 || index >= (int32_t)r.segs.size()) {
        if (n_segments && index == -1) return PS_OK;  // count only
        return ctx->fail(PS_ERR_INVALID, "ps_host_segment: no such segment");
    }
    const Req::Seg& sg = r.segs[(size_t)index];
    if (ptr) *ptr = ctx->host_pool ? (void*)(ctx->host_pool + sg.off) : nullptr;
    if (bytes) *bytes = sg.bytes;
    if (blk_lo) *blk_lo = sg.lo;
    if (blk_hi) *blk_hi = sg.hi;
    return PS_OK;
}

int32_t ps_swap_in_begin(ps_ctx* ctx, int64_t req) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_swap_in_begin: unknown request");
    Req& r = it->second;
    if (r.state != PS_REQ_HOST) return ctx->fail(PS_ERR_STATE, "ps_swap_in_begin: request is not on host");
    const int32_t n = blocks_for(ctx, r.n_tokens);
    if (n > (int32_t)ctx->free_stack.size()) return ctx->fail(PS_ERR_NOMEM, "ps_swap_in_begin: not enough free blocks");
    r.table.clear();
    for (int32_t i = 0; i < n; ++i) {
        r.table.push_back(ctx->free_stack.back());
        ctx->free_stack.pop_back();
    }
    r.layer_done.assign((size_t)ctx->cfg.num_layers, 0);
    r.state = PS_REQ_SWAPPING_IN;
    ctx->in_fifo.push_back(req);
    ctx->table_epoch++;
    if (n == 0) {  // nothing to copy: resident at once
        for (int32_t l = 0; l < ctx->cfg.num_layers; ++l) {
            int32_t rc = note_layer_issued(ctx, req, r, l, 0);
            if (rc != PS_OK) return rc;
            if (r.state == PS_REQ_RESIDENT) break;
        }
    }
    return PS_OK;
}

int32_t ps_swap_in_cancel(ps_ctx* ctx, int64_t req) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_swap_in_cancel: unknown request");
    Req& r = it->second;
    if (r.state != PS_REQ_SWAPPING_IN) return ctx->fail(PS_ERR_STATE, "ps_swap_in_cancel: request is not being reloaded");
    for (int32_t d : r.layer_done)
        if (d != 0) return ctx->fail(PS_ERR_BUSY, "ps_swap_in_cancel: blocks already issued");
    push_table(ctx, r.table);
    r.layer_done.clear();
    r.state = PS_REQ_HOST;
    for (auto f = ctx->in_fifo.begin(); f != ctx->in_fifo.end(); ++f)
        if (*f == req) {
            ctx->in_fifo.erase(f);
            break;
        }
    return PS_OK;
}

int32_t ps_swap_in_layer(ps_ctx* ctx, int64_t req, int32_t layer, int32_t blk_lo, int32_t blk_hi) {
    if (!ctx) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_swap_in_layer: unknown request");
    Req& r = it->second;
    if (r.state != PS_REQ_SWAPPING_IN) return ctx->fail(PS_ERR_STATE, "ps_swap_in_layer: request is not being reloaded");
    const int32_t n = (int32_t)r.table.size();
    if (layer < 0 || layer >= ctx->cfg.num_layers || blk_lo < 0 || blk_lo > blk_hi || blk_hi > n ||
        blk_lo != r.layer_done[(size_t)layer])
        return ctx->fail(PS_ERR_INVALID, "ps_swap_in_layer: range must extend the layer's issued prefix");
    if (blk_hi > blk_lo) {
        int32_t rc = order_scatter_after_compute(ctx);
        if (rc != PS_OK) return rc;
        rc = issue_reload_layer(ctx, layer, {{req, blk_lo, blk_hi}});
        if (rc != PS_OK) return rc;
    }
    return note_layer_issued(ctx, req, r, layer, blk_hi);
}

int32_t ps_missing_blocks(ps_ctx* ctx, int64_t req, int32_t* out) {
    if (!ctx || !out) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_missing_blocks: unknown request");
    *out = missing_of(it->second);
    return PS_OK;
}

int32_t ps_decode_attn(ps_ctx* ctx, int32_t layer, const void* q, void* out, float* lse, const int64_t* reqs,
                       int32_t batch) {
    if (!ctx) return PS_ERR_INVALID;
    if (ctx->bk) return ctx->fail(PS_ERR_INVALID, "ps_decode_attn: context holds no device (bookkeeping only)");
    if (layer < 0 || layer >= ctx->cfg.num_layers || batch < 0 || batch > ctx->cfg.max_batch ||
        (batch > 0 && (!q || !out || !reqs)))
        return ctx->fail(PS_ERR_INVALID, "ps_decode_attn: bad argument");
    if (batch == 0) return PS_OK;
    bool any_gated = false;
    for (int32_t b = 0; b < batch; ++b) {
        auto it = ctx->reqs.find(reqs[b]);
        if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_decode_attn: unknown request");
        if (it->second.state != PS_REQ_RESIDENT) return ctx->fail(PS_ERR_STATE, "ps_decode_attn: request is not resident");
        any_gated |= it->second.gated;
    }
    if (any_gated) {
        int32_t rc = do_poll(ctx, nullptr);  // the copies may have landed since
        if (rc != PS_OK) return rc;
    }
    std::vector<char> active((size_t)batch, 1), gated((size_t)batch, 0);
    for (int32_t b = 0; b < batch; ++b) gated[(size_t)b] = ctx->reqs[reqs[b]].gated ? 1 : 0;
    int32_t rc = prepare_batch(ctx, reqs, batch, active, gated, /*want_lanes=*/false, /*contended=*/false);
    if (rc != PS_OK) return rc;
    int32_t launched = 0;
    return launch_layer_attn(ctx, layer, q, out, lse, ctx->meta.n_gated_rows ? ctx->ev_in[(size_t)layer] : nullptr,
                             /*follows_own=*/false, &launched);
}

int32_t ps_step(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs, int32_t batch,
                int64_t copy_budget_bytes, int32_t* decoded_mask, ps_step_stats* stats) {
    if (!ctx) return PS_ERR_INVALID;
    if (batch < 0 || (batch > 0 && !reqs)) return ctx->fail(PS_ERR_INVALID, "ps_step: bad batch");
    const bool want_attn = q_all_layers != nullptr || out_all_layers != nullptr;
    if (want_attn && (ctx->bk || !q_all_layers || !out_all_layers || batch > ctx->cfg.max_batch))
        return ctx->fail(PS_ERR_INVALID, "ps_step: attention needs q and out on a device context, batch <= max_batch");
    ps_step_stats st{};
    int32_t reaped = 0;
    int32_t rc = do_poll(ctx, &reaped);
    if (rc != PS_OK) return rc;
    st.swapouts_reaped = reaped;

    // 1. the copy budget is consumed over the reload queue
    const std::vector<PlanEntry> plan = make_plan(ctx, copy_budget_bytes);
    std::vector<char> completes(plan.size(), 0);
    for (size_t i = 0; i < plan.size(); ++i) {
        st.blocks_copied += plan[i].hi - plan[i].lo;
        completes[i] = plan[i].hi == (int32_t)ctx->reqs[plan[i].req].table.size();
    }
    st.h2d_bytes = st.blocks_copied * ctx->block_bytes;
    const int L = ctx->cfg.num_layers;
    const int64_t launches_before = ctx->launches;

    // 2. the decode set: resident now, or made complete by this step's reload (those wait on events)
    std::vector<char> active((size_t)batch, 0), gated((size_t)batch, 0);
    for (int32_t b = 0; b < batch; ++b) {
        auto it = ctx->reqs.find(reqs[b]);
        if (it == ctx->reqs.end()) {
            if (decoded_mask) decoded_mask[b] = 0;
            continue;
        }
        if (it->second.state == PS_REQ_RESIDENT) {
            active[(size_t)b] = 1;
            gated[(size_t)b] = it->second.gated ? 1 : 0;
        } else if (it->second.state == PS_REQ_SWAPPING_IN) {
            for (size_t i = 0; i < plan.size(); ++i)
                if (plan[i].req == reqs[b] && completes[i]) active[(size_t)b] = gated[(size_t)b] = 1;
        }
        if (decoded_mask) decoded_mask[b] = active[(size_t)b];
        st.decoded += active[(size_t)b];
    }
    const bool attn = want_attn && st.decoded > 0;
    if (attn) {
        rc = prepare_batch(ctx, reqs, batch, active, gated, (ctx->cfg.flags & PS_FLAG_SYNC_RELOAD) == 0,
                           /*contended=*/!plan.empty() && (ctx->cfg.flags & PS_FLAG_SYNC_RELOAD) == 0);
        if (rc != PS_OK) return rc;
        st.gated = ctx->meta.n_gated_rows;
    }

    // 3. per layer: reload chunk on the copy streams, then that layer's attention on the compute stream
    if (!plan.empty()) {
        rc = order_scatter_after_compute(ctx);
        if (rc != PS_OK) return rc;
    }
    const bool sync_reload = (ctx->cfg.flags & PS_FLAG_SYNC_RELOAD) != 0 || !attn;
    if (sync_reload)
        for (int l = 0; l < L; ++l) {
            rc = issue_reload_layer(ctx, l, plan);
            if (rc != PS_OK) return rc;
        }
    if (attn) {
        const int64_t layer_bytes = (int64_t)batch * ctx->cfg.num_q_heads * ctx->cfg.head_dim * 2;
        const bool any_gated = ctx->meta.n_gated_rows > 0;
        const bool lanes = ctx->meta.two_lanes;
        if (lanes) {  // the reload lane starts where the compute stream stands now (metadata uploaded)
            CK(cudaEventRecord(ctx->e_fork, ctx->compute));
            CK(cudaStreamWaitEvent(ctx->s_lane, ctx->e_fork, 0));
        }
        for (int l = 0; l < L; ++l) {
            if (!sync_reload) {
                rc = issue_reload_layer(ctx, l, plan);
                if (rc != PS_OK) return rc;
            }
            cudaEvent_t wait = nullptr;
            if (any_gated) {
                if (!sync_reload)
                    wait = ctx->ev_in[(size_t)l];
                else if (l == 0)
                    wait = ctx->ev_in[(size_t)L - 1];  // the whole reload, once, before the first layer
            }
            int32_t launched = 0;
            rc = launch_layer_attn(ctx, l, (const char*)q_all_layers + l * layer_bytes,
                                   (char*)out_all_layers + l * layer_bytes, nullptr, wait, /*follows_own=*/l > 0, &launched);
            if (rc != PS_OK) return rc;
        }
        if (lanes) {  // the step is complete on the compute stream only when the reload lane is
            CK(cudaEventRecord(ctx->e_join, ctx->s_lane));
            CK(cudaStreamWaitEvent(ctx->compute, ctx->e_join, 0));
        }
    }

    // 4. request states follow what was issued
    for (size_t i = 0; i < plan.size(); ++i) {
        Req& r = ctx->reqs[plan[i].req];
        for (int l = 0; l < L; ++l) {
            rc = note_layer_issued(ctx, plan[i].req, r, l, plan[i].hi);
            if (rc != PS_OK) return rc;
            if (r.state == PS_REQ_RESIDENT) break;
        }
        if (completes[i]) st.reloads_completed++;
    }
    if (attn && ctx->meta.n_gated_rows > 0) {
        // the compute stream is now ordered after every layer's reload event: later launches over
        // these requests need no wait
        for (int32_t b = 0; b < batch; ++b)
            if (active[(size_t)b] && gated[(size_t)b]) {
                auto it = ctx->reqs.find(reqs[b]);
                if (it != ctx->reqs.end()) it->second.gated = false;
            }
    }
    st.kernel_launches = (int32_t)(ctx->launches - launches_before);
    if (stats) *stats = st;
    return PS_OK;
}

int32_t ps_copy_budget(ps_ctx* ctx, const int64_t* reqs, int32_t batch, const ps_budget_model* model,
                       int64_t* budget_blocks, int64_t* budget_bytes, int32_t* which_case) {
    if (!ctx) return PS_ERR_INVALID;
    if (!model || !budget_blocks || batch < 0 || (batch > 0 && !reqs))
        return ctx->fail(PS_ERR_INVALID, "ps_copy_budget: null argument");
    const double a_d = model->a_d_us_per_token, b_d = model->b_d_us, t_c = model->t_c_us;
    const double t_block = model->t_block_us, t_budget = model->t_budget_us;
    if (!(t_block > 0.0) || a_d < 0.0 || b_d < 0.0 || t_c < 0.0 || t_budget < 0.0)
        return ctx->fail(PS_ERR_INVALID, "ps_copy_budget: t_block must be positive, the other terms non-negative");
    // the step's requests: resident ones decode whatever is copied; queued reloads decode once complete
    std::unordered_map<int64_t, char> in_batch;
    double t_resident = t_c, t_all = t_c;
    for (int32_t b = 0; b < batch; ++b) {
        auto it = ctx->reqs.find(reqs[b]);
        if (it == ctx->reqs.end()) continue;
        const Req& r = it->second;
        if (r.state != PS_REQ_RESIDENT && r.state != PS_REQ_SWAPPING_IN) continue;
        if (in_batch.count(reqs[b])) continue;
        in_batch[reqs[b]] = 1;
        const double t = a_d * (double)r.n_tokens + b_d;
        t_all += t;
        if (r.state == PS_REQ_RESIDENT) t_resident += t;
    }
    // the reload queue in order: missing blocks and what the request adds to the step once complete
    std::vector<int64_t> cum_miss;
    std::vector<double> cum_time;
    int64_t missing = 0;
    double t_added = 0.0;
    for (int64_t id : ctx->in_fifo) {
        const Req& r = ctx->reqs[id];
        const int32_t miss = missing_of(r);
        if (miss == 0) continue;
        missing += miss;
        if (in_batch.count(id)) t_added += a_d * (double)r.n_tokens + b_d;
        cum_miss.push_back(missing);
        cum_time.push_back(t_added);
    }
    const double t_fwd_min = t_all;
    const double t_trans_max = (double)missing * t_block;
    int64_t B = 0;
    int32_t wc = 0;
    if (t_fwd_min > t_budget) {
        wc = 1;
        B = (int64_t)std::floor(t_budget / t_block);
    } else if (t_fwd_min > t_trans_max) {
        wc = 21;
        B = missing;
    } else {
        wc = 22;
        if (!(t_block > a_d * (double)ctx->cfg.block_size))
            return ctx->fail(PS_ERR_INVALID, "ps_copy_budget: the search needs t_block > a_d * block_size");
        auto step_time_after = [&](int64_t blocks) {  // requests whose last missing block is among the first `blocks`
            double t = t_resident;
            for (size_t i = 0; i < cum_miss.size() && cum_miss[i] <= blocks; ++i) t = t_resident + cum_time[i];
            return t;
        };
        int64_t lo = 0, hi = missing;  // lo is feasible (0 blocks take no time)
        while (lo < hi) {
            const int64_t mid = lo + (hi - lo + 1) / 2;
            if ((double)mid * t_block <= step_time_after(mid))
                lo = mid;
            else
                hi = mid - 1;
        }
        B = lo;
    }
    *budget_blocks = B;
    if (budget_bytes) *budget_bytes = B * ctx->block_bytes;
    if (which_case) *which_case = wc;
    return PS_OK;
}

int32_t ps_select_victims(ps_ctx* ctx, const int64_t* queue, int32_t n, const double* waited_us, double tau_us,
                          double near_frac, int32_t blocks_needed, int64_t* victims, int32_t cap, int32_t* n_victims,
                          int32_t* blocks_freed) {
    if (!ctx) return PS_ERR_INVALID;
    if (n < 0 || (n > 0 && (!queue || !waited_us)) || cap < 0 || (cap > 0 && !victims) || !n_victims ||
        !(near_frac > 0.0 && near_frac <= 1.0) || tau_us < 0.0 || blocks_needed < 0)
        return ctx->fail(PS_ERR_INVALID, "ps_select_victims: bad argument");
    int32_t count = 0, freed = 0;
    for (int32_t i = n - 1; i >= 0 && freed < blocks_needed && count < cap; --i) {
        auto it = ctx->reqs.find(queue[i]);
        if (it == ctx->reqs.end()) continue;
        const Req& r = it->second;
        if (r.state != PS_REQ_RESIDENT || r.table.empty()) continue;
        if (waited_us[i] >= near_frac * tau_us) continue;  // close to starving: about to be promoted to the head
        bool dup = false;
        for (int32_t k = 0; k < count; ++k) dup |= victims[k] == queue[i];
        if (dup) continue;
        victims[count++] = queue[i];
        freed += (int32_t)r.table.size();
    }
    *n_victims = count;
    if (blocks_freed) *blocks_freed = freed;
    return PS_OK;
}

int32_t ps_copy_condition(int32_t l_comp, int32_t l_comp_max, int32_t b_miss, int32_t b_rem, int32_t s_blk,
                          double beta, int32_t* allowed) {
    if (!allowed || l_comp < 0 || l_comp_max < 0 || b_miss < 0 || b_rem < 0 || s_blk <= 0 || !(beta > 1.0))
        return PS_ERR_INVALID;
    if (b_rem >= b_miss)
        *allowed = 1;
    else if (l_comp >= l_comp_max)
        *allowed = 1;
    else
        *allowed = (double)l_comp / ((double)(b_miss - b_rem) * (double)s_blk) > beta ? 1 : 0;
    return PS_OK;
}

int32_t ps_poll(ps_ctx* ctx, int32_t* n_reaped) {
    if (!ctx) return PS_ERR_INVALID;
    return do_poll(ctx, n_reaped);
}

int32_t ps_sync(ps_ctx* ctx, int32_t timeout_ms) {
    if (!ctx) return PS_ERR_INVALID;
    if (!ctx->bk) {
        uint64_t t;
        int32_t rc = tracker_mark(ctx, ctx->t_d2h, &t);
        if (rc == PS_OK) rc = tracker_mark(ctx, ctx->t_scatter, &t);
        if (rc == PS_OK) rc = tracker_mark(ctx, ctx->t_compute, &t);
        if (rc != PS_OK) return rc;
        const bool bounded = timeout_ms >= 0;
        const auto deadline = std::chrono::steady_clock::now() + std::chrono::milliseconds(bounded ? timeout_ms : 0);
        for (Tracker* tr : {&ctx->t_d2h, &ctx->t_scatter, &ctx->t_compute}) {
            rc = tracker_drain(ctx, *tr, bounded, deadline);
            if (rc != PS_OK) return rc;
        }
        resolve_profile(ctx);
    }
    return do_poll(ctx, nullptr);
}

int32_t ps_launch_count(ps_ctx* ctx, int64_t* out) {
    if (!ctx || !out) return PS_ERR_INVALID;
    *out = ctx->launches;
    return PS_OK;
}

int32_t ps_get_profile(ps_ctx* ctx, ps_profile* out, int32_t reset) {
    if (!ctx || !out) return PS_ERR_INVALID;
    if (!ctx->bk) resolve_profile(ctx);
    out->attn_ms = ctx->prof_ms[kProfAttn];
    out->attn_launches = ctx->prof_n[kProfAttn];
    out->attn_kv_bytes = ctx->prof_bytes[kProfAttn];
    out->merge_ms = ctx->prof_ms[kProfMerge];
    out->merge_launches = ctx->prof_n[kProfMerge];
    out->gather_ms = ctx->prof_ms[kProfGather];
    out->gather_launches = ctx->prof_n[kProfGather];
    out->gather_bytes = ctx->prof_bytes[kProfGather];
    out->scatter_ms = ctx->prof_ms[kProfScatter];
    out->scatter_launches = ctx->prof_n[kProfScatter];
    out->scatter_bytes = ctx->prof_bytes[kProfScatter];
    out->d2h_ms = ctx->prof_ms[kProfD2H];
    out->d2h_copies = ctx->prof_n[kProfD2H];
    out->d2h_bytes = ctx->prof_bytes[kProfD2H];
    out->h2d_ms = ctx->prof_ms[kProfH2D];
    out->h2d_copies = ctx->prof_n[kProfH2D];
    out->h2d_bytes = ctx->prof_bytes[kProfH2D];
    if (reset) {
        for (int k = 0; k < kProfKinds; ++k) {
            ctx->prof_ms[k] = 0;
            ctx->prof_n[k] = 0;
            ctx->prof_bytes[k] = 0;
        }
    }
    return PS_OK;
}

int32_t ps_trace(ps_ctx* ctx, int32_t enable) {
    if (!ctx) return PS_ERR_INVALID;
    if (ctx->bk || !ctx->profile) return ctx->fail(PS_ERR_INVALID, "ps_trace: needs a device context created with PS_FLAG_PROFILE");
    ctx->trace.clear();
    ctx->tracing = enable != 0;
    if (ctx->tracing) {
        if (!ctx->trace_base) CK(cudaEventCreate(&ctx->trace_base));
        CK(cudaEventRecord(ctx->trace_base, ctx->compute));
    }
    return PS_OK;
}

int32_t ps_trace_read(ps_ctx* ctx, ps_trace_span* out, int32_t cap, int32_t* n) {
    if (!ctx || !n || cap < 0 || (cap > 0 && !out)) return PS_ERR_INVALID;
    if (!ctx->bk) resolve_profile(ctx);
    const int32_t have = (int32_t)ctx->trace.size();
    const int32_t m = std::min(cap, have);
    if (m > 0) memcpy(out, ctx->trace.data(), (size_t)m * sizeof(ps_trace_span));
    *n = have;
    return PS_OK;
}

int32_t ps_copy_blocks(ps_ctx* ctx, int32_t layer, const int32_t* ids, int32_t n_blocks, void* staging,
                       int32_t direction) {
    if (!ctx) return PS_ERR_INVALID;
    if (ctx->bk) return ctx->fail(PS_ERR_INVALID, "ps_copy_blocks: context holds no device (bookkeeping only)");
    if (layer < 0 || layer >= ctx->cfg.num_layers || !ids || n_blocks < 0 || n_blocks > ctx->cfg.num_gpu_blocks ||
        !staging || (direction != 0 && direction != 1))
        return ctx->fail(PS_ERR_INVALID, "ps_copy_blocks: bad argument");
    if (n_blocks == 0) return PS_OK;
    for (int32_t i = 0; i < n_blocks; ++i)
        if (ids[i] < 0 || ids[i] >= ctx->cfg.num_gpu_blocks) return ctx->fail(PS_ERR_INVALID, "ps_copy_blocks: bad block id");
    // the ids travel through a descriptor ring on the compute stream (no host wait between calls); a call with
    // the same ids as the previous one reuses that upload
    size_t ioff = ctx->ids_cache_off;
    if (ctx->ids_cache.size() != (size_t)n_blocks || memcmp(ctx->ids_cache.data(), ids, (size_t)n_blocks * 4) != 0) {
        int32_t rc = arena_alloc(ctx, ctx->a_ids, (size_t)n_blocks * 4, &ioff);
        if (rc != PS_OK) return rc;
        memcpy(ctx->a_ids.h + ioff, ids, (size_t)n_blocks * 4);
        CK(ps::launch_upload(ctx->a_ids.d + ioff, ctx->a_ids.hd + ioff, (size_t)round_up((int64_t)n_blocks * 4, 16),
                             ctx->compute));
        ctx->launches++;
        ctx->ids_cache.assign(ids, ids + n_blocks);
        ctx->ids_cache_off = ioff;
    }
    const int32_t* d_ids = (const int32_t*)(ctx->a_ids.d + ioff);
    const int64_t bytes = (int64_t)n_blocks * ctx->layer_block_bytes;
    if (direction == 0) {
        ProfScope prof(ctx, kProfGather, ctx->compute, bytes);
        CK(ps::launch_gather_layer(ctx->kpools[(size_t)layer], ctx->vpools[(size_t)layer], d_ids, n_blocks, staging,
                                   ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status, ctx->compute));
    } else {
        ProfScope prof(ctx, kProfScatter, ctx->compute, bytes);
        CK(ps::launch_scatter_layer(ctx->kpools[(size_t)layer], ctx->vpools[(size_t)layer], d_ids, n_blocks, staging,
                                    ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status, ctx->compute));
    }
    ctx->launches++;
    return PS_OK;
}

int32_t ps_link_probe(int64_t bytes, int32_t direction, int32_t iters, double* gb_per_s) {
    if (bytes <= 0 || iters <= 0 || !gb_per_s || direction < 0 || direction > 2) return PS_ERR_INVALID;
    void *h0 = nullptr, *h1 = nullptr, *d0 = nullptr, *d1 = nullptr;
    cudaStream_t s0 = nullptr, s1 = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr, e2 = nullptr;
    int32_t rc = PS_OK;
    double best = 0.0;
#define CKP(call)                        \
    do {                                 \
        if ((call) != cudaSuccess) {     \
            rc = PS_ERR_CUDA;            \
            g_create_error = #call;      \
            goto done;                   \
        }                                \
    } while (0)
    CKP(cudaHostAlloc(&h0, (size_t)bytes, cudaHostAllocDefault));
    CKP(cudaMalloc(&d0, (size_t)bytes));
    memset(h0, 1, (size_t)bytes);
    if (direction == 2) {
        CKP(cudaHostAlloc(&h1, (size_t)bytes, cudaHostAllocDefault));
        CKP(cudaMalloc(&d1, (size_t)bytes));
        CKP(cudaMemset(d1, 2, (size_t)bytes));
    }
    CKP(cudaStreamCreateWithFlags(&s0, cudaStreamNonBlocking));
    CKP(cudaStreamCreateWithFlags(&s1, cudaStreamNonBlocking));
    CKP(cudaEventCreate(&e0));
    CKP(cudaEventCreate(&e1));
    CKP(cudaEventCreate(&e2));
    for (int it = 0; it < iters + 1; ++it) {  // first pass warms up
        CKP(cudaEventRecord(e0, s0));
        if (direction == 2) CKP(cudaStreamWaitEvent(s1, e0, 0));
        if (direction == 0 || direction == 2) CKP(cudaMemcpyAsync(d0, h0, (size_t)bytes, cudaMemcpyHostToDevice, s0));
        if (direction == 1) CKP(cudaMemcpyAsync(h0, d0, (size_t)bytes, cudaMemcpyDeviceToHost, s0));
        if (direction == 2) {
            CKP(cudaMemcpyAsync(h1, d1, (size_t)bytes, cudaMemcpyDeviceToHost, s1));
            CKP(cudaEventRecord(e2, s1));
            CKP(cudaStreamWaitEvent(s0, e2, 0));
        }
        CKP(cudaEventRecord(e1, s0));
        CKP(cudaEventSynchronize(e1));
        float ms = 0.f;
        CKP(cudaEventElapsedTime(&ms, e0, e1));
        if (it > 0 && ms > 0.f) best = std::max(best, (direction == 2 ? 2.0 : 1.0) * (double)bytes / (ms * 1e-3) / 1e9);
    }
    *gb_per_s = best;
done:
#undef CKP
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (e2) cudaEventDestroy(e2);
    if (s0) cudaStreamDestroy(s0);
    if (s1) cudaStreamDestroy(s1);
    if (h0) cudaFreeHost(h0);
    if (h1) cudaFreeHost(h1);
    if (d0) cudaFree(d0);
    if (d1) cudaFree(d1);
    cudaGetLastError();
    return rc;
}

}  // extern "C"
