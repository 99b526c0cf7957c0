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
// and a kernel never reads a slot the engine is still filling.  Reload pieces smaller than a slot are
// packed into the current slot one after the other.
#include "ps_ctx.h"

namespace psrt {

std::string& create_error() {
    static std::string text = "";
    return text;
}

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
    if (t.via_worker) {  // the worker records the event when it reaches this point of its queue
        OutChunk c;
        c.ticket = *ticket;
        {
            std::lock_guard<std::mutex> lk(ctx->out_mu);
            ctx->out_pending.push_back(c);
        }
        ctx->out_cv.notify_one();
        return PS_OK;
    }
    cudaEvent_t ev;
    CK(get_event(ctx, false, &ev));
    CK(cudaEventRecord(ev, t.s));
    t.pending.emplace_back(*ticket, ev);
    return PS_OK;
}

int32_t tracker_poll(ps_ctx* ctx, Tracker& t) {
    std::unique_lock<std::mutex> lk(t.mu, std::defer_lock);
    if (t.via_worker) lk.lock();
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

// Waits until every ticket handed out so far is complete or the deadline passes.
int32_t tracker_drain(ps_ctx* ctx, Tracker& t, bool bounded, std::chrono::steady_clock::time_point deadline) {
    while (t.done + 1 < t.next) {
        cudaEvent_t last = nullptr;
        {
            std::unique_lock<std::mutex> lk(t.mu, std::defer_lock);
            if (t.via_worker) lk.lock();
            if (!t.pending.empty()) last = t.pending.back().second;
        }
        if (!bounded && last != nullptr) CK(cudaEventSynchronize(last));
        int32_t rc = tracker_poll(ctx, t);
        if (rc != PS_OK) return rc;
        if (t.done + 1 >= t.next) break;
        if (t.via_worker && ctx->out_failed.load()) {
            std::lock_guard<std::mutex> lk(ctx->out_mu);
            return ctx->fail(PS_ERR_CUDA, "offload worker: " + ctx->out_error);
        }
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

int32_t arena_next_chunk(ps_ctx* ctx, Arena& a, bool record_fence) {
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

void push_table(ps_ctx* ctx, std::vector<int32_t>& table) {
    for (int32_t id : table) ctx->free_stack.push_back(id);  // table order: the last entry ends on top
    table.clear();
    ctx->table_epoch++;
}

// Kernels report through one mapped word: 1 = a copy kernel met a block id outside the pool, 2 = an attention
// kernel did, 3 = a bounded wait inside the tensor-core attention kernel ran out and its CTAs left early.
// After 3 the launch's outputs are undefined and its CTAs did not re-arm the kernel's chunk and arrival
// counters, so these are cleared on their streams before anything else is launched over them.
int32_t check_status_word(ps_ctx* ctx) {
    if (ctx->status && *(volatile int32_t*)ctx->status != 0) {
        const int v = *(volatile int32_t*)ctx->status;
        *(volatile int32_t*)ctx->status = 0;
        if (v == 3) {
            if (!ctx->bk) {
                const size_t done_bytes = (size_t)std::max(ctx->cfg.max_batch, 1) * ctx->cfg.num_kv_heads * sizeof(int32_t);
                for (int i = 0; i < 3; ++i) {
                    cudaStream_t st = i == 2 ? ctx->s_lane : ctx->compute;
                    if (ctx->d_sched[i]) CK(cudaMemsetAsync(ctx->d_sched[i], 0, 4 * sizeof(int32_t), st));
                    if (ctx->d_row_done[i]) CK(cudaMemsetAsync(ctx->d_row_done[i], 0, done_bytes, st));
                }
            }
            ctx->meta.valid = false;
            return ctx->fail(PS_ERR_TIMEOUT,
                             "attention kernel: a bounded wait on a shared-memory barrier ran out; the outputs of the "
                             "launches in flight are undefined; the kernel's counters have been reset");
        }
        return ctx->fail(PS_ERR_BOUNDS, v == 2 ? "attention kernel met a block id outside the pool"
                                               : "copy kernel met a block id outside the pool");
    }
    return PS_OK;
}

int32_t do_poll(ps_ctx* ctx, int32_t* n_reaped, bool reap_offloads) {
    int32_t reaped = 0;
    int32_t rc = tracker_poll(ctx, ctx->t_d2h);
    if (rc != PS_OK) return rc;
    while (reap_offloads && !ctx->out_fifo.empty()) {
        Req& r = ctx->reqs[ctx->out_fifo.front()];
        if (r.out_ticket > ctx->t_d2h.done) break;  // offloads complete in issue order
        push_table(ctx, r.table);
        r.state = PS_REQ_HOST;
        ctx->out_fifo.pop_front();
        ++reaped;
    }
    while (!ctx->host_release.empty() && ctx->host_release.front().first <= ctx->t_d2h.done) {
        ctx->hpool.release(ctx->host_release.front().second.first, ctx->host_release.front().second.second);
        ctx->host_release.pop_front();
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
    if (ctx->out_failed.load()) {
        std::lock_guard<std::mutex> lk(ctx->out_mu);
        return ctx->fail(PS_ERR_CUDA, "offload worker: " + ctx->out_error);
    }
    return check_status_word(ctx);
}

void destroy_ctx(ps_ctx* ctx) {
    if (ctx->out_thread.joinable()) {
        {
            std::lock_guard<std::mutex> lk(ctx->out_mu);
            ctx->out_stop = true;
        }
        ctx->out_cv.notify_all();
        ctx->out_thread.join();
    }
    if (!ctx->bk) {
        // If the caller's bounded wait ran out, copies into the staging slots and the pinned pool may still be
        // queued (the worker, joined above, issues none any more): nothing is freed under them.  What is left
        // is finite (transfers, and kernels whose own waits are bounded), so the streams are waited for here
        // without a limit; on an idle context this costs nothing.
        bool any_stream = false;
        for (cudaStream_t s : {ctx->s_gather, ctx->s_d2h, ctx->s_h2d, ctx->s_scatter, ctx->s_lane})
            if (s) {
                cudaStreamSynchronize(s);
                any_stream = true;
            }
        if (any_stream) cudaStreamSynchronize(ctx->compute);
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
        arena_free(ctx->a_scatter);
        if (ctx->io_q) cudaFree(ctx->io_q);
        if (ctx->io_out) cudaFree(ctx->io_out);
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
        ctx->status = nullptr;
        if (ctx->own_host_pool && ctx->host_pool) cudaFreeHost(ctx->host_pool);
        cudaGetLastError();
    }
    if (ctx->bk && ctx->status) free(ctx->status);
    delete ctx;
}

int32_t create_fail(ps_ctx* ctx, int32_t code) {
    create_error() = ctx->err;
    destroy_ctx(ctx);
    return code;
}

}  // namespace psrt

// =====================================================================================================
// C ABI: context, block pool, completion, measurement read-out
// =====================================================================================================

extern "C" {

const char* ps_last_error(const ps_ctx* ctx) { return ctx ? ctx->err.c_str() : create_error().c_str(); }

int32_t ps_create(const ps_config* cfg, void* const* k_pools, void* const* v_pools, void* host_pool,
                  void* compute_stream, ps_ctx** out) {
    if (!cfg || !out) {
        create_error() = "null argument";
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
        const bool g_ok = ctx->G >= 1 && ctx->G <= 8;
        if (!g_ok || (cfg->head_dim != 64 && cfg->head_dim != 128)) {
            ctx->err = "unsupported attention shape: head_dim must be 64 or 128, Hq/Hkv from 1 to 8";
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
    ctx->chunk_min_bytes = cfg->layer_chunk_bytes == 0 ? (2LL << 20) : std::max<int64_t>(cfg->layer_chunk_bytes, 0);
    ctx->ev_of_layer.resize((size_t)cfg->num_layers);
    for (int32_t l = 0; l < cfg->num_layers; ++l) ctx->ev_of_layer[(size_t)l] = l;
    if (ctx->bk) {
        ctx->status = (int32_t*)calloc(16, sizeof(int32_t));  // no kernel writes it; the status path stays testable
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
    CKC(cudaGetDevice(&ctx->device));
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
    CKR(arena_init(ctx, ctx->a_scatter, (size_t)cfg->num_gpu_blocks * 4, 4, ctx->s_scatter));  // reload plans
    {
        int dev = 0, pitch = 0;
        CKC(cudaGetDevice(&dev));
        CKC(cudaDeviceGetAttribute(&pitch, cudaDevAttrMaxPitch, dev));
        ctx->max_pitch = pitch;
    }

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
        if (ctx->attn_kernel == PS_ATTN_MMA && ctx->tmaps.empty() && cfg->num_kv_heads != 8) {
            // the row-copy form of the kernel exists for 8 KV heads only
            if (cfg->attn_kernel != PS_ATTN_AUTO) {
                ctx->err = "the tensor-core attention kernel needs tensor maps for fewer than 8 KV heads";
                return create_fail(ctx, PS_ERR_INVALID);
            }
            ctx->attn_kernel = PS_ATTN_SIMT;
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
    // the offload worker; contexts that time every launch issue their offloads on the caller's thread instead
    if (!ctx->profile) {
        ctx->out_paced = true;
        ctx->t_d2h.via_worker = true;
        ctx->out_thread = std::thread(out_worker_main, ctx);
    }
    *out = ctx;
    return PS_OK;
}

int32_t ps_destroy(ps_ctx* ctx) {
    if (!ctx) return PS_ERR_INVALID;
    int32_t rc = PS_OK;
    if (!ctx->bk) {
        rc = ps_sync(ctx, 10000);
    }
    destroy_ctx(ctx);
    return rc == PS_ERR_TIMEOUT ? PS_ERR_TIMEOUT : PS_OK;
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
            int32_t rc = do_poll(ctx, nullptr, /*reap_offloads=*/false);
            if (rc != PS_OK) return rc;
            if (r.gated) return ctx->fail(PS_ERR_BUSY, "ps_kv_free: reload copies still in flight");
        }
        if (!r.segs.empty()) {  // proactive copies: their transfers must have ended before the image goes
            int32_t rc = do_poll(ctx, nullptr, /*reap_offloads=*/false);
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
    *out = ctx->launches.load();
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

}  // extern "C"
