// Swap-out (gather into staging slots, slot by slot to the host image, on demand or ahead of eviction) and
// swap-in (host image -> staging -> scatter into fresh blocks, one completion event per layer).
// Section 4.3 "Asynchronous Offloading" and "Pipelined Reloading"; Appendix B.
#include "ps_ctx.h"

namespace psrt {

// ---- swap-in issue ------------------------------------------------------------------------------------

// Orders the scatter stream after everything already enqueued on the compute stream: a fresh block
// may have been released by a request whose last attention launch is still running.
int32_t order_scatter_after_compute(ps_ctx* ctx) {
    if (ctx->bk) return PS_OK;
    CK(cudaEventRecord(ctx->e_mark, ctx->compute));
    CK(cudaStreamWaitEvent(ctx->s_scatter, ctx->e_mark, 0));
    return PS_OK;
}

// Uploads the block ids of a reload plan (plan order) to the device on the scatter stream and returns where
// they sit.  A block id is the same in every layer, so one upload serves all the layer chunks of a step; a
// repeat of the previous upload (the caller-driven layer loop over one block range) reuses it.
int32_t upload_plan_ids(ps_ctx* ctx, const std::vector<PlanEntry>& plan, const int32_t** d_ids) {
    *d_ids = nullptr;
    if (ctx->bk || plan.empty()) return PS_OK;
    std::vector<int32_t> ids;
    for (const PlanEntry& e : plan) {
        const Req& r = ctx->reqs[e.req];
        ids.insert(ids.end(), r.table.begin() + e.lo, r.table.begin() + e.hi);
    }
    if (ids.empty()) return PS_OK;
    if (ids != ctx->scatter_ids_cache) {
        size_t off = 0;
        int32_t rc = arena_alloc(ctx, ctx->a_scatter, ids.size() * 4, &off);
        if (rc != PS_OK) return rc;
        memcpy(ctx->a_scatter.h + off, ids.data(), ids.size() * 4);
        CK(ps::launch_upload(ctx->a_scatter.d + off, ctx->a_scatter.hd + off, (size_t)round_up((int64_t)ids.size() * 4, 16),
                             ctx->s_scatter));
        ctx->launches++;
        ctx->scatter_ids_cache.swap(ids);
        ctx->scatter_ids_off = off;
    }
    *d_ids = (const int32_t*)(ctx->a_scatter.d + ctx->scatter_ids_off);
    return PS_OK;
}

// Issues one layer chunk of a reload plan: layers [l0, l0 + g) of every (request, block range) of the plan.
// Host image -> staging on the H2D stream (per request and image segment one copy: a contiguous range for
// g = 1, a strided one of g rows otherwise, since a layer's blocks are contiguous in the image and the
// layers are a fixed stride apart), then one scatter launch per staging piece on the scatter stream, then
// the chunk's completion event (Appendix B: one event per layer chunk), which every layer of the chunk
// refers to.  d_ids: the plan's ids on the device (upload_plan_ids).  Pieces are packed into the current
// staging slot while they fit, so small chunks never wait for a slot.
int32_t issue_reload_group(ps_ctx* ctx, int32_t l0, int32_t g, const std::vector<PlanEntry>& plan,
                           const int32_t* d_ids) {
    if (ctx->bk || plan.empty()) return PS_OK;
    const int64_t Bl = ctx->layer_block_bytes;
    int64_t left = 0;
    for (const PlanEntry& e : plan) left += e.hi - e.lo;
    if (left == 0) return PS_OK;
    const int64_t cap = std::max<int64_t>(ctx->slot_bytes / (g * Bl), 1);  // blocks per staging piece
    size_t i = 0;
    int32_t lo = plan[0].lo;
    int64_t id_off = 0;
    while (left > 0) {
        while (i < plan.size() && lo >= plan[i].hi) {
            ++i;
            if (i < plan.size()) lo = plan[i].lo;
        }
        const int64_t n_c = std::min(cap, left);
        const int64_t bytes = g * n_c * Bl;
        if (ctx->in_slot < 0 || ctx->in_fill + bytes > ctx->slot_bytes) {
            ctx->in_slot = (int)(ctx->in_next++ % kSlots);
            ctx->in_fill = 0;
            if (ctx->in_used[ctx->in_slot]) CK(cudaStreamWaitEvent(ctx->s_h2d, ctx->e_scattered[ctx->in_slot], 0));
        }
        const int slot = ctx->in_slot;
        char* sp = ctx->stage_in + (int64_t)slot * ctx->slot_bytes + ctx->in_fill;
        ctx->in_fill += bytes;
        int64_t used = 0;
        while (used < n_c) {
            Req& r = ctx->reqs[plan[i].req];
            const int64_t take = std::min<int64_t>(plan[i].hi - lo, n_c - used);
            if (take <= 0) {  // an empty range in the plan
                ++i;
                lo = plan[i].lo;
                continue;
            }
            // a run of blocks is cut at the borders of the image's segments
            for (int64_t j = lo, done = 0; done < take;) {
                const Req::Seg* sg = nullptr;
                for (const Req::Seg& c : r.segs)
                    if (j >= c.lo && j < c.hi) sg = &c;
                if (sg == nullptr) return ctx->fail(PS_ERR_STATE, "reload: block outside the host image");
                const int64_t piece = std::min<int64_t>(take - done, sg->hi - j);
                const int64_t seg_pitch = (int64_t)(sg->hi - sg->lo) * Bl;  // bytes between layers in the image
                const char* src = ctx->host_pool + sg->off + (int64_t)l0 * seg_pitch + (j - sg->lo) * Bl;
                char* dst = sp + (used + done) * Bl;
                ProfScope prof(ctx, kProfH2D, ctx->s_h2d, g * piece * Bl, l0);
                if (g == 1) {
                    CK(cudaMemcpyAsync(dst, src, (size_t)(piece * Bl), cudaMemcpyHostToDevice, ctx->s_h2d));
                } else if (seg_pitch <= ctx->max_pitch && n_c * Bl <= ctx->max_pitch) {
                    CK(cudaMemcpy2DAsync(dst, (size_t)(n_c * Bl), src, (size_t)seg_pitch, (size_t)(piece * Bl), (size_t)g,
                                         cudaMemcpyHostToDevice, ctx->s_h2d));
                } else {
                    for (int32_t l = 0; l < g; ++l)
                        CK(cudaMemcpyAsync(dst + l * n_c * Bl, src + l * seg_pitch, (size_t)(piece * Bl),
                                           cudaMemcpyHostToDevice, ctx->s_h2d));
                }
                j += piece;
                done += piece;
            }
            used += take;
            lo += (int32_t)take;
            if (lo >= plan[i].hi && used < n_c) {
                ++i;
                lo = plan[i].lo;
            }
        }
        CK(cudaEventRecord(ctx->e_loaded[slot], ctx->s_h2d));
        CK(cudaStreamWaitEvent(ctx->s_scatter, ctx->e_loaded[slot], 0));
        {
            ProfScope prof(ctx, kProfScatter, ctx->s_scatter, bytes, l0);
            CK(ps::launch_image_copy(/*scatter=*/true, ctx->d_kpools, ctx->d_vpools, d_ids + id_off, (int32_t)n_c, l0, 0,
                                     2 * n_c * g, sp, ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status,
                                     ctx->s_scatter));
            ctx->launches++;
        }
        CK(cudaEventRecord(ctx->e_scattered[slot], ctx->s_scatter));
        ctx->in_used[slot] = true;
        id_off += n_c;
        left -= n_c;
    }
    CK(cudaEventRecord(ctx->ev_in[(size_t)l0], ctx->s_scatter));
    for (int32_t l = l0; l < l0 + g; ++l) ctx->ev_of_layer[(size_t)l] = l0;
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

// Gathers one staging slot's worth of an image and copies it to the host (slot -> host on the D2H stream).
cudaError_t issue_out_chunk(ps_ctx* ctx, const OutChunk& c, int slot, bool profiled) {
    char* sp = ctx->stage_out + (int64_t)slot * ctx->slot_bytes;
    cudaError_t e = cudaSuccess;
    if (ctx->out_used[slot]) e = cudaStreamWaitEvent(ctx->s_gather, ctx->e_drained[slot], 0);
    if (e != cudaSuccess) return e;
    const int64_t bytes = c.cnt * ctx->slab_bytes;
    {
        ProfScope prof(ctx, kProfGather, ctx->s_gather, profiled ? bytes : 0, -1, profiled);
        e = ps::launch_image_copy(/*scatter=*/false, ctx->d_kpools, ctx->d_vpools, c.d_table, c.n_blk, 0, c.s0, c.cnt, sp,
                                  ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status, ctx->s_gather);
        ctx->launches++;
    }
    if (e == cudaSuccess) e = cudaEventRecord(ctx->e_gathered[slot], ctx->s_gather);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->s_d2h, ctx->e_gathered[slot], 0);
    if (e != cudaSuccess) return e;
    {
        ProfScope prof(ctx, kProfD2H, ctx->s_d2h, profiled ? bytes : 0, -1, profiled);
        e = cudaMemcpyAsync(c.host_dst, sp, (size_t)bytes, cudaMemcpyDeviceToHost, ctx->s_d2h);
    }
    if (e == cudaSuccess) e = cudaEventRecord(ctx->e_drained[slot], ctx->s_d2h);
    if (e == cudaSuccess) ctx->out_used[slot] = true;
    return e;
}

// The offload worker: takes chunks in issue order and keeps at most kOutInflight of them with the copy engine.
// The copy engine serves device-to-host copies in the order they were submitted, whatever their stream, so an
// offload submitted whole would hold every later copy of the process (a step's results, sampled tokens) for its
// full duration.  Completion tickets are recorded here too, behind the chunks queued before them.
void out_worker_main(ps_ctx* ctx) {
    cudaSetDevice(ctx->device);
    std::deque<int> inflight;  // slots whose copy has been submitted, oldest first
    for (;;) {
        OutChunk c;
        {
            std::unique_lock<std::mutex> lk(ctx->out_mu);
            ctx->out_cv.wait(lk, [&] { return ctx->out_stop || !ctx->out_pending.empty(); });
            if (ctx->out_stop) return;
            c = ctx->out_pending.front();
            ctx->out_pending.pop_front();
        }
        cudaError_t e = cudaSuccess;
        const char* what = "";
        if (c.cnt > 0 && !ctx->out_failed.load()) {
            if ((int)inflight.size() >= kOutInflight) {
                e = cudaEventSynchronize(ctx->e_drained[inflight.front()]);
                what = "waiting for a staging slot to drain";
                inflight.pop_front();
            }
            if (e == cudaSuccess) {
                const int slot = (int)(ctx->out_next++ % kSlots);
                e = issue_out_chunk(ctx, c, slot, /*profiled=*/false);
                what = "offload chunk (gather + device-to-host copy)";
                inflight.push_back(slot);
            }
        }
        if (c.ticket != 0) {  // recorded even after a failure, so that waits on the ticket end
            cudaEvent_t ev = nullptr;
            cudaError_t e2 = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
            if (e2 == cudaSuccess) e2 = cudaEventRecord(ev, ctx->s_d2h);
            if (e2 == cudaSuccess) {
                std::lock_guard<std::mutex> lk(ctx->t_d2h.mu);
                ctx->t_d2h.pending.emplace_back(c.ticket, ev);
            } else if (e == cudaSuccess) {
                e = e2;
                what = "recording an offload's completion event";
            }
        }
        if (e != cudaSuccess && !ctx->out_failed.load()) {
            std::lock_guard<std::mutex> lk(ctx->out_mu);
            ctx->out_error = std::string(what) + ": " + cudaGetErrorString(e);
            ctx->out_failed.store(true);
        }
    }
}

// Starts the offload of logical blocks [lo, hi) of a request as a new image segment: gather through the
// table into staging slots, slot by slot to the host.  Ordered after everything already enqueued on the
// compute stream (and after the scatters of a reload that is still landing).
int32_t offload_segment(ps_ctx* ctx, Req& r, int32_t lo, int32_t hi) {
    const int64_t n_blk = hi - lo;
    const int64_t bytes = n_blk * ctx->block_bytes;
    int64_t off = ctx->hpool.alloc(bytes);
    if (off < 0) {  // images of reloads that have landed since the last poll may still be held
        int32_t rc = do_poll(ctx, nullptr, /*reap_offloads=*/false);
        if (rc != PS_OK) return rc;
        off = ctx->hpool.alloc(bytes);
    }
    if (off < 0) return ctx->fail(PS_ERR_HOST_NOMEM, "host pool cannot hold the image");
    if (ctx->out_failed.load()) {
        ctx->hpool.release(off, bytes);
        std::lock_guard<std::mutex> lk(ctx->out_mu);
        return ctx->fail(PS_ERR_CUDA, "an earlier offload failed: " + ctx->out_error);
    }

    std::vector<OutChunk> chunks;
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
        e = ps::launch_upload(ctx->a_gather.d + toff, ctx->a_gather.hd + toff, (size_t)round_up(n_blk * 4, 16),
                              ctx->s_gather);
        ctx->launches++;
        if (e != cudaSuccess) {
            ctx->hpool.release(off, bytes);
            return ctx->fail_cuda(e, "table upload");
        }
        const int64_t total_slabs = 2 * n_blk * ctx->cfg.num_layers;
        const int64_t slot_slabs = ctx->slot_bytes / ctx->slab_bytes;
        for (int64_t s0 = 0; s0 < total_slabs; s0 += slot_slabs) {
            OutChunk c;
            c.d_table = (const int32_t*)(ctx->a_gather.d + toff);
            c.n_blk = (int32_t)n_blk;
            c.s0 = s0;
            c.cnt = std::min(slot_slabs, total_slabs - s0);
            c.host_dst = ctx->host_pool + off + s0 * ctx->slab_bytes;
            chunks.push_back(c);
        }
    }
    Req::Seg sg{lo, hi, off, bytes, 0};
    if (ctx->out_paced) {
        // The block tables of queued chunks live in the descriptor ring, whose chunks are reused after a few MiB
        // of newer tables: tables of pending chunks add up to less than the pool's ids plus 256 bytes per
        // segment, so bounding the queue keeps them far from reuse.
        for (;;) {
            {
                std::lock_guard<std::mutex> lk(ctx->out_mu);
                if (ctx->out_pending.size() < 4096 || ctx->out_failed.load()) break;
            }
            std::this_thread::sleep_for(std::chrono::microseconds(100));
        }
        // the worker issues the chunks; the segment's ticket rides on the last one (or on an empty chunk)
        sg.ticket = ctx->t_d2h.next++;
        if (chunks.empty()) chunks.emplace_back();
        chunks.back().ticket = sg.ticket;
        {
            std::lock_guard<std::mutex> lk(ctx->out_mu);
            for (const OutChunk& c : chunks) ctx->out_pending.push_back(c);
        }
        ctx->out_cv.notify_one();
    } else {
        // issued here, slot after slot (contexts that time every launch, or hold no device)
        bool copies_enqueued = false;
        for (const OutChunk& c : chunks) {
            const int slot = (int)(ctx->out_next++ % kSlots);
            cudaError_t e = issue_out_chunk(ctx, c, slot, /*profiled=*/true);
            if (e != cudaSuccess) {
                // a range that copies already in flight write into is parked behind a ticket, never reused early
                uint64_t ticket = 0;
                if (!copies_enqueued)
                    ctx->hpool.release(off, bytes);
                else if (tracker_mark(ctx, ctx->t_d2h, &ticket) == PS_OK)
                    ctx->host_release.push_back({ticket, {off, bytes}});
                return ctx->fail_cuda(e, "offload chunk (gather + device-to-host copy)");
            }
            copies_enqueued = true;
        }
        int32_t rc = tracker_mark(ctx, ctx->t_d2h, &sg.ticket);
        if (rc != PS_OK) return rc;  // the range stays reserved: copies may be in flight and nothing tells when they end
    }
    r.segs.push_back(sg);
    r.host_issued = hi;
    return PS_OK;
}

}  // namespace psrt

extern "C" {

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

int32_t ps_offload_sweep(ps_ctx* ctx, const int64_t* reqs, const int32_t* n_off, int32_t batch,
                         int64_t* issued_blocks) {
    if (!ctx) return PS_ERR_INVALID;
    if (issued_blocks) *issued_blocks = 0;
    if (batch < 0 || (batch > 0 && (!reqs || !n_off))) return ctx->fail(PS_ERR_INVALID, "ps_offload_sweep: bad argument");
    for (int32_t i = 0; i < batch; ++i)
        if (n_off[i] <= 0) return ctx->fail(PS_ERR_INVALID, "ps_offload_sweep: thresholds must be positive");
    int64_t total = 0;
    for (int32_t i = 0; i < batch; ++i) {
        auto it = ctx->reqs.find(reqs[i]);
        if (it == ctx->reqs.end() || it->second.state != PS_REQ_RESIDENT) continue;
        int32_t issued = 0;
        int32_t rc = ps_offload_progress(ctx, reqs[i], n_off[i], &issued);
        total += issued;
        if (issued_blocks) *issued_blocks = total;
        if (rc != PS_OK) return rc;
    }
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
        const std::vector<PlanEntry> plan{{req, blk_lo, blk_hi}};
        const int32_t* d_ids = nullptr;
        rc = upload_plan_ids(ctx, plan, &d_ids);
        if (rc != PS_OK) return rc;
        rc = issue_reload_group(ctx, layer, 1, plan, d_ids);
        if (rc != PS_OK) return rc;
    }
    return note_layer_issued(ctx, req, r, layer, blk_hi);
}

int32_t ps_reload_fence(ps_ctx* ctx, int32_t layer) {
    if (!ctx) return PS_ERR_INVALID;
    if (layer < -1 || layer >= ctx->cfg.num_layers) return ctx->fail(PS_ERR_INVALID, "ps_reload_fence: layer out of range");
    if (ctx->bk) return PS_OK;
    // the event of the layer's chunk was last recorded behind its most recent scatter, and the scatter stream
    // runs in order
    const int lo = layer < 0 ? 0 : layer, hi = layer < 0 ? ctx->cfg.num_layers : layer + 1;
    for (int l = lo; l < hi; ++l) {
        if (l > lo && ctx->ev_of_layer[(size_t)l] == ctx->ev_of_layer[(size_t)l - 1]) continue;  // same layer chunk
        CK(cudaStreamWaitEvent(ctx->compute, ctx->ev_in[(size_t)ctx->ev_of_layer[(size_t)l]], 0));
    }
    return PS_OK;
}

int32_t ps_missing_blocks(ps_ctx* ctx, int64_t req, int32_t* out) {
    if (!ctx || !out) return PS_ERR_INVALID;
    auto it = ctx->reqs.find(req);
    if (it == ctx->reqs.end()) return ctx->fail(PS_ERR_INVALID, "ps_missing_blocks: unknown request");
    *out = missing_of(it->second);
    return PS_OK;
}

}  // extern "C"
