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

// Starts the offload of logical blocks [lo, hi) of a request as a new image segment: gather through the
// table into staging slots, slot by slot to the host.  Ordered after everything already enqueued on the
// compute stream (and after the scatters of a reload that is still landing).
int32_t offload_segment(ps_ctx* ctx, Req& r, int32_t lo, int32_t hi) {
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
        rc = issue_reload_layer(ctx, layer, {{req, blk_lo, blk_hi}});
        if (rc != PS_OK) return rc;
    }
    return note_layer_issued(ctx, req, r, layer, blk_hi);
}

int32_t ps_reload_fence(ps_ctx* ctx, int32_t layer) {
    if (!ctx) return PS_ERR_INVALID;
    if (layer < -1 || layer >= ctx->cfg.num_layers) return ctx->fail(PS_ERR_INVALID, "ps_reload_fence: layer out of range");
    if (ctx->bk) return PS_OK;
    // the layer's event was last recorded behind its most recent scatter, and the scatter stream runs in order
    const int lo = layer < 0 ? 0 : layer, hi = layer < 0 ? ctx->cfg.num_layers : layer + 1;
    for (int l = lo; l < hi; ++l) CK(cudaStreamWaitEvent(ctx->compute, ctx->ev_in[(size_t)l], 0));
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
