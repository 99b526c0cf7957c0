// One engine step under the copy budget: budget consumption over the reload queue, the decode batch's device
// metadata and work split, per-layer attention launches gated on the reload events (Section 4.3 "Put it
// Together"; Appendix B).
#include "ps_ctx.h"

namespace psrt {

// Copy-budget consumption (Alg. 1, ConsumeCopyBudget, with the byte budget turned into blocks): FIFO, whole
// request if it fits, otherwise the residual -- always (rule == nullptr or the request is not listed in it), or
// only if SatisfyCopyCondition holds for the request (Section 4.3 "Put it Together": l_comp reaches the round's
// limit, or l_comp / ((b_miss - B_rem) * s_blk) > beta); a request that fails the test is skipped for this
// round and the next one in the queue is tried with the budget unchanged.
std::vector<PlanEntry> make_plan(ps_ctx* ctx, int64_t copy_budget_bytes, const ps_copy_rule* rule) {
    std::vector<PlanEntry> plan;
    const bool unlimited = copy_budget_bytes < 0;
    int64_t left = unlimited ? 0 : copy_budget_bytes / ctx->block_bytes;
    for (int64_t id : ctx->in_fifo) {
        Req& r = ctx->reqs[id];
        const int32_t miss = missing_of(r);
        if (miss == 0) continue;
        const int32_t lo = (int32_t)r.table.size() - miss;
        if (!unlimited && left == 0) break;
        int64_t take = miss;
        if (!unlimited && miss > left) {
            bool allowed = true;
            if (rule != nullptr)
                for (int32_t k = 0; k < rule->n; ++k)
                    if (rule->reqs[k] == id) {
                        int32_t ok = 1;
                        ps_copy_condition(rule->l_comp[k], rule->l_comp_max[k], miss, (int32_t)left, ctx->cfg.block_size,
                                          rule->beta, &ok);
                        allowed = ok != 0;
                        break;
                    }
            if (!allowed) continue;
            take = left;
        }
        plan.push_back({id, lo, lo + (int32_t)take});
        if (!unlimited) left -= take;
    }
    return plan;
}

// Layers per chunk for a step that reloads n_blocks blocks: one layer's share of the step (n_blocks * layer
// block bytes) may be far below what a copy engine needs to run at link rate, so consecutive layers are
// grouped until a chunk carries chunk_min_bytes (Appendix B speaks of a completion event per layer *chunk*).
// A chunk must fit a staging slot.
int32_t layers_per_chunk(const ps_ctx* ctx, int64_t n_blocks) {
    const int64_t per_layer = n_blocks * ctx->layer_block_bytes;
    if (ctx->chunk_min_bytes <= 0 || per_layer <= 0 || per_layer >= ctx->chunk_min_bytes) return 1;
    int64_t g = (ctx->chunk_min_bytes + per_layer - 1) / per_layer;
    g = std::min<int64_t>(g, ctx->slot_bytes / per_layer);
    return (int32_t)std::max<int64_t>(1, std::min<int64_t>(g, ctx->cfg.num_layers));
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
                      const std::vector<char>& gated, bool want_lanes, int tail_mode) {
    BatchMeta& m = ctx->meta;
    // two work lists (lanes) only for the tensor-core kernel and only when some row is gated
    bool two_lanes = false;
    if (want_lanes && ctx->attn_kernel == PS_ATTN_MMA)
        for (int32_t b = 0; b < B; ++b) two_lanes |= active[b] && gated[b];
    if (m.valid && m.epoch == ctx->table_epoch && (int32_t)m.reqs.size() == B && m.two_lanes == two_lanes &&
        m.tail_mode == tail_mode &&
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
            // only the rows cut by share borders need combining.  With tail_mode 1 (reload traffic beside the
            // step: scatter kernels and the reload lane take SM time unevenly) the last 5 % of the sequence
            // become chunks that the CTAs take dynamically through an atomic counter.  Without contention a
            // dynamic part only costs: every chunk is one more partial result to write and combine (172
            // against 189 us per 1 GiB launch for a 5 % tail; handing out the last 3 % of every share instead,
            // 148 small chunks at share borders, took an isolated 537 MB launch from 89 to 93 us), so launches
            // on their own keep equal static shares.  An item is the part of a row that falls into one share
            // or chunk.
            const ps::AttnShape shape{ctx->cfg.num_kv_heads, ctx->cfg.num_q_heads, ctx->cfg.head_dim, ctx->cfg.block_size,
                                      ctx->cfg.num_gpu_blocks};
            const int kTile = ps::attn_mma_tile_tokens(shape);
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
            if (tail_mode == 1 && n_cta > 0 && total_tiles >= 32 * n_cta) {
                dyn_tiles = total_tiles * 5 / 100;
                chunk = std::max<int64_t>(kDynMinChunk, (dyn_tiles + kDynChunksPerCta * n_cta - 1) / (kDynChunksPerCta * n_cta));
            }
            const int64_t static_tiles = total_tiles - dyn_tiles;
            const int64_t per = n_cta > 0 ? std::max<int64_t>((static_tiles + n_cta - 1) / n_cta, 1) : 1;
            // Owner of sequence position pos: a CTA (its static share) or -1 (dynamic); *bound = where that ends.
            auto owner_at = [&](int64_t pos, int64_t* bound) -> int64_t {
                if (pos >= static_tiles) {  // tail_mode 1: chunks of the sequence's end
                    const int64_t k = (pos - static_tiles) / chunk;
                    *bound = std::min(total_tiles, static_tiles + (k + 1) * chunk);
                    return -1;
                }
                const int64_t c = std::min(pos / per, n_cta - 1);
                *bound = std::min((c + 1) * per, static_tiles);
                return c;
            };
            struct Piece {
                ps::AttnItem it;
                int64_t owner;
            };
            std::vector<Piece> pieces;  // in sequence order
            int64_t pos = 0;
            for (int32_t b = 0; b < B; ++b) {
                if (!active[b] || (two_lanes && (gated[b] ? 1 : 0) != pass)) continue;
                const Req& r = ctx->reqs[reqs[b]];
                const int64_t tiles_b = (r.n_tokens + kTile - 1) / kTile;
                const size_t first_piece = pieces.size();
                ctx_len[b] = r.n_tokens;
                row_first[b] = parts;
                if (tiles_b == 0) {  // empty context: one item without tiles writes the zero row
                    ps::AttnItem it{};
                    it.b = b;
                    pieces.push_back({it, std::min(pos / per, n_cta - 1)});
                }
                for (int64_t lo = 0; lo < tiles_b;) {
                    int64_t bound = 0;
                    const int64_t owner = owner_at(pos, &bound);
                    const int64_t take = std::min(tiles_b - lo, std::max<int64_t>(bound - pos, 1));
                    ps::AttnItem it{};
                    it.b = b;
                    it.t_begin = (int32_t)(lo * kTile);
                    it.t_end = (int32_t)std::min<int64_t>(r.n_tokens, (lo + take) * kTile);
                    pieces.push_back({it, owner});
                    lo += take;
                    pos += take;
                }
                const int32_t n = (int32_t)(pieces.size() - first_piece);
                for (size_t k = first_piece; k < pieces.size(); ++k) {
                    pieces[k].it.part = parts + (int32_t)(k - first_piece);
                    pieces[k].it.n_parts = n;
                }
                row_parts[b] = n;
                parts += n;
                any_multi |= n > 1;
                lane_multi[pass] |= n > 1;
                if (gated[b]) ++n_gated_rows;
            }
            // the lane's item list: the static items CTA by CTA (their owners never decrease along the sequence),
            // then the dynamic ones in sequence order
            if (n_cta > 0) {
                int64_t next_cta = 0;
                for (const Piece& pc : pieces) {
                    if (pc.owner < 0) continue;
                    while (next_cta <= pc.owner) {
                        cta_begin[pass].push_back((int32_t)items.size());
                        ++next_cta;
                    }
                    items.push_back(pc.it);
                }
                while (next_cta <= n_cta) {  // CTAs without items, and entry n_cta: where the dynamic items start
                    cta_begin[pass].push_back((int32_t)items.size());
                    ++next_cta;
                }
                for (const Piece& pc : pieces)
                    if (pc.owner < 0) items.push_back(pc.it);
            }
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
    m.tail_mode = tail_mode;
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
        // one layer per call: the caller's kernels sit between the launches, so only the set-up may run early
        const bool early_setup = !follows_own && mma && !ctx->profile && wait_event == nullptr &&
                                 (ctx->cfg.flags & PS_FLAG_ATTN_PLAIN_LAUNCH) == 0;
        const int set = ctx->scratch_set;
        ctx->scratch_set ^= 1;
        const int64_t bytes = m.kv_bytes_per_layer * m.n_ungated_items / m.n_items;
        {
            ProfScope prof(ctx, kProfAttn, ctx->compute, bytes, wait_event && !lanes ? 1000 + layer : layer);
            CK(ps::launch_decode_attn(ctx->attn_kernel, sh, ctx->kpools[layer], ctx->vpools[layer], maps, q, out, lse, m.dev,
                                      0, ctx->partials[set], ctx->d_sched[set], ctx->d_row_done[set], ctx->d_status,
                                      overlap ? 1 : early_setup ? 2 : 0, ctx->compute));
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
                                  ctx->partials[2], ctx->d_sched[2], ctx->d_row_done[2], ctx->d_status, 0, ctx->s_lane));
        ctx->launches++;
        ++*n_launched;
    }
    return PS_OK;
}

}  // namespace psrt

extern "C" {

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
        int32_t rc = do_poll(ctx, nullptr, /*reap_offloads=*/false);  // the copies may have landed since
        if (rc != PS_OK) return rc;
    }
    std::vector<char> active((size_t)batch, 1), gated((size_t)batch, 0);
    for (int32_t b = 0; b < batch; ++b) gated[(size_t)b] = ctx->reqs[reqs[b]].gated ? 1 : 0;
    int32_t rc = prepare_batch(ctx, reqs, batch, active, gated, /*want_lanes=*/false, /*tail_mode=*/0);
    if (rc != PS_OK) return rc;
    int32_t launched = 0;
    return launch_layer_attn(ctx, layer, q, out, lse,
                             ctx->meta.n_gated_rows ? ctx->ev_in[(size_t)ctx->ev_of_layer[(size_t)layer]] : nullptr,
                             /*follows_own=*/false, &launched);
}

static int32_t step_impl(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs,
                         int32_t batch, int64_t copy_budget_bytes, const ps_copy_rule* rule, int32_t* decoded_mask,
                         ps_step_stats* stats) {
    if (batch < 0 || (batch > 0 && !reqs)) return ctx->fail(PS_ERR_INVALID, "ps_step: bad batch");
    if (rule != nullptr && (!(rule->beta > 1.0) || rule->n < 0 ||
                            (rule->n > 0 && (!rule->reqs || !rule->l_comp || !rule->l_comp_max))))
        return ctx->fail(PS_ERR_INVALID, "ps_step_ruled: beta must exceed 1 and the rule's arrays must be given");
    if (rule != nullptr)
        for (int32_t k = 0; k < rule->n; ++k)
            if (rule->l_comp[k] < 0 || rule->l_comp_max[k] < 0)
                return ctx->fail(PS_ERR_INVALID, "ps_step_ruled: negative token count in the rule");
    const bool want_attn = q_all_layers != nullptr || out_all_layers != nullptr;
    if (want_attn && (ctx->bk || !q_all_layers || !out_all_layers || batch > ctx->cfg.max_batch))
        return ctx->fail(PS_ERR_INVALID, "ps_step: attention needs q and out on a device context, batch <= max_batch");
    ps_step_stats st{};
    int32_t reaped = 0;
    int32_t rc = do_poll(ctx, &reaped);
    if (rc != PS_OK) return rc;
    st.swapouts_reaped = reaped;

    // 1. the copy budget is consumed over the reload queue
    const std::vector<PlanEntry> plan = make_plan(ctx, copy_budget_bytes, rule);
    std::vector<char> completes(plan.size(), 0);
    for (size_t i = 0; i < plan.size(); ++i) {
        st.blocks_copied += plan[i].hi - plan[i].lo;
        completes[i] = plan[i].hi == (int32_t)ctx->reqs[plan[i].req].table.size();
    }
    st.h2d_bytes = st.blocks_copied * ctx->block_bytes;
    const int L = ctx->cfg.num_layers;
    const int64_t launches_before = ctx->launches.load();

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
        // a reload of 32 MiB or more per step slows SMs unevenly enough for a dynamic tail to pay off
        const bool pipelined = (ctx->cfg.flags & PS_FLAG_SYNC_RELOAD) == 0;
        rc = prepare_batch(ctx, reqs, batch, active, gated, pipelined,
                           /*tail_mode=*/pipelined && st.h2d_bytes >= (32LL << 20) ? 1 : 0);
        if (rc != PS_OK) return rc;
        st.gated = ctx->meta.n_gated_rows;
    }

    // 3. the step's layer chunks: first_of[l] = size of the chunk that starts at layer l, else 0.  When rows of
    // the batch wait for this step's reload, the first chunk is a single layer, so that their first layer
    // starts after the smallest possible transfer.
    std::vector<int32_t> first_of((size_t)L, 0);
    const int32_t* d_ids = nullptr;
    if (!plan.empty()) {
        rc = order_scatter_after_compute(ctx);
        if (rc != PS_OK) return rc;
        rc = upload_plan_ids(ctx, plan, &d_ids);
        if (rc != PS_OK) return rc;
        const int32_t g = layers_per_chunk(ctx, st.blocks_copied);
        int32_t l = 0;
        if (g > 1 && attn && ctx->meta.n_gated_rows > 0) first_of[(size_t)l++] = 1;
        while (l < L) {
            first_of[(size_t)l] = std::min<int32_t>(g, L - l);
            l += first_of[(size_t)l];
        }
    }

    // 4. per layer: its reload chunk (if one starts here) on the copy streams, then the layer's attention on
    // the compute stream
    const bool sync_reload = (ctx->cfg.flags & PS_FLAG_SYNC_RELOAD) != 0 || !attn;
    if (sync_reload && !plan.empty())
        for (int l = 0; l < L; ++l)
            if (first_of[(size_t)l] > 0) {
                rc = issue_reload_group(ctx, l, first_of[(size_t)l], plan, d_ids);
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
            if (!sync_reload && !plan.empty() && first_of[(size_t)l] > 0) {
                rc = issue_reload_group(ctx, l, first_of[(size_t)l], plan, d_ids);
                if (rc != PS_OK) return rc;
            }
            cudaEvent_t wait = nullptr;
            if (any_gated) {
                if (!sync_reload)
                    wait = ctx->ev_in[(size_t)ctx->ev_of_layer[(size_t)l]];
                else if (l == 0)
                    wait = ctx->ev_in[(size_t)ctx->ev_of_layer[(size_t)L - 1]];  // the whole reload, once, before the first layer
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

    if (!plan.empty() && !ctx->bk) {  // what ps_reload_backlog reports until these copies have been seen complete
        uint64_t ticket = 0;
        rc = tracker_mark(ctx, ctx->t_scatter, &ticket);
        if (rc != PS_OK) return rc;
        ctx->reload_inflight.push_back({ticket, st.h2d_bytes});
    }

    // 5. request states follow what was issued
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
    st.kernel_launches = (int32_t)(ctx->launches.load() - launches_before);
    if (stats) *stats = st;
    return PS_OK;
}

int32_t ps_step(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs, int32_t batch,
                int64_t copy_budget_bytes, int32_t* decoded_mask, ps_step_stats* stats) {
    if (!ctx) return PS_ERR_INVALID;
    return step_impl(ctx, q_all_layers, out_all_layers, reqs, batch, copy_budget_bytes, nullptr, decoded_mask, stats);
}

int32_t ps_step_ruled(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs, int32_t batch,
                      int64_t copy_budget_bytes, const ps_copy_rule* rule, int32_t* decoded_mask, ps_step_stats* stats) {
    if (!ctx) return PS_ERR_INVALID;
    return step_impl(ctx, q_all_layers, out_all_layers, reqs, batch, copy_budget_bytes, rule, decoded_mask, stats);
}

int32_t ps_reload_backlog(ps_ctx* ctx, int64_t* bytes_in_flight) {
    if (!ctx || !bytes_in_flight) return PS_ERR_INVALID;
    *bytes_in_flight = 0;
    if (ctx->bk) return PS_OK;
    int32_t rc = tracker_poll(ctx, ctx->t_scatter);
    if (rc != PS_OK) return rc;
    while (!ctx->reload_inflight.empty() && ctx->reload_inflight.front().first <= ctx->t_scatter.done)
        ctx->reload_inflight.pop_front();
    for (const auto& e : ctx->reload_inflight) *bytes_in_flight += e.second;
    return PS_OK;
}

int32_t ps_step_host(ps_ctx* ctx, const void* q_host, void* out_host, const int64_t* reqs, int32_t batch,
                     int64_t copy_budget_bytes, int32_t* decoded_mask, ps_step_stats* stats) {
    if (!ctx) return PS_ERR_INVALID;
    if (ctx->bk) return ctx->fail(PS_ERR_INVALID, "ps_step_host: context holds no device (bookkeeping only)");
    if (batch <= 0 || batch > ctx->cfg.max_batch || !q_host || !out_host || !reqs)
        return ctx->fail(PS_ERR_INVALID, "ps_step_host: needs q, out and 1 <= batch <= max_batch");
    const size_t row = (size_t)ctx->cfg.num_q_heads * ctx->cfg.head_dim * 2;
    const size_t bytes = (size_t)ctx->cfg.num_layers * batch * row;
    if (ctx->io_q == nullptr) {  // first use: device buffers for the largest batch
        const size_t cap = (size_t)ctx->cfg.num_layers * ctx->cfg.max_batch * row;
        CK(cudaMalloc((void**)&ctx->io_q, cap));
        cudaError_t e = cudaMalloc((void**)&ctx->io_out, cap);
        if (e != cudaSuccess) {
            cudaFree(ctx->io_q);
            ctx->io_q = nullptr;
            return ctx->fail_cuda(e, "cudaMalloc(step output buffer)");
        }
    }
    CK(cudaMemcpyAsync(ctx->io_q, q_host, bytes, cudaMemcpyHostToDevice, ctx->compute));
    CK(cudaMemsetAsync(ctx->io_out, 0, bytes, ctx->compute));
    int32_t rc = step_impl(ctx, ctx->io_q, ctx->io_out, reqs, batch, copy_budget_bytes, nullptr, decoded_mask, stats);
    if (rc != PS_OK) return rc;
    // The outputs go back through a small kernel that stores into the pinned buffer (16-byte coalesced stores
    // over the host link) when the device can address it: a copy-engine transfer would queue behind every
    // device-to-host copy already submitted, i.e. behind a whole offload in flight, and hold the step for
    // its duration.  Pageable memory takes the copy engine.
    void* out_dev = nullptr;
    if (bytes % 16 == 0 && cudaHostGetDevicePointer(&out_dev, out_host, 0) == cudaSuccess && out_dev != nullptr) {
        CK(ps::launch_upload(out_dev, ctx->io_out, bytes, ctx->compute));
        ctx->launches++;
    } else {
        cudaGetLastError();
        CK(cudaMemcpyAsync(out_host, ctx->io_out, bytes, cudaMemcpyDeviceToHost, ctx->compute));
    }
    return PS_OK;
}

}  // extern "C"
