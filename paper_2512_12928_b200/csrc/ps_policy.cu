// Decisions of Section 4.3 as host arithmetic: adaptive copy budget, eviction policy, partial-copy rule.
#include "ps_ctx.h"

extern "C" {

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
        // The estimated step time after copying B blocks is a step function of B: it jumps up by a request's
        // decode time when the request's last missing block is among the first B.  "B * t_block <= step time"
        // can therefore hold again beyond a point where it fails, and a binary search may stop far below the
        // largest feasible B.  Between two jumps the step time is constant, so the largest feasible B of
        // every such interval is known in closed form; the answer is the largest over the intervals.
        const size_t nq = cum_miss.size();
        for (size_t i = 0; i <= nq; ++i) {  // interval i: the first i queued requests are complete
            const int64_t lo = i == 0 ? 0 : cum_miss[i - 1];
            const int64_t hi = i == nq ? missing : cum_miss[i] - 1;
            if (hi < lo) continue;
            const double t = t_resident + (i == 0 ? 0.0 : cum_time[i - 1]);
            int64_t cand = (int64_t)std::floor(t / t_block);
            while ((double)(cand + 1) * t_block <= t) ++cand;  // the decision is "B * t_block <= t", exactly
            while (cand > 0 && (double)cand * t_block > t) --cand;
            cand = std::min(cand, hi);
            if (cand >= lo && cand > B) B = cand;
        }
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

int32_t ps_order_queue(int32_t n, const double* exec_us, const double* remain_us, const double* weight,
                       const double* waited_us, const ps_sched_params* params, int32_t* order, int32_t* urgent,
                       double* t_budget_us) {
    if (n < 0 || !params || (n > 0 && (!exec_us || !remain_us || !weight || !order))) return PS_ERR_INVALID;
    double t_min = INFINITY, sum_exec = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        if (!(exec_us[i] > 0.0)) return PS_ERR_INVALID;
        t_min = std::min(t_min, remain_us[i]);
        sum_exec += exec_us[i];
    }
    const double t_budget = n > 0 ? std::max(t_min, params->eta_us) : params->eta_us;
    if (t_budget_us) *t_budget_us = t_budget;
    if (n == 0) return PS_OK;
    if (!(t_budget > params->t_c_us)) return PS_ERR_INVALID;
    const double phi = t_budget / (t_budget - params->t_c_us) * sum_exec;
    std::vector<int32_t> cls((size_t)n);  // 2 starving, 1 urgent, 0 normal
    for (int32_t i = 0; i < n; ++i) {
        if (waited_us && waited_us[i] > params->tau_us)
            cls[(size_t)i] = 2;
        else
            cls[(size_t)i] = remain_us[i] < params->gamma * phi ? 1 : 0;
        order[i] = i;
    }
    std::stable_sort(order, order + n, [&](int32_t a, int32_t b) {
        if (cls[(size_t)a] != cls[(size_t)b]) return cls[(size_t)a] > cls[(size_t)b];
        if (cls[(size_t)a] == 1) return weight[a] / exec_us[a] > weight[b] / exec_us[b];
        if (cls[(size_t)a] == 0) return remain_us[a] < remain_us[b];
        return false;
    });
    if (urgent)
        for (int32_t i = 0; i < n; ++i) urgent[i] = cls[(size_t)i];
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

static bool latency_model_ok(const ps_latency_model* m) {
    return m && m->a_p_us >= 0.0 && m->b_p_us >= 0.0 && m->c_p_us >= 0.0 && m->a_d_us >= 0.0 && m->b_d_us >= 0.0 &&
           m->t_c_us >= 0.0;
}

static double prefill_us(const ps_latency_model* m, double l_q, double l_kv) {
    return m->a_p_us * l_q * l_q + m->b_p_us * l_q * l_kv + m->c_p_us * l_q;
}

int32_t ps_estimate_batch(const ps_latency_model* model, int32_t n_prefill, const int32_t* l_q,
                          const int32_t* l_kv_prefill, int32_t n_decode, const int32_t* l_kv_decode,
                          double* batch_us) {
    if (!latency_model_ok(model) || !batch_us || n_prefill < 0 || n_decode < 0) return PS_ERR_INVALID;
    if ((n_prefill > 0 && (!l_q || !l_kv_prefill)) || (n_decode > 0 && !l_kv_decode)) return PS_ERR_INVALID;
    double t = 0.0;
    for (int32_t i = 0; i < n_prefill; ++i) {
        if (l_q[i] < 0 || l_kv_prefill[i] < 0) return PS_ERR_INVALID;
        t += prefill_us(model, (double)l_q[i], (double)l_kv_prefill[i]);
    }
    for (int32_t i = 0; i < n_decode; ++i) {
        if (l_kv_decode[i] < 0) return PS_ERR_INVALID;
        t += model->a_d_us * (double)l_kv_decode[i] + model->b_d_us;
    }
    *batch_us = t + model->t_c_us;
    return PS_OK;
}

int32_t ps_resume_cost(const ps_latency_model* model, int32_t n_tokens, int32_t chunk_tokens, int32_t s_blk,
                       double t_block_us, double* reload_us, double* recompute_us) {
    if (!latency_model_ok(model) || !reload_us || !recompute_us || n_tokens < 0 || chunk_tokens < 0 || s_blk <= 0 ||
        !(t_block_us >= 0.0))
        return PS_ERR_INVALID;
    const int64_t b_miss = ((int64_t)n_tokens + s_blk - 1) / s_blk;
    *reload_us = (double)b_miss * t_block_us;
    const int64_t chunk = chunk_tokens > 0 ? chunk_tokens : n_tokens;
    double t = 0.0;
    for (int64_t done = 0; done < n_tokens; done += chunk) {
        const int64_t l_q = n_tokens - done < chunk ? n_tokens - done : chunk;
        t += prefill_us(model, (double)l_q, (double)done) + model->t_c_us;
    }
    *recompute_us = t;
    return PS_OK;
}

}  // extern "C"
