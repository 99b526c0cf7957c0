// Measurement entry points: gather / scatter kernels alone, pinned-copy host link probe.
#include "ps_ctx.h"

extern "C" {

int32_t ps_copy_blocks(ps_ctx* ctx, int32_t layer, int32_t n_layers, const int32_t* ids, int32_t n_blocks,
                       void* staging, int32_t direction) {
    if (!ctx) return PS_ERR_INVALID;
    if (ctx->bk) return ctx->fail(PS_ERR_INVALID, "ps_copy_blocks: context holds no device (bookkeeping only)");
    if (layer < 0 || n_layers < 1 || layer + n_layers > ctx->cfg.num_layers || !ids || n_blocks < 0 ||
        n_blocks > ctx->cfg.num_gpu_blocks || !staging || (direction != 0 && direction != 1))
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
    const int64_t bytes = (int64_t)n_layers * n_blocks * ctx->layer_block_bytes;
    {
        // the launch swap-out (direction 0) and swap-in (direction 1) make, on the compute stream
        ProfScope prof(ctx, direction == 0 ? kProfGather : kProfScatter, ctx->compute, bytes);
        CK(ps::launch_image_copy(direction == 1, ctx->d_kpools, ctx->d_vpools, d_ids, n_blocks, layer, 0,
                                 2LL * n_blocks * n_layers, staging, ctx->slab_vec, ctx->cfg.num_gpu_blocks, ctx->d_status,
                                 ctx->compute));
    }
    ctx->launches++;
    return PS_OK;
}

int32_t ps_inject_status(ps_ctx* ctx, int32_t value) {
    if (!ctx || !ctx->status) return PS_ERR_INVALID;
    if (value < 1 || value > 3) return ctx->fail(PS_ERR_INVALID, "ps_inject_status: value must be 1, 2 or 3");
    if (value == 3 && !ctx->bk) {
        // what CTAs that gave up leave behind: chunk and arrival counters that were not re-armed
        const size_t done_bytes = (size_t)std::max(ctx->cfg.max_batch, 1) * ctx->cfg.num_kv_heads * sizeof(int32_t);
        for (int i = 0; i < 3; ++i) {
            cudaStream_t st = i == 2 ? ctx->s_lane : ctx->compute;
            if (ctx->d_sched[i]) CK(cudaMemsetAsync(ctx->d_sched[i], 0x01, 4 * sizeof(int32_t), st));
            if (ctx->d_row_done[i]) CK(cudaMemsetAsync(ctx->d_row_done[i], 0x01, done_bytes, st));
        }
    }
    *(volatile int32_t*)ctx->status = value;
    return PS_OK;
}

int32_t ps_hbm_probe(int64_t bytes, int32_t mode, int32_t iters, double* gb_per_s) {
    if (bytes < (1 << 20) || bytes % 16 || iters <= 0 || !gb_per_s || mode < 0 || mode > 1) return PS_ERR_INVALID;
    void *src = nullptr, *dst = nullptr;
    uint32_t* sink = nullptr;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int32_t rc = PS_OK;
    double best = 0.0;
    int dev = 0, sms = 0;
#define CKP(call)                        \
    do {                                 \
        if ((call) != cudaSuccess) {     \
            rc = PS_ERR_CUDA;            \
            create_error() = #call;      \
            goto done;                   \
        }                                \
    } while (0)
    CKP(cudaGetDevice(&dev));
    CKP(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    {
        const int32_t ctas = sms * 8;  // 2048 threads per SM, four 16-byte loads in flight each
        CKP(cudaMalloc(&src, (size_t)bytes));
        CKP(cudaMemset(src, 1, (size_t)bytes));
        if (mode == 1) CKP(cudaMalloc(&dst, (size_t)bytes));
        CKP(cudaMalloc((void**)&sink, (size_t)ctas * 256 * sizeof(uint32_t)));
        CKP(cudaEventCreate(&e0));
        CKP(cudaEventCreate(&e1));
        for (int it = 0; it < iters + 1; ++it) {  // first pass warms up
            CKP(cudaEventRecord(e0, 0));
            CKP(ps::launch_stream_probe(mode == 1, src, dst, bytes, sink, ctas, 0));
            CKP(cudaEventRecord(e1, 0));
            CKP(cudaEventSynchronize(e1));
            float ms = 0.f;
            CKP(cudaEventElapsedTime(&ms, e0, e1));
            if (it > 0 && ms > 0.f) best = std::max(best, (mode == 1 ? 2.0 : 1.0) * (double)bytes / (ms * 1e-3) / 1e9);
        }
        *gb_per_s = best;
    }
done:
#undef CKP
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    if (src) cudaFree(src);
    if (dst) cudaFree(dst);
    if (sink) cudaFree(sink);
    cudaGetLastError();
    return rc;
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
            create_error() = #call;      \
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
