// ps_decode_attn_static: paged decode attention for callers that must not allocate.
//
// Some hosts of this library cannot call cudaMalloc at the point where they need attention: an
// engine that has handed all device memory to its own pool allocator at start-up, a plug-in that
// runs inside somebody else's memory budget, a real-time loop where an allocation (which may
// synchronise the whole device) is forbidden.  The context-based entry point ps_decode_attn gets
// its split-KV scratch (partial results, work-item list) from cudaMalloc'ed buffers made by
// ps_create.  This variant keeps that scratch in one fixed array that is part of the library image
// itself, so it needs no context and makes no allocation of any kind: the caller passes the pools,
// the queries, the block tables and the output, and that is all the memory involved.
//
// The price: the array has a fixed, modest size (kScratchBytes, about 16 MiB, resident on every GPU
// that loads the library until the process exits), every call on a device uses the same array, and
// two calls whose kernels may overlap on the GPU (different streams without an ordering between
// them) would overwrite each other's partial results.  Calls on one stream are safe back to back.
//
// The array's name is only a host-side handle in host code; the device address is looked up once
// per device with cudaGetSymbolAddress (with that device current) and cached.  That look-up happens
// inside the first call on a device, which therefore should be made before any stream capture
// begins.
//
// The kernels are the library's CUDA-core attention and merge kernels, unchanged; only the source
// of the scratch differs, and the work-item list is built by a small kernel on the device from the
// context lengths, which travel as kernel parameters.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>

#include "ps_internal.h"
#include "ps_kvswap.h"

namespace {

constexpr int kMaxBatch = PS_STATIC_MAX_BATCH;
constexpr int kMaxItems = 4096;
constexpr size_t kOffStatus = 0;                                   // one word, 256 bytes reserved
constexpr size_t kOffCtx = 256;                                    // int32[kMaxBatch]
constexpr size_t kOffFirst = kOffCtx + 4 * kMaxBatch;              // int32[kMaxBatch]
constexpr size_t kOffParts = kOffFirst + 4 * kMaxBatch;            // int32[kMaxBatch]
constexpr size_t kOffLane = kOffParts + 4 * kMaxBatch;             // int32[kMaxBatch], all zero
constexpr size_t kOffItems = kOffLane + 4 * kMaxBatch;             // AttnItem[kMaxItems]
constexpr size_t kMetaBytes = 192 << 10;
constexpr size_t kPartialBytes = PS_STATIC_SCRATCH_BYTES - kMetaBytes;
constexpr size_t kScratchBytes = PS_STATIC_SCRATCH_BYTES;
static_assert(kOffItems + kMaxItems * sizeof(ps::AttnItem) <= kMetaBytes, "metadata region too small");
static_assert(kMetaBytes % 256 == 0, "partials start on a 256-byte boundary");

// The scratch itself.  Device code in this file may name it; host code must go through the address
// that cudaGetSymbolAddress returns.
static __device__ __align__(256) unsigned char g_attn_scratch[kScratchBytes];

struct CtxLens {
    int32_t v[kMaxBatch];
};

// One CTA.  Rebuilds the whole metadata region for this call: nothing of the previous call's
// metadata survives, and the status word starts at zero.  Row b is cut into ceil(ctx/split) items
// (one item for an empty row, which then writes the zero output).
__global__ void __launch_bounds__(kMaxBatch)
static_plan_kernel(const __grid_constant__ CtxLens ctx, int32_t batch, int32_t split, unsigned char* scratch) {
    __shared__ int32_t first[kMaxBatch];
    int32_t* d_status = reinterpret_cast<int32_t*>(scratch + kOffStatus);
    int32_t* d_ctx = reinterpret_cast<int32_t*>(scratch + kOffCtx);
    int32_t* d_first = reinterpret_cast<int32_t*>(scratch + kOffFirst);
    int32_t* d_parts = reinterpret_cast<int32_t*>(scratch + kOffParts);
    int32_t* d_lane = reinterpret_cast<int32_t*>(scratch + kOffLane);
    ps::AttnItem* d_items = reinterpret_cast<ps::AttnItem*>(scratch + kOffItems);
    const int b = threadIdx.x;
    if (b == 0) {
        *d_status = 0;
        int32_t acc = 0;
        for (int i = 0; i < batch; ++i) {
            first[i] = acc;
            const int32_t n = ctx.v[i] > 0 ? (ctx.v[i] + split - 1) / split : 1;
            acc += n;
        }
    }
    __syncthreads();
    if (b >= batch) return;
    const int32_t len = ctx.v[b];
    const int32_t n = len > 0 ? (len + split - 1) / split : 1;
    d_ctx[b] = len;
    d_first[b] = first[b];
    d_parts[b] = n;
    d_lane[b] = 0;
    for (int32_t k = 0; k < n; ++k) {
        ps::AttnItem it;
        it.b = b;
        it.t_begin = k * split;
        it.t_end = min(len, (k + 1) * split);
        it.part = first[b] + k;
        it.n_parts = n;
        it.pad0 = it.pad1 = it.pad2 = 0;
        d_items[first[b] + k] = it;
    }
}

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};

int32_t fail(char* err_buf, int32_t err_cap, int32_t code, const char* msg) {
    if (err_buf && err_cap > 0) {
        snprintf(err_buf, (size_t)err_cap, "%s", msg);
    }
    return code;
}

// Device address of the scratch on the current device: looked up once per device, then cached.
cudaError_t scratch_on_current_device(unsigned char** out, int* dev_out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_attn_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    *dev_out = dev;
    return cudaSuccess;
}

}  // namespace

extern "C" int32_t ps_decode_attn_static(const void* kpool, const void* vpool, const void* q, void* out, float* lse,
                                         const int32_t* block_tables, int32_t table_stride, const int32_t* ctx_lens,
                                         int32_t batch, int32_t num_kv_heads, int32_t num_q_heads, int32_t head_dim,
                                         int32_t block_size, int32_t num_gpu_blocks, int32_t kv_split_tokens,
                                         int32_t* status_word, void* stream, char* err_buf, int32_t err_cap) {
    if (err_buf && err_cap > 0) err_buf[0] = 0;
    if (batch == 0) return PS_OK;
    if (!kpool || !vpool || !q || !out || !block_tables || !ctx_lens || batch < 0 || table_stride <= 0 ||
        num_kv_heads <= 0 || num_q_heads <= 0 || block_size <= 0 || num_gpu_blocks <= 0 || kv_split_tokens < 0)
        return fail(err_buf, err_cap, PS_ERR_INVALID, "ps_decode_attn_static: null pointer or non-positive size");
    if (num_q_heads % num_kv_heads != 0)
        return fail(err_buf, err_cap, PS_ERR_INVALID, "ps_decode_attn_static: num_q_heads must be a multiple of num_kv_heads");
    const int G = num_q_heads / num_kv_heads;
    if ((head_dim != 64 && head_dim != 128) || G < 1 || G > 8)
        return fail(err_buf, err_cap, PS_ERR_INVALID,
                    "ps_decode_attn_static: unsupported shape (head_dim 64 or 128, Hq/Hkv from 1 to 8)");
    char msg[400];
    if (batch > kMaxBatch) {
        snprintf(msg, sizeof msg, "ps_decode_attn_static: batch %d exceeds the fixed maximum of %d", batch, kMaxBatch);
        return fail(err_buf, err_cap, PS_ERR_INVALID, msg);
    }
    int64_t total_tokens = 0;
    for (int32_t b = 0; b < batch; ++b) {
        if (ctx_lens[b] < 0) return fail(err_buf, err_cap, PS_ERR_INVALID, "ps_decode_attn_static: negative context length");
        if (((int64_t)ctx_lens[b] + block_size - 1) / block_size > table_stride)
            return fail(err_buf, err_cap, PS_ERR_INVALID,
                        "ps_decode_attn_static: a context needs more blocks than table_stride holds");
        total_tokens += ctx_lens[b];
    }
    int64_t split = kv_split_tokens;
    if (split == 0) {  // about 2048 CTAs (items x KV heads) whatever the context mix
        const int64_t target_items = 2048 / num_kv_heads > 0 ? 2048 / num_kv_heads : 1;
        split = (total_tokens + target_items - 1) / target_items;
        split = (split + 63) / 64 * 64;
        if (split < 256) split = 256;
    }
    if (split > (1 << 30)) split = 1 << 30;
    int64_t n_items = 0;
    bool any_multi = false;
    for (int32_t b = 0; b < batch; ++b) {
        const int64_t n = ctx_lens[b] > 0 ? (ctx_lens[b] + split - 1) / split : 1;
        n_items += n;
        any_multi |= n > 1;
    }
    const ps::AttnShape sh{num_kv_heads, num_q_heads, head_dim, block_size, num_gpu_blocks};
    if (n_items > kMaxItems || ps::attn_partial_bytes(sh, (int32_t)n_items) > kPartialBytes) {
        snprintf(msg, sizeof msg,
                 "ps_decode_attn_static: %lld work items (%zu bytes of partial results) exceed the fixed scratch "
                 "(%d items, %zu bytes); use a larger kv_split_tokens or a smaller batch",
                 (long long)n_items, ps::attn_partial_bytes(sh, (int32_t)std::min<int64_t>(n_items, 1 << 24)), kMaxItems,
                 kPartialBytes);
        return fail(err_buf, err_cap, PS_ERR_INVALID, msg);
    }

    unsigned char* scratch = nullptr;
    int dev = -1;
    cudaError_t e = scratch_on_current_device(&scratch, &dev);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof msg, "ps_decode_attn_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        cudaGetLastError();
        return fail(err_buf, err_cap, PS_ERR_CUDA, msg);
    }
    cudaStream_t s = (cudaStream_t)stream;
    CtxLens cl;
    memset(&cl, 0, sizeof cl);
    memcpy(cl.v, ctx_lens, sizeof(int32_t) * (size_t)batch);
    static_plan_kernel<<<1, kMaxBatch, 0, s>>>(cl, batch, (int32_t)split, scratch);
    e = cudaGetLastError();
    ps::AttnBatch ab{};
    ab.block_tables = block_tables;
    ab.ctx_len = reinterpret_cast<const int32_t*>(scratch + kOffCtx);
    ab.row_first_part = reinterpret_cast<const int32_t*>(scratch + kOffFirst);
    ab.row_parts = reinterpret_cast<const int32_t*>(scratch + kOffParts);
    ab.row_lane = reinterpret_cast<const int32_t*>(scratch + kOffLane);
    ab.items = reinterpret_cast<const ps::AttnItem*>(scratch + kOffItems);
    ab.lane_items[0] = 0;
    ab.lane_items[1] = ab.lane_items[2] = (int32_t)n_items;
    ab.table_stride = table_stride;
    ab.batch = batch;
    float* partials = reinterpret_cast<float*>(scratch + kMetaBytes);
    int32_t* status = status_word ? status_word : reinterpret_cast<int32_t*>(scratch + kOffStatus);
    if (e == cudaSuccess)
        e = ps::launch_decode_attn(/*SIMT kernel*/ 1, sh, kpool, vpool, nullptr, q, out, lse, ab, 0, partials, nullptr, nullptr, status, false, s);
    if (e == cudaSuccess && any_multi) e = ps::launch_attn_merge(sh, out, lse, ab, partials, -1, s);
    if (e != cudaSuccess) {
        snprintf(msg, sizeof msg, "ps_decode_attn_static: kernel launch: %s", cudaGetErrorString(e));
        return fail(err_buf, err_cap, PS_ERR_CUDA, msg);
    }
    return PS_OK;
}
