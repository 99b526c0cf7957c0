// Block gather / scatter kernels: the device half of swap-out and swap-in.
//
// A swapped request's KV lives in scattered slabs (one block of one layer in the K or V pool,
// contiguous, 8-64 KiB).  Offloading gathers them through the block table into a contiguous
// staging range that the copy engine then moves to pinned host memory; reloading scatters a
// staging range that the copy engine filled back into freshly allocated blocks (Section 4.3,
// "Asynchronous Offloading" and "Pipelined Reloading").  Pure byte movement: HBM-bound, 16-byte
// coalesced accesses, several independent loads in flight per thread.
//
// Both directions walk the same "image range": slab s of the range belongs to layer
// layer0 + s / (2 n), logical block (s % (2 n)) / 2 and tensor s & 1 (K, V), where n is the number
// of block ids.  The staging side is contiguous in s; the pool side is pool[layer][tensor] at block
// ids[j].  A block id is the same in every layer, so one id list serves a whole group of layers.
#include "ps_internal.h"

namespace ps {
namespace {

constexpr int kCopyThreads = 256;
constexpr int kCopyUnroll = 4;
constexpr int kPieceVec = kCopyThreads * kCopyUnroll;  // 1024 x 16 B = 16 KiB per CTA

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// Copies vectors [first, first + kPieceVec) ∩ [0, n_vec) of a slab.
__device__ __forceinline__ void copy_piece(const uint4* __restrict__ src, uint4* __restrict__ dst, int first,
                                           int n_vec) {
    uint4 v[kCopyUnroll];
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
        const int i = first + threadIdx.x + u * kCopyThreads;
        if (i < n_vec) v[u] = ld_stream(src + i);
    }
#pragma unroll
    for (int u = 0; u < kCopyUnroll; ++u) {
        const int i = first + threadIdx.x + u * kCopyThreads;
        if (i < n_vec) dst[i] = v[u];
    }
}

// One CTA per 16 KiB piece of a slab.  kScatter = false: pool -> staging; true: staging -> pool.
template <bool kScatter>
__device__ __forceinline__ void image_copy(uint4* const* __restrict__ kpools, uint4* const* __restrict__ vpools,
                                           const int32_t* __restrict__ ids, int32_t n, int32_t layer0,
                                           int64_t slab_begin, uint4* __restrict__ staging, int32_t slab_vec,
                                           int32_t pieces, int32_t num_blocks, int32_t* status) {
    const int64_t local = blockIdx.x / pieces;  // slab inside this launch; staging is addressed from it
    const int piece = blockIdx.x - (int)(local * pieces);
    const int64_t s = slab_begin + local;
    const int64_t per_layer = 2 * (int64_t)n;
    const int l = (int)(s / per_layer);
    const int rem = (int)(s - (int64_t)l * per_layer);
    const int id = ids[rem >> 1];
    if ((unsigned)id >= (unsigned)num_blocks) {
        if (threadIdx.x == 0) *(volatile int32_t*)status = 1;
        return;
    }
    uint4* pool_slab = ((rem & 1) ? vpools[layer0 + l] : kpools[layer0 + l]) + (int64_t)id * slab_vec;
    uint4* stage_slab = staging + local * slab_vec;
    if (kScatter)
        copy_piece(stage_slab, pool_slab, piece * kPieceVec, slab_vec);
    else
        copy_piece(pool_slab, stage_slab, piece * kPieceVec, slab_vec);
}

__global__ void __launch_bounds__(kCopyThreads)
gather_image_kernel(uint4* const* __restrict__ kpools, uint4* const* __restrict__ vpools,
                    const int32_t* __restrict__ ids, int32_t n, int32_t layer0, int64_t slab_begin,
                    uint4* __restrict__ staging, int32_t slab_vec, int32_t pieces, int32_t num_blocks,
                    int32_t* status) {
    image_copy<false>(kpools, vpools, ids, n, layer0, slab_begin, staging, slab_vec, pieces, num_blocks, status);
}

__global__ void __launch_bounds__(kCopyThreads)
scatter_image_kernel(uint4* const* __restrict__ kpools, uint4* const* __restrict__ vpools,
                     const int32_t* __restrict__ ids, int32_t n, int32_t layer0, int64_t slab_begin,
                     uint4* __restrict__ staging, int32_t slab_vec, int32_t pieces, int32_t num_blocks,
                     int32_t* status) {
    image_copy<true>(kpools, vpools, ids, n, layer0, slab_begin, staging, slab_vec, pieces, num_blocks, status);
}

__global__ void __launch_bounds__(256)
upload_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

inline int pieces_for(int32_t slab_vec) { return (slab_vec + kPieceVec - 1) / kPieceVec; }

}  // namespace

cudaError_t launch_image_copy(bool scatter, void* const* d_kpools, void* const* d_vpools, const int32_t* d_ids,
                              int32_t n, int32_t layer0, int64_t slab_begin, int64_t slab_count, void* staging,
                              int32_t slab_vec, int32_t num_blocks, int32_t* d_status, cudaStream_t stream) {
    if (slab_count <= 0) return cudaSuccess;
    if (n <= 0) return cudaErrorInvalidValue;
    const int pieces = pieces_for(slab_vec);
    const int64_t grid = slab_count * pieces;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    if (scatter)
        scatter_image_kernel<<<(unsigned)grid, kCopyThreads, 0, stream>>>(
            (uint4* const*)d_kpools, (uint4* const*)d_vpools, d_ids, n, layer0, slab_begin, (uint4*)staging, slab_vec,
            pieces, num_blocks, d_status);
    else
        gather_image_kernel<<<(unsigned)grid, kCopyThreads, 0, stream>>>(
            (uint4* const*)d_kpools, (uint4* const*)d_vpools, d_ids, n, layer0, slab_begin, (uint4*)staging, slab_vec,
            pieces, num_blocks, d_status);
    return cudaGetLastError();
}

cudaError_t launch_upload(void* dst, const void* src_mapped, size_t bytes, cudaStream_t stream) {
    if (bytes == 0) return cudaSuccess;
    if (bytes % 16) return cudaErrorInvalidValue;
    const int64_t n_vec = (int64_t)(bytes / 16);
    const int64_t want = (n_vec + 255) / 256;
    const unsigned grid = (unsigned)(want < 64 ? want : 64);
    upload_kernel<<<grid, 256, 0, stream>>>((uint4*)dst, (const uint4*)src_mapped, n_vec);
    return cudaGetLastError();
}

}  // namespace ps

// ---- plain streaming kernels for the bandwidth probe -------------------------------------------------
namespace ps {
namespace {

// Every thread streams 16-byte vectors with a grid stride, four loads in flight, and folds them into one
// word that is stored at the end (so the loads cannot be dropped).  kCopy also stores every vector.
template <bool kCopy>
__global__ void __launch_bounds__(256)
stream_probe_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t n_vec, uint32_t* __restrict__ sink) {
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t acc = 0;
    for (; i + 3 * stride < n_vec; i += 4 * stride) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_stream(src + i + u * stride);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (kCopy) dst[i + u * stride] = v[u];
            acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
        }
    }
    for (; i < n_vec; i += stride) {
        const uint4 v = ld_stream(src + i);
        if (kCopy) dst[i] = v;
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
    if (!kCopy) sink[(int64_t)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

}  // namespace

cudaError_t launch_stream_probe(bool copy, const void* src, void* dst, int64_t bytes, uint32_t* sink, int32_t ctas,
                                cudaStream_t stream) {
    if (bytes <= 0 || bytes % 16 || ctas <= 0) return cudaErrorInvalidValue;
    if (copy)
        stream_probe_kernel<true><<<(unsigned)ctas, 256, 0, stream>>>((const uint4*)src, (uint4*)dst, bytes / 16, sink);
    else
        stream_probe_kernel<false><<<(unsigned)ctas, 256, 0, stream>>>((const uint4*)src, (uint4*)dst, bytes / 16, sink);
    return cudaGetLastError();
}

}  // namespace ps
