// Block gather / scatter kernels: the device half of swap-out and swap-in.
//
// A swapped request's KV lives in scattered slabs (one block of one layer in the K or V pool,
// contiguous, 8-64 KiB).  Offloading gathers them through the block table into a contiguous
// staging range that the copy engine then moves to pinned host memory; reloading scatters a
// staging range that the copy engine filled back into freshly allocated blocks (Section 4.3,
// "Asynchronous Offloading" and "Pipelined Reloading").  Pure byte movement: HBM-bound, 16-byte
// coalesced accesses, several independent loads in flight per thread.
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

__global__ void __launch_bounds__(kCopyThreads)
gather_image_kernel(const uint4* const* __restrict__ kpools, const uint4* const* __restrict__ vpools,
                    const int32_t* __restrict__ table, int32_t n_blk, int64_t slab_begin, uint4* __restrict__ dst,
                    int32_t slab_vec, int32_t pieces, int32_t num_blocks, int32_t* status) {
    const int64_t local = blockIdx.x / pieces;
    const int piece = blockIdx.x - (int)(local * pieces);
    const int64_t s = slab_begin + local;
    const int64_t per_layer = 2 * (int64_t)n_blk;
    const int l = (int)(s / per_layer);
    const int rem = (int)(s - (int64_t)l * per_layer);
    const int j = rem >> 1;
    const int id = table[j];
    if ((unsigned)id >= (unsigned)num_blocks) {
        if (threadIdx.x == 0) *(volatile int32_t*)status = 1;
        return;
    }
    const uint4* pool = (rem & 1) ? vpools[l] : kpools[l];
    copy_piece(pool + (int64_t)id * slab_vec, dst + local * slab_vec, piece * kPieceVec, slab_vec);
}

// kScatter = false: pool -> pairs; true: pairs -> pool.
template <bool kScatter>
__global__ void __launch_bounds__(kCopyThreads)
layer_copy_kernel(uint4* __restrict__ kpool, uint4* __restrict__ vpool, const int32_t* __restrict__ ids,
                  uint4* __restrict__ pairs, int32_t slab_vec, int32_t pieces, int32_t num_blocks, int32_t* status) {
    const int local = blockIdx.x / pieces;  // slab index inside the pair array: 2 i + t
    const int piece = blockIdx.x - local * pieces;
    const int id = ids[local >> 1];
    if ((unsigned)id >= (unsigned)num_blocks) {
        if (threadIdx.x == 0) *(volatile int32_t*)status = 1;
        return;
    }
    uint4* pool_slab = ((local & 1) ? vpool : kpool) + (int64_t)id * slab_vec;
    uint4* pair_slab = pairs + (int64_t)local * slab_vec;
    if (kScatter)
        copy_piece(pair_slab, pool_slab, piece * kPieceVec, slab_vec);
    else
        copy_piece(pool_slab, pair_slab, piece * kPieceVec, slab_vec);
}

struct ParamIds {
    int32_t ids[kMaxParamIds];
};

__global__ void __launch_bounds__(kCopyThreads)
scatter_param_ids_kernel(uint4* __restrict__ kpool, uint4* __restrict__ vpool, const __grid_constant__ ParamIds ids,
                         const uint4* __restrict__ pairs, int32_t slab_vec, int32_t pieces, int32_t num_blocks,
                         int32_t* status) {
    const int local = blockIdx.x / pieces;
    const int piece = blockIdx.x - local * pieces;
    const int id = ids.ids[local >> 1];
    if ((unsigned)id >= (unsigned)num_blocks) {
        if (threadIdx.x == 0) *(volatile int32_t*)status = 1;
        return;
    }
    uint4* pool_slab = ((local & 1) ? vpool : kpool) + (int64_t)id * slab_vec;
    copy_piece(pairs + (int64_t)local * slab_vec, pool_slab, piece * kPieceVec, slab_vec);
}

__global__ void __launch_bounds__(256)
upload_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, int64_t n_vec) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

inline int pieces_for(int32_t slab_vec) { return (slab_vec + kPieceVec - 1) / kPieceVec; }

}  // namespace

cudaError_t launch_gather_image(const void* const* d_kpools, const void* const* d_vpools, const int32_t* d_table,
                                int32_t n_blk, int64_t slab_begin, int64_t slab_count, void* dst, int32_t slab_vec,
                                int32_t num_blocks, int32_t* d_status, cudaStream_t stream) {
    if (slab_count <= 0) return cudaSuccess;
    const int pieces = pieces_for(slab_vec);
    const int64_t grid = slab_count * pieces;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    gather_image_kernel<<<(unsigned)grid, kCopyThreads, 0, stream>>>(
        (const uint4* const*)d_kpools, (const uint4* const*)d_vpools, d_table, n_blk, slab_begin, (uint4*)dst,
        slab_vec, pieces, num_blocks, d_status);
    return cudaGetLastError();
}

cudaError_t launch_scatter_layer(void* kpool, void* vpool, const int32_t* d_ids, int32_t n, const void* src,
                                 int32_t slab_vec, int32_t num_blocks, int32_t* d_status, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    const int pieces = pieces_for(slab_vec);
    const int64_t grid = 2LL * n * pieces;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    layer_copy_kernel<true><<<(unsigned)grid, kCopyThreads, 0, stream>>>(
        (uint4*)kpool, (uint4*)vpool, d_ids, (uint4*)const_cast<void*>(src), slab_vec, pieces, num_blocks, d_status);
    return cudaGetLastError();
}

cudaError_t launch_scatter_layer_ids(void* kpool, void* vpool, const int32_t* h_ids, int32_t n, const void* src,
                                     int32_t slab_vec, int32_t num_blocks, int32_t* d_status, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    if (n > kMaxParamIds) return cudaErrorInvalidValue;
    ParamIds ids;
    for (int32_t i = 0; i < n; ++i) ids.ids[i] = h_ids[i];
    for (int32_t i = n; i < kMaxParamIds; ++i) ids.ids[i] = 0;
    const int pieces = pieces_for(slab_vec);
    const int64_t grid = 2LL * n * pieces;
    scatter_param_ids_kernel<<<(unsigned)grid, kCopyThreads, 0, stream>>>(
        (uint4*)kpool, (uint4*)vpool, ids, (const uint4*)src, slab_vec, pieces, num_blocks, d_status);
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

cudaError_t launch_gather_layer(const void* kpool, const void* vpool, const int32_t* d_ids, int32_t n, void* dst,
                                int32_t slab_vec, int32_t num_blocks, int32_t* d_status, cudaStream_t stream) {
    if (n <= 0) return cudaSuccess;
    const int pieces = pieces_for(slab_vec);
    const int64_t grid = 2LL * n * pieces;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidValue;
    layer_copy_kernel<false><<<(unsigned)grid, kCopyThreads, 0, stream>>>(
        (uint4*)const_cast<void*>(kpool), (uint4*)const_cast<void*>(vpool), d_ids, (uint4*)dst, slab_vec, pieces,
        num_blocks, d_status);
    return cudaGetLastError();
}

}  // namespace ps
