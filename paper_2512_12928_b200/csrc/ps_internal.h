// Internal declarations shared by the runtime and the kernel translation units.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace ps {

// ---- block gather / scatter (swap-out and swap-in kernels) -----------------------------------

// A "slab" is one block of one layer in one pool: slab_vec 16-byte vectors, contiguous.
//
// Image range over n block ids and the layers from layer0 on: slab s lives at layer layer0 + s / (2 n),
// logical block j = (s % (2 n)) / 2, tensor t = s & 1 (0 = K, 1 = V).  The launch moves slabs
// [slab_begin, slab_begin + slab_count) between pool[layer][t] + d_ids[j] * slab and
// staging + (s - slab_begin) * slab: pool -> staging (gather, swap-out) or staging -> pool (scatter,
// swap-in).  d_kpools / d_vpools are device arrays of the per-layer pool pointers, d_ids a device array.
// An id outside [0, num_blocks) sets *d_status to 1 and its slabs are skipped.
cudaError_t launch_image_copy(bool scatter, void* const* d_kpools, void* const* d_vpools, const int32_t* d_ids,
                              int32_t n, int32_t layer0, int64_t slab_begin, int64_t slab_count, void* staging,
                              int32_t slab_vec, int32_t num_blocks, int32_t* d_status, cudaStream_t stream);

// Copies `bytes` (a multiple of 16) between device-addressable ranges with a small kernel: from mapped
// pinned host memory (device view src) to device memory, so that descriptor uploads never queue behind
// bulk transfers in a copy engine, or from device memory into pinned host memory (results of a step).
cudaError_t launch_upload(void* dst, const void* src_mapped, size_t bytes, cudaStream_t stream);

// Streams `bytes` (a multiple of 16) of src with `ctas` CTAs of 256 threads: read-only (every thread folds what
// it read into one word of sink, which holds ctas * 256 words) or as a copy into dst.  For the bandwidth probe.
cudaError_t launch_stream_probe(bool copy, const void* src, void* dst, int64_t bytes, uint32_t* sink, int32_t ctas,
                                cudaStream_t stream);

// ---- paged decode attention --------------------------------------------------------------------

// One split-KV work item: tokens [t_begin, t_end) of batch row b.  `part` indexes the partial
// result slot; `n_parts` is how many items row b has (1 = the kernel writes the final output).
struct AttnItem {
    int32_t b;
    int32_t t_begin;
    int32_t t_end;
    int32_t part;
    int32_t n_parts;
    int32_t pad0, pad1, pad2;
};

struct AttnShape {
    int32_t num_kv_heads, num_q_heads, head_dim, block_size, num_blocks;
};

struct AttnBatch {                 // device pointers to the per-batch metadata
    const int32_t* block_tables;   // [B][table_stride]
    const int32_t* ctx_len;        // [B]
    const AttnItem* items;         // [n_items]
    const int32_t* row_first_part; // [B] first partial slot of the row
    const int32_t* row_parts;      // [B] number of partial slots of the row
    const int32_t* row_lane;       // [B] 0 = main lane, 1 = reload lane (attention waits on reload events)
    const int32_t* cta_begin[2];   // tensor-core kernel: per lane, [n_cta + 1]: first static item of every
                                   // CTA; entry n_cta is where the lane's dynamic chunks start
    int32_t n_cta[2];
    int32_t lane_items[3];         // items of lane 0 are [lane_items[0], lane_items[1]), lane 1 [.. [1], [2])
    int32_t table_stride;
    int32_t batch;
};

// Partial results: per (part, q head): D floats of unnormalised output, then the running max
// (log2 units) and the running sum.  The CUDA-core kernel and the merge kernel use a row stride of
// D + 2 floats, the tensor-core kernel D + 4 (16-byte aligned rows); the buffer is sized for D + 4.
size_t attn_partial_bytes(const AttnShape& sh, int32_t max_parts);

// Launches the attention kernel for the items of one lane.  kernel: 1 = SIMT (one CTA per item and
// KV head; rows with several parts need launch_attn_merge afterwards), 2 = MMA (CTA c of the lane walks
// items [cta_begin[c], cta_begin[c+1]), then takes dynamic chunks through the counters in sched: 2 int32
// per lane, zero before the first launch, re-armed by the kernel itself; rows with several parts are
// combined inside the kernel by whichever warp delivers the last part, counted in row_done:
// batch x num_kv_heads int32, zero before the first launch, re-armed by the kernel).  sched and
// row_done may be null for the SIMT kernel.
// maps: the layer's tensor maps (attn_make_tensor_maps) for the tensor-core kernel, whose tiles then arrive as
// two 32 KiB box copies; null = one 2 KiB bulk copy per token row.
struct AttnTensorMaps {
    alignas(64) unsigned char k[128];
    alignas(64) unsigned char v[128];
};
cudaError_t attn_make_tensor_maps(const AttnShape& sh, const void* kpool, const void* vpool, AttnTensorMaps* out);
cudaError_t launch_decode_attn(int kernel, const AttnShape& sh, const void* kpool, const void* vpool,
                               const AttnTensorMaps* maps, const void* q, void* out, float* lse, const AttnBatch& batch,
                               int32_t lane, float* partials, int32_t* sched, int32_t* row_done, int32_t* d_status,
                               int dep_mode, cudaStream_t stream);
// dep_mode (tensor-core kernel only): 0 = an ordinary launch.  2 = programmatically dependent on whatever kernel
// precedes it on `stream`, the kernel waiting for that kernel's completion right after its own set-up and before
// it reads any input (safe after any predecessor; gains the launch latency and the set-up when the predecessor
// lets dependents start early, as this kernel does).  1 = the previous kernel on `stream` is a launch of the same kernel
// whose inputs and outputs are independent of this one's; the launch is then made programmatically
// dependent on it, so its CTAs start as that launch's CTAs retire.  The kernel waits for its predecessor's
// completion before it first touches partials / sched / row_done, so consecutive launches may even share
// them (the runtime alternates two sets all the same).

// Token granularity of the tensor-core kernel's copies; a context is split at multiples of
// attn_mma_tile_tokens(shape) = 16 * 8 / num_kv_heads tokens (one ring stage).
constexpr int kMmaTileTokens = 16;
int32_t attn_mma_tile_tokens(const AttnShape& sh);

// Merges the partial results of every row with more than one part into out / lse.  lane: 0 or 1
// restricts the merge to the rows of that lane, -1 takes all rows.
cudaError_t launch_attn_merge(const AttnShape& sh, void* out, float* lse, const AttnBatch& batch,
                              const float* partials, int32_t lane, cudaStream_t stream);

// Whether the tensor-core kernel supports the shape.
bool attn_mma_supported(const AttnShape& sh);

// One-time per-process kernel attribute set-up (dynamic shared memory opt-in).
cudaError_t attn_init();

}  // namespace ps
