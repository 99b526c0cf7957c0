/*
 * ps_kvswap.h -- C ABI of the KV-block swap / paged decode library (single GPU, sm_100a).
 *
 * The calls implement the data path underneath ProServe's engine-layer block management
 * (Section 4.3 "Efficient Block Management"; Appendix B "Implementation Details"):
 *   - a device pool of M KV blocks of s_blk tokens with a free count b_f (Section 4.3, App. A),
 *   - asynchronous offloading of a preempted request's blocks to host memory on a copy stream,
 *     the device blocks being reclaimable only once the transfer has completed,
 *   - pipelined reloading: host-to-device copies on a dedicated copy stream, one completion
 *     event per layer chunk, the compute stream waiting on a chunk's event only before it
 *     runs that chunk,
 *   - a per-step host-to-device copy budget B_copy consumed in queue order at request
 *     granularity, partially for the request that does not fit (Alg. 1: GetCopyBudget, ConsumeCopyBudget),
 *   - the decode forward the reload overlaps with, here its KV-consuming part: paged
 *     grouped-query attention over the block table.
 * Which request to evict and how large the budget should be are scheduler decisions and stay
 * with the caller.
 *
 * Conventions
 *   - Every function returns a ps_status (0 = PS_OK, negative = error).  On error nothing is
 *     partially applied (allocation is all-or-nothing).  No function throws or aborts.
 *   - "device pointer" = address in the memory of the CUDA device that was current when
 *     ps_create was called; "host pointer" = ordinary process memory unless it says pinned.
 *   - One caller thread per context (the context runs one worker thread of its own, for offloads).  All GPU work is asynchronous with respect to the host
 *     unless a function says it waits.  Asynchronous CUDA failures surface as PS_ERR_CUDA (and
 *     kernel-side id checks as PS_ERR_BOUNDS, a kernel-side wait that ran out as PS_ERR_TIMEOUT) from the
 *     next ps_poll / ps_sync / ps_step.
 *   - Layouts.  bf16 everywhere.  Per layer there is one K pool and one V pool, each
 *     [num_gpu_blocks][block_size][num_kv_heads][head_dim]; the "slab" of a block is its
 *     block_size*num_kv_heads*head_dim contiguous elements in one pool.  The host image of a
 *     swapped-out request with n blocks is [num_layers][n][2 (K,V)][block_size][num_kv_heads]
 *     [head_dim]: for one layer, a run of logical blocks is one contiguous byte range.
 *   - The KV pools and the compute stream belong to the caller and must outlive the context.
 *     The context owns its copy streams, events, staging buffers, descriptor buffers, attention
 *     scratch and (unless one is passed in) the pinned host pool.
 */
#ifndef PS_KVSWAP_H
#define PS_KVSWAP_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ps_ctx ps_ctx;

enum ps_status {
    PS_OK = 0,
    PS_ERR_INVALID = -1,     /* bad argument, unknown request, unsupported shape */
    PS_ERR_NOMEM = -2,       /* not enough free device blocks */
    PS_ERR_HOST_NOMEM = -3,  /* host pool cannot hold the image */
    PS_ERR_STATE = -4,       /* request is in the wrong state for this call */
    PS_ERR_BUSY = -5,        /* a transfer of this request is still in flight */
    PS_ERR_TIMEOUT = -6,     /* a bounded wait ran out: ps_sync's on the host, or one inside the attention
                                kernel (then the launches in flight produced undefined outputs) */
    PS_ERR_CUDA = -7,        /* a CUDA call failed; see ps_last_error */
    PS_ERR_BOUNDS = -8       /* a kernel met a block id outside the pool and skipped it */
};

enum ps_req_state {
    PS_REQ_NONE = 0,
    PS_REQ_RESIDENT = 1,      /* all blocks on the device (may still be gated on reload events) */
    PS_REQ_SWAPPING_OUT = 2,  /* offload in flight; blocks still owned */
    PS_REQ_HOST = 3,          /* image on host; owns no device block */
    PS_REQ_SWAPPING_IN = 4    /* queued for / in the middle of a reload; owns fresh blocks */
};

enum ps_flags {
    /* Block tables, states, budget plans and error codes only: no CUDA call is made, no byte is
       moved, transfers "complete" at once.  For host-logic tests on machines without a GPU;
       ps_decode_attn and the q/out arguments of ps_step are rejected in this mode. */
    PS_FLAG_BOOKKEEPING_ONLY = 1,
    /* Record CUDA events around every kernel and transfer so that ps_get_profile can report
       per-kind device times.  Costs two event records per launch; while a host transfer saturates
       the link these records delay the compute stream's commands noticeably (a decode step grew
       from 3.8 to 6.4 ms in one measurement), so use it for diagnosis, not inside timed runs. */
    PS_FLAG_PROFILE = 2,
    /* Ablation (Section 5, block-management ablation "w/o async"): ps_step finishes the whole
       reload before the first attention launch instead of pipelining it layer by layer. */
    PS_FLAG_SYNC_RELOAD = 4,
    /* By default ps_decode_attn (one layer per call) launches the tensor-core kernel programmatically
       dependent on the kernel that precedes it on the compute stream: its CTAs are scheduled and set up
       under that kernel's tail and wait for its completion before they read the queries, the KV pools or the
       batch metadata.  Results are the same after any predecessor; time is gained only after kernels that
       let dependents start early (this library's attention kernel does; an engine's own kernels may, with
       cudaTriggerProgrammaticLaunchCompletion).  This flag turns that off: an ordinary launch, for
       comparison and diagnosis. */
    PS_FLAG_ATTN_PLAIN_LAUNCH = 8
};

enum ps_attn_kernel {
    PS_ATTN_AUTO = 0,
    PS_ATTN_SIMT = 1,   /* CUDA-core kernel, warp-shuffle softmax; any supported shape */
    PS_ATTN_MMA = 2,    /* tensor-core kernel (head_dim 128; 1, 2, 4 or 8 KV heads): tiles staged by tensor-map
                           box copies when the driver accepts the maps, else (8 KV heads) as PS_ATTN_MMA_ROWS */
    PS_ATTN_MMA_ROWS = 3 /* the same kernel with one bulk copy per token row (8 KV heads only) */
};

typedef struct ps_config {
    int32_t num_layers;          /* L */
    int32_t num_kv_heads;        /* Hkv */
    int32_t num_q_heads;         /* Hq, a multiple of Hkv; group G = Hq/Hkv from 1 to 8 */
    int32_t head_dim;            /* D in {64, 128} */
    int32_t block_size;          /* s_blk, tokens per block */
    int32_t num_gpu_blocks;      /* M, blocks in every per-layer pool */
    int32_t max_blocks_per_req;  /* longest block table */
    int32_t max_batch;           /* largest decode batch passed to ps_decode_attn / ps_step */
    int32_t flags;               /* OR of ps_flags */
    int32_t attn_kernel;         /* ps_attn_kernel */
    int32_t kv_split_tokens;     /* tokens per split-KV work item; 0 = chosen per batch */
    int32_t layer_chunk_bytes;   /* ps_step reloads in layer chunks (Appendix B: one completion event per layer
                                    chunk): consecutive layers share one host copy, one scatter launch and one
                                    event until the chunk carries this many bytes, because a single layer's share
                                    of a small copy budget is too small for the copy engine to reach link rate.
                                    0 = 2 MiB; negative = always one layer per chunk */
    int64_t host_pool_bytes;     /* capacity for host images */
    int64_t staging_bytes;       /* device staging per direction (split into 4 slots); 0 = 256 MiB */
    const int32_t* initial_free_order; /* host pointer to a permutation of 0..M-1: the order in
                                          which block ids are first handed out; NULL = 0,1,2,.. */
} ps_config;

typedef struct ps_step_stats {
    int64_t h2d_bytes;          /* reload bytes issued by this step */
    int64_t blocks_copied;      /* blocks (all layers) issued by this step */
    int32_t reloads_completed;  /* requests whose last missing block was issued by this step */
    int32_t swapouts_reaped;    /* offloads found complete; their blocks went back to the pool */
    int32_t decoded;            /* requests that ran attention in this step */
    int32_t gated;              /* of those, requests whose attention waited on reload events */
    int32_t kernel_launches;    /* kernels of this library launched by this step */
    int32_t reserved0;
} ps_step_stats;

typedef struct ps_profile {
    double attn_ms;     int64_t attn_launches;     int64_t attn_kv_bytes;   /* K+V bytes addressed */
    double merge_ms;    int64_t merge_launches;
    double gather_ms;   int64_t gather_launches;   int64_t gather_bytes;    /* payload bytes (read once, written once) */
    double scatter_ms;  int64_t scatter_launches;  int64_t scatter_bytes;
    double d2h_ms;      int64_t d2h_copies;        int64_t d2h_bytes;
    double h2d_ms;      int64_t h2d_copies;        int64_t h2d_bytes;
} ps_profile;

/* One timed span of the trace: what ran, for which layer, and when (microseconds after ps_trace
 * was switched on, device clock).  kind: 0 attention, 1 split-KV merge, 2 gather, 3 scatter,
 * 4 device-to-host copy, 5 host-to-device copy.  tag: the layer (attention launches that waited on
 * a reload event carry 1000 + layer), or -1. */
typedef struct ps_trace_span {
    int32_t kind;
    int32_t tag;
    float start_us;
    float end_us;
} ps_trace_span;

/* ---- context ---------------------------------------------------------------------------- */

/* Creates a context on the current CUDA device.
 *   k_pools, v_pools : host arrays of num_layers device pointers (the per-layer pools above).
 *   host_pool        : pinned host memory of host_pool_bytes, or NULL to let the library pin its own.
 *   compute_stream   : the caller's cudaStream_t (0 = legacy default stream) on which attention
 *                      runs and against which block reuse is ordered.
 * The first allocation order of block ids is initial_free_order; afterwards the pool is a LIFO
 * stack: ps_kv_alloc pops one id at a time, a release pushes a table's ids in table order.
 * Errors: PS_ERR_INVALID (shape outside the supported set, bad permutation), PS_ERR_CUDA,
 * PS_ERR_HOST_NOMEM (pinning failed). */
int32_t ps_create(const ps_config* cfg, void* const* k_pools, void* const* v_pools, void* host_pool,
                  void* compute_stream, ps_ctx** out);

/* Waits up to 10 s for the context's outstanding work (as ps_sync does); if that runs out, waits for its
 * streams and the compute stream without a limit, so that no staging slot or pinned range is freed under a
 * copy still queued.  Frees everything the context owns either way; returns PS_ERR_TIMEOUT if the bounded
 * wait ran out, else PS_OK.  The pools and the compute stream stay the caller's. */
int32_t ps_destroy(ps_ctx* ctx);

/* Text of the most recent error of this context (static storage inside the context; never NULL).
   With ctx == NULL: the most recent ps_create failure. */
const char* ps_last_error(const ps_ctx* ctx);

/* ---- block pool (Section 4.3: pool of M blocks, b_f free; per-request b_device) ---------- */

/* Grows request `req` (created on first use) so that it can hold n_tokens_total tokens, i.e. to
 * ceil(n_tokens_total / block_size) blocks.  All-or-nothing.  Only RESIDENT requests grow.
 * Errors: PS_ERR_NOMEM, PS_ERR_STATE, PS_ERR_INVALID (shrinking, table would exceed
 * max_blocks_per_req). */
int32_t ps_kv_alloc(ps_ctx* ctx, int64_t req, int32_t n_tokens_total);

/* Forgets the request.  RESIDENT: its blocks go back to the pool; HOST: its image is released.
 * PS_ERR_BUSY while a transfer of it is in flight (SWAPPING_OUT, SWAPPING_IN, or a reload whose
 * copies have not been seen complete yet). */
int32_t ps_kv_free(ps_ctx* ctx, int64_t req);

/* Copies the request's block table into out_ids (host, capacity cap; may be NULL with cap 0) and
 * reports its length, state (ps_req_state) and token count.  Any out pointer may be NULL. */
int32_t ps_block_table(ps_ctx* ctx, int64_t req, int32_t* out_ids, int32_t cap, int32_t* n_blocks,
                       int32_t* state, int32_t* n_tokens);

int32_t ps_num_free_blocks(ps_ctx* ctx, int32_t* out);

/* ---- swap-out (Section 4.3 "Asynchronous Offloading"; App. B: D2H on a separate stream) --- */

/* Starts the offload of a RESIDENT request: its blocks, every layer, are gathered through the
 * block table into device staging and copied to a host image, ordered after all work already
 * enqueued on the compute stream.  Returns at once; the request is SWAPPING_OUT and still owns
 * its blocks.  When a later ps_poll / ps_step / ps_sync finds the transfer complete (offloads
 * complete in issue order) the blocks are pushed back to the pool and the state becomes HOST.
 * Blocks already covered by ps_offload_progress are not copied again.
 * The copies are handed to the copy engine by a worker thread of the context, two staging slots at a time
 * (Section 4.3: a separate thread copies the accumulated blocks).  The engine serves device-to-host copies in
 * submission order whatever their stream, so an offload submitted whole would hold every later copy of the
 * process -- a step's results, sampled tokens -- for its full duration; paced, such a copy waits behind at most
 * two slots.  A failure inside the worker surfaces as PS_ERR_CUDA from the next ps_poll / ps_step / ps_sync.
 * Errors: PS_ERR_STATE, PS_ERR_HOST_NOMEM, PS_ERR_INVALID, PS_ERR_CUDA. */
int32_t ps_swap_out(ps_ctx* ctx, int64_t req);

/* Proactive incremental offloading (Section 4.3 "Asynchronous Offloading"): offloads a request's filled blocks
 * in groups of n_off ahead of any eviction; the caller passes a smaller n_off for requests it expects to
 * preempt sooner.  If the RESIDENT request has at least n_off blocks that are completely filled
 * (n_tokens / block_size) and not yet offloaded, the largest whole number of groups of n_off such blocks
 * is copied to the host as a new image segment, asynchronously and ordered after the work already
 * enqueued on the compute stream; the request stays RESIDENT and keeps decoding and growing.  Filled
 * blocks must not be rewritten afterwards (decode only appends).  *issued_blocks (may be NULL) = blocks
 * issued by this call, possibly 0.  A later ps_swap_out then only offloads the remaining tail (the paper
 * drops that tail and recomputes it on resume; this path has no recomputation, so it is copied), which
 * shortens the time until the device blocks can be reclaimed.  Which n_off to use is the caller's policy.
 * Errors: PS_ERR_STATE, PS_ERR_INVALID, PS_ERR_HOST_NOMEM, PS_ERR_CUDA. */
int32_t ps_offload_progress(ps_ctx* ctx, int64_t req, int32_t n_off, int32_t* issued_blocks);

/* ps_offload_progress for a whole batch, e.g. once after every decode step: request reqs[i] with its own
 * threshold n_off[i] (the paper's n_off^r: smaller for lower-priority requests, which are more likely to be
 * preempted).  Entries that are unknown or not RESIDENT are skipped.  *issued_blocks (may be NULL) = blocks
 * issued over the batch.  The entries are taken in order and the call stops at the first failing one
 * (typically PS_ERR_HOST_NOMEM): copies issued for earlier entries stay issued, the failing entry and the
 * later ones are untouched.
 * Errors: PS_ERR_INVALID (null arrays with batch > 0, a non-positive threshold), and those of
 * ps_offload_progress. */
int32_t ps_offload_sweep(ps_ctx* ctx, const int64_t* reqs, const int32_t* n_off, int32_t batch,
                         int64_t* issued_blocks);

/* b_host of Section 4.3 for one request: blocks whose offload has been issued, and blocks whose copy has
 * been seen complete (as of the last ps_poll / ps_step / ps_sync).  Either pointer may be NULL. */
int32_t ps_host_blocks(ps_ctx* ctx, int64_t req, int32_t* issued, int32_t* on_host);

/* Host address and size of a HOST / SWAPPING_IN request's image (valid until the reload completes
 * or the request is freed).  For checks; the bytes are final only once the state is HOST.
 * PS_ERR_STATE when the image consists of several segments (proactive offloading). */
int32_t ps_host_image(ps_ctx* ctx, int64_t req, void** ptr, int64_t* bytes);

/* Segment `index` of a request's host image: logical blocks [*blk_lo, *blk_hi) in the layout
 * [num_layers][blk_hi - blk_lo][2 (K,V)][slab].  *n_segments receives the number of segments; index -1
 * asks for the count only.  Any out pointer may be NULL. */
int32_t ps_host_segment(ps_ctx* ctx, int64_t req, int32_t index, void** ptr, int64_t* bytes, int32_t* blk_lo,
                        int32_t* blk_hi, int32_t* n_segments);

/* ---- swap-in (Section 4.3 "Pipelined Reloading"; App. B: per-layer-chunk events) ---------- */

/* Queues a HOST request for reload: gives it fresh blocks for its whole table (all-or-nothing)
 * and appends it to the reload FIFO that ps_step consumes.  State becomes SWAPPING_IN.
 * Errors: PS_ERR_STATE, PS_ERR_NOMEM. */
int32_t ps_swap_in_begin(ps_ctx* ctx, int64_t req);

/* Withdraws a queued reload of which no block has been issued yet: blocks go back to the pool in
 * table order, state returns to HOST.  PS_ERR_BUSY once any block has been issued. */
int32_t ps_swap_in_cancel(ps_ctx* ctx, int64_t req);

/* Issues, on the copy streams, the reload of logical blocks [blk_lo, blk_hi) of one layer: one
 * contiguous host range -> device staging -> scattered into the request's fresh blocks, then
 * records that layer's completion event.  blk_lo must equal the number of blocks already issued
 * for this layer (a prefix that grows).  When every layer has reached the table's length the
 * request becomes RESIDENT; attention over it waits on the layers' events until the copies have
 * been seen complete.  ps_step calls this path for every layer itself; the entry point is for
 * callers that drive the layer loop on their own.
 * Errors: PS_ERR_STATE, PS_ERR_INVALID, PS_ERR_CUDA. */
int32_t ps_swap_in_layer(ps_ctx* ctx, int64_t req, int32_t layer, int32_t blk_lo, int32_t blk_hi);

/* Orders the compute stream after every reload issued so far into `layer` (layer = -1: into every layer):
 * work the caller enqueues on the compute stream afterwards finds those blocks of that layer complete
 * (Appendix B: the computation synchronises on a layer chunk's event before it executes that chunk).  For
 * callers that drive the layer loop themselves and write into reloaded blocks, e.g. a decode forward that
 * appends the new token's K and V to a request readmitted in this step before that layer's attention: without
 * the fence the scatter of the block's reloaded bytes could land after the caller's write.  ps_decode_attn
 * and ps_step order their own launches and need no fence.  A stream-side wait; the host does not block.
 * Errors: PS_ERR_INVALID (layer out of range), PS_ERR_CUDA. */
int32_t ps_reload_fence(ps_ctx* ctx, int32_t layer);

/* b_miss of Section 4.3 for one request: blocks on host not yet issued to the device. */
int32_t ps_missing_blocks(ps_ctx* ctx, int64_t req, int32_t* out);

/* ---- decode attention (the forward the reload hides under) -------------------------------- */

/* One layer of paged grouped-query decode attention on the compute stream:
 *   out[b][h][:] = softmax_t( q[b][h] . K[t][h/G] / sqrt(head_dim) ) . V[t][h/G],  t < n_tokens(reqs[b]),
 * K/V addressed through the request's block table; bf16 inputs, fp32 accumulation, bf16 output
 * (round to nearest even).  A request with 0 tokens gives zeros (lse = -inf).
 *   q, out : device pointers, bf16 [batch][num_q_heads][head_dim]
 *   lse    : device pointer, fp32 [batch][num_q_heads] (natural log of the softmax denominator
 *            including the max), or NULL
 *   reqs   : host array of `batch` request ids, all RESIDENT, batch <= max_batch
 * If a request's reload copies are not known to be complete the launch is ordered after this
 * layer's reload event.  Errors: PS_ERR_STATE, PS_ERR_INVALID, PS_ERR_CUDA. */
int32_t ps_decode_attn(ps_ctx* ctx, int32_t layer, const void* q, void* out, float* lse,
                       const int64_t* reqs, int32_t batch);

/* ---- decode attention without any allocation ---------------------------------------------- */

/* The paper has no counterpart to this call; it exists for hosts that may not allocate.
 *
 * Some users of this library cannot call cudaMalloc (or anything that does so for them) when they
 * need attention: an inference engine that gave all device memory to its own pool allocator at
 * start-up, code living inside another program's memory budget, a latency-critical loop in which
 * an allocation, which can synchronise the whole device, is not allowed.  ps_decode_attn above
 * needs a context, and ps_create allocates that context's split-KV scratch.  This entry point
 * computes the same attention with no context and no allocation: its scratch is a fixed array of
 * PS_STATIC_SCRATCH_BYTES that is part of the library image (every GPU that loads the library
 * holds it until the process exits), and everything else is the caller's memory.
 *
 *   kpool, vpool : device, bf16 [num_gpu_blocks][block_size][num_kv_heads][head_dim], one layer
 *   q, out       : device, bf16 [batch][num_q_heads][head_dim]
 *   lse          : device, fp32 [batch][num_q_heads], or NULL
 *   block_tables : device, int32 [batch][table_stride]; row b lists the blocks of request b
 *   ctx_lens     : HOST, int32 [batch]; tokens of request b (0 gives a zero row, lse = -inf)
 *   kv_split_tokens : tokens per split-KV work item, 0 = chosen from the batch
 *   status_word  : device int32 the kernels set to 2 when they meet a block id outside
 *                  [0, num_gpu_blocks) (the access is skipped), or NULL to ignore
 *   stream       : cudaStream_t on which everything is enqueued (asynchronous)
 *   err_buf      : host buffer of err_cap bytes that receives the error text, or NULL
 *
 * Limits (PS_ERR_INVALID with a message naming the limit when exceeded): batch <=
 * PS_STATIC_MAX_BATCH; at most 4096 work items (sum over requests of ceil(ctx / split)); their
 * partial results, num_q_heads * (head_dim + 4) floats per item, must fit in the scratch less
 * 192 KiB.  Shapes as for ps_decode_attn: head_dim 64 or 128, num_q_heads / num_kv_heads from
 * 1 to 8.  Results equal those of ps_decode_attn with the CUDA-core kernel.
 *
 * The first call on a device looks up the scratch's device address (cudaGetSymbolAddress, with that
 * device current) and caches it; make that first call before any stream capture begins.  All calls
 * on a device share the one array, which still holds the previous call's contents: every call
 * rewrites all metadata and the status word it owns before use, and partial results are written
 * before they are read, so back-to-back calls on one stream are independent.  Calls whose kernels
 * can overlap on the GPU (different streams with no ordering between them, or several host threads
 * doing so) race on the array and give wrong results: order them.
 * Errors: PS_ERR_INVALID, PS_ERR_CUDA.  Calls no cudaMalloc / cudaFree and no allocating routine. */
#define PS_STATIC_MAX_BATCH 256
#define PS_STATIC_SCRATCH_BYTES (16 * 1024 * 1024)
int32_t ps_decode_attn_static(const void* kpool, const void* vpool, const void* q, void* out, float* lse,
                              const int32_t* block_tables, int32_t table_stride, const int32_t* ctx_lens,
                              int32_t batch, int32_t num_kv_heads, int32_t num_q_heads, int32_t head_dim,
                              int32_t block_size, int32_t num_gpu_blocks, int32_t kv_split_tokens,
                              int32_t* status_word, void* stream, char* err_buf, int32_t err_cap);

/* ---- one engine step under the copy budget (Section 4.3 "Put it Together"; Alg. 1) -------- */

/* In order: reaps finished offloads; turns copy_budget_bytes into blocks (floor(bytes /
 * (num_layers * 2 * slab bytes)); negative = unlimited) and consumes the reload FIFO in order --
 * a request whose missing blocks fit is taken whole, the first that does not fit gets what is
 * left; then for each layer issues that layer's reload (as ps_swap_in_layer) and launches that
 * layer's attention for the requests of `reqs` that are RESIDENT once this step's reload is
 * issued.  Requests completed by this step have each layer's attention wait on that layer's
 * reload event (and on nothing later), so the reload of layer i+1 runs under the attention of
 * layer i; with the tensor-core kernel they run in a launch of their own on a side stream, so
 * that the other requests never wait, and the compute stream joins that stream at the end of the
 * step.  The queries of all layers are inputs, so consecutive layers are independent and their
 * launches may overlap head to tail.  Everything is enqueued asynchronously.
 *   q_all_layers, out_all_layers : device, bf16 [num_layers][batch][num_q_heads][head_dim]; rows of
 *                                  requests that do not decode are left untouched.  Both may be
 *                                  NULL with batch 0 for a copy-only step.
 *   decoded_mask                 : host int32[batch] (or NULL): 1 where the request decoded
 *   stats                        : host (or NULL)
 * Errors: PS_ERR_INVALID, PS_ERR_CUDA, PS_ERR_BOUNDS. */
int32_t ps_step(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs,
                int32_t batch, int64_t copy_budget_bytes, int32_t* decoded_mask, ps_step_stats* stats);

/* ps_step with the partial-copy admission test of Section 4.3 "Put it Together" (Alg. 1, SatisfyCopyCondition)
 * applied while the budget is consumed.  When the residual budget b_rem does not cover the b_miss missing blocks
 * of a queued request that `rule` lists, the request receives the residual only if ps_copy_condition(l_comp,
 * l_comp_max, b_miss, b_rem, block_size, beta) allows it; otherwise it is skipped in this step and the next
 * request of the reload queue is tried with the budget unchanged.  Requests that `rule` does not list, and every
 * request when rule == NULL, follow ps_step's reduced rule (the residual is always given).
 *   rule->reqs[i]       : request id
 *   rule->l_comp[i]     : tokens the scheduler could still compute for it in this round after a partial copy
 *                         (0 for a request that only decodes: it cannot run before its last block is back)
 *   rule->l_comp_max[i] : the round's computable-token limit for it
 * Errors: those of ps_step; PS_ERR_INVALID for beta <= 1, null arrays with n > 0, negative counts. */
typedef struct ps_copy_rule {
    double beta;
    int32_t n;
    int32_t reserved0;
    const int64_t* reqs;
    const int32_t* l_comp;
    const int32_t* l_comp_max;
} ps_copy_rule;
int32_t ps_step_ruled(ps_ctx* ctx, const void* q_all_layers, void* out_all_layers, const int64_t* reqs,
                      int32_t batch, int64_t copy_budget_bytes, const ps_copy_rule* rule, int32_t* decoded_mask,
                      ps_step_stats* stats);

/* Reload bytes that ps_step calls have issued and whose copies have not been seen complete yet (a non-blocking
 * look at the copy streams).  The budget rule of Section 4.3 assumes that a step's transfer ends within the step;
 * when the link runs below the profiled t_block the queue of copies grows from step to step and the step that
 * completes a request then waits for all of it.  A scheduler can subtract this figure from the budget it passes
 * to the next ps_step.  Timing-dependent by nature: 0 on a context without a device. */
int32_t ps_reload_backlog(ps_ctx* ctx, int64_t* bytes_in_flight);

/* ps_step for callers whose queries and outputs live in HOST memory: copies q_host to a device buffer of the
 * context on the compute stream, runs the step, and copies the outputs back, all asynchronously on the compute
 * stream (synchronise that stream, or call ps_sync, before reading out_host).
 *   q_host, out_host : host, bf16 [num_layers][batch][num_q_heads][head_dim]; pinned memory keeps the copies
 *                      asynchronous.  Rows of out_host whose request did not decode are zero.  Into pinned
 *                      memory the outputs are stored by a kernel, not by a copy engine, so that a step never
 *                      waits behind the device-to-host copies of an offload in flight.
 * The context's two device buffers ([num_layers][max_batch][num_q_heads][head_dim] each) are allocated by the
 * first call.  Errors: those of ps_step; PS_ERR_INVALID (batch 0, null buffers, bookkeeping-only context). */
int32_t ps_step_host(ps_ctx* ctx, const void* q_host, void* out_host, const int64_t* reqs, int32_t batch,
                     int64_t copy_budget_bytes, int32_t* decoded_mask, ps_step_stats* stats);

/* ---- adaptive copy budget (Section 4.3 "Adaptive Copy-Budget Control") -------------------- */

/* Latency model of one decode step and of the host link, in microseconds (Section 4.1: a decode request
 * costs a_d * l_kv + b_d, a batch the sum over its requests plus the constant t_c; Section 4.3: t_block
 * is the profiled copy time of one block, all layers). */
typedef struct ps_budget_model {
    double a_d_us_per_token;  /* a_d */
    double b_d_us;            /* b_d */
    double t_c_us;            /* t_c */
    double t_block_us;        /* t_block */
    double t_budget_us;       /* the scheduler's latency budget for this step */
} ps_budget_model;

/* Chooses B_copy, the number of blocks to reload in the coming step, by the paper's decision procedure:
 *   T_fwd_min   = estimated step time with every queued reload complete (all of `reqs` decode),
 *   T_trans_max = (missing blocks over the reload queue) * t_block;
 *   case 1  T_fwd_min > t_budget        : B_copy = floor(t_budget / t_block)
 *   case 2  T_fwd_min <= t_budget and
 *     2i    T_fwd_min > T_trans_max     : B_copy = all missing blocks
 *     2ii   otherwise                   : the largest B with
 *                                         B * t_block <= estimated step time after copying B blocks,
 * where "after copying B blocks" means: the requests of `reqs` that are resident now, plus those the
 * reload queue completes when it consumes B blocks in order.  (The paper finds that B by binary search over a
 * latency that falls as more is copied.  This library's path has no recomputation: the estimate is a step
 * function that rises whenever a queued request becomes complete, the test can fail and hold again, so the
 * intervals between those steps are scanned instead, one closed-form candidate each.)
 *   reqs          : host array, the decode batch of the coming step (as for ps_step)
 *   budget_blocks : B_copy;  budget_bytes : B_copy * bytes of a block over all layers, for ps_step
 *   which_case    : 1, 21 or 22 (may be NULL)
 * Decisions are taken in double precision.  Errors: PS_ERR_INVALID (non-positive t_block, negative terms). */
int32_t ps_copy_budget(ps_ctx* ctx, const int64_t* reqs, int32_t batch, const ps_budget_model* model,
                       int64_t* budget_blocks, int64_t* budget_bytes, int32_t* which_case);

/* ---- eviction policy and partial-copy admission (Section 4.3) ----------------------------- */

/* Victim choice under memory pressure (Section 4.3 "Eviction Policy").
 *   queue      : host array of n request ids in the scheduler's order, head (next to run) first
 *   waited_us  : host array of n waiting times
 *   tau_us     : the starvation threshold; near_frac in (0, 1]: "close to" means waited >= near_frac * tau
 *   blocks_needed : device blocks to free
 * Walks the queue from its tail and takes RESIDENT requests that hold blocks and are not close to
 * starvation until their blocks add up to blocks_needed; writes them to victims (capacity cap) in
 * eviction order.  *blocks_freed may end below blocks_needed when the queue does not hold enough.
 * Chooses only; the caller evicts with ps_swap_out.  Errors: PS_ERR_INVALID. */
int32_t ps_select_victims(ps_ctx* ctx, const int64_t* queue, int32_t n, const double* waited_us, double tau_us,
                          double near_frac, int32_t blocks_needed, int64_t* victims, int32_t cap, int32_t* n_victims,
                          int32_t* blocks_freed);

/* "Put it Together": whether request r may be copied in this round when the residual budget b_rem does
 * not cover its b_miss missing blocks.  A full copy (b_rem >= b_miss) is always allowed; a partial copy
 * only if the tokens still computable for r after it, l_comp, reach the round's limit l_comp_max, or if
 * l_comp / ((b_miss - b_rem) * s_blk) > beta (beta > 1).  *allowed = 1 or 0.  Pure arithmetic, for
 * schedulers built on this library: ps_step itself always allows partial copies (its decode-only batch
 * has no computable-token notion).  Errors: PS_ERR_INVALID (negative counts, s_blk <= 0, beta <= 1). */
int32_t ps_copy_condition(int32_t l_comp, int32_t l_comp_max, int32_t b_miss, int32_t b_rem, int32_t s_blk,
                          double beta, int32_t* allowed);

/* Queue ordering of the local scheduler (Section 4.2, SlideBatching, with the co-located load judgment of
 * Eq. "phi(Q)" and the starvation rule), as arithmetic for callers that want to drive the block management
 * in the paper's closed loop: the ordered queue feeds ps_select_victims (tail) and the reload order (head),
 * *t_budget_us feeds ps_copy_budget.
 *   exec_us[i]   : estimated execution time of request i in the coming batch (Section 4.1)
 *   remain_us[i] : time left to its deadline;  weight[i] : its token-level gain;  density = weight / exec
 *   waited_us    : waiting times, or NULL (no starvation rule)
 *   t_budget = max(min_i remain, eta);  phi = t_budget / (t_budget - t_c) * sum_i exec  (needs t_budget > t_c)
 *   request i is URGENT if remain[i] < gamma * phi, else NORMAL
 *   order: starving requests (waited > tau) first, in input order; then URGENT by density, largest first;
 *          then NORMAL by remaining time, smallest first; ties keep the input order.
 *   order   : out, n indices into the input arrays, head of the queue first
 *   urgent  : out, n flags per input index (1 urgent, 0 normal, 2 starving), or NULL
 * Errors: PS_ERR_INVALID (n < 0, null arrays, non-positive exec, t_budget <= t_c). */
typedef struct ps_sched_params {
    double eta_us;    /* lower bound of the latency budget */
    double gamma;     /* aggressiveness coefficient */
    double t_c_us;    /* constant per-batch overhead */
    double tau_us;    /* starvation threshold (used only with waited_us) */
} ps_sched_params;
int32_t ps_order_queue(int32_t n, const double* exec_us, const double* remain_us, const double* weight,
                       const double* waited_us, const ps_sched_params* params, int32_t* order, int32_t* urgent,
                       double* t_budget_us);

/* ---- batch latency estimator and the cost of resuming an evicted request ------------------- */

/* Coefficients of the batch latency estimator (Section 4.1, "Batch Latency Estimator"), microseconds:
 *   prefill request  T~_p = a_p * l_q^2 + b_p * l_q * l_kv + c_p * l_q
 *   decode request   T~_d = a_d * l_kv + b_d
 *   batch            T(B) = sum of T~ over its requests + t_c
 * l_q = tokens processed in this forward pass, l_kv = KV-cache length before it. */
typedef struct ps_latency_model {
    double a_p_us, b_p_us, c_p_us;
    double a_d_us, b_d_us;
    double t_c_us;
} ps_latency_model;

/* Estimated execution time of one batch (the batch equation of Section 4.1).
 *   l_q, l_kv_prefill : host int32[n_prefill];  l_kv_decode : host int32[n_decode]
 * An empty batch costs t_c.  Errors: PS_ERR_INVALID (null arrays with a positive count, negative lengths
 * or coefficients). */
int32_t ps_estimate_batch(const ps_latency_model* model, int32_t n_prefill, const int32_t* l_q,
                          const int32_t* l_kv_prefill, int32_t n_decode, const int32_t* l_kv_decode,
                          double* batch_us);

/* The two ways of bringing an evicted request of n_tokens back, compared by the estimator: the paper spills
 * evicted blocks to host memory and reloads them (Section 4.3, "Eviction Policy"); its ablation arm
 * "Recompute" discards them instead, so the context is prefilled again.  The paper prints no cost formula
 * for that arm; here it is the estimator's own prefill time of the whole context, run in chunks of
 * chunk_tokens (chunk k processes l_q = min(chunk, n - k*chunk) tokens on l_kv = k*chunk cached ones; every
 * chunk is a batch of its own and pays t_c; chunk_tokens = 0 means one pass):
 *   recompute_us = sum over chunks of (T~_p(l_q, l_kv) + t_c)
 *   reload_us    = ceil(n_tokens / s_blk) * t_block_us        (Section 4.3: T_trans = b_miss * t_block)
 * The reload figure is the full transfer time; how much of it hides under decode steps is what ps_step's
 * statistics measure.  Pure arithmetic.  Errors: PS_ERR_INVALID (negative n_tokens or chunk, s_blk <= 0,
 * negative coefficients or t_block). */
int32_t ps_resume_cost(const ps_latency_model* model, int32_t n_tokens, int32_t chunk_tokens, int32_t s_blk,
                       double t_block_us, double* reload_us, double* recompute_us);

/* ---- completion ------------------------------------------------------------------------- */

/* Non-blocking: reaps finished offloads (in issue order), releases host images of finished
 * reloads.  *n_reaped (may be NULL) = offloads reaped by this call. */
int32_t ps_poll(ps_ctx* ctx, int32_t* n_reaped);

/* Waits until every transfer and kernel this context has enqueued (copy streams and the compute
 * stream) is complete, then reaps as ps_poll.  timeout_ms < 0 waits without limit.
 * PS_ERR_TIMEOUT leaves everything in flight. */
int32_t ps_sync(ps_ctx* ctx, int32_t timeout_ms);

/* ---- measurement ------------------------------------------------------------------------ */

/* Kernels launched by this context since creation. */
int32_t ps_launch_count(ps_ctx* ctx, int64_t* out);

/* Accumulated device times per kind since the last reset (needs PS_FLAG_PROFILE; call after
 * ps_sync).  reset != 0 clears the accumulators afterwards. */
int32_t ps_get_profile(ps_ctx* ctx, ps_profile* out, int32_t reset);

/* Timeline of the copy streams against the compute stream (the per-layer-chunk overlap of
 * Appendix B made visible).  ps_trace(ctx, 1) starts recording every kernel and transfer span of a
 * PS_FLAG_PROFILE context relative to "now" on the compute stream; ps_trace(ctx, 0) stops.
 * ps_trace_read copies up to cap spans (call after ps_sync) and reports how many exist. */
int32_t ps_trace(ps_ctx* ctx, int32_t enable);
int32_t ps_trace_read(ps_ctx* ctx, ps_trace_span* out, int32_t cap, int32_t* n);

/* Pinned-memory host link probe: best-of-`iters` cudaMemcpyAsync of `bytes` between a pinned host
 * buffer and a device buffer, timed with CUDA events.  direction 0 = host-to-device, 1 = device-
 * to-host, 2 = both at once on two streams (reports the sum).  *gb_per_s in 1e9 bytes/s.
 * Allocates and frees its own buffers; needs no context. */
int32_t ps_link_probe(int64_t bytes, int32_t direction, int32_t iters, double* gb_per_s);

/* Device-memory bandwidth probe with a plain streaming kernel of this library: best of `iters` passes over
 * `bytes` (a multiple of 16, at least 1 MiB; use more than the L2 holds), timed with CUDA events on the default
 * stream.  mode 0 = read only (the traffic pattern of decode attention: KV is read, almost nothing written),
 * mode 1 = copy (bytes read + bytes written are counted, the accounting of a gather or scatter).  *gb_per_s in
 * 1e9 bytes/s.  Allocates and frees its own buffers; needs no context. */
int32_t ps_hbm_probe(int64_t bytes, int32_t mode, int32_t iters, double* gb_per_s);

/* The gather kernel of ps_swap_out (direction 0: pools -> staging) or the scatter kernel of ps_swap_in_layer /
 * ps_step (direction 1: staging -> pools) alone, without any host transfer, on the compute stream: the same
 * kernels in the launch shape the swap path gives them, for measuring them against HBM bandwidth.  One launch
 * moves `n_blocks` blocks of the layers [layer, layer + n_layers); `staging` is a device pointer with room for
 * n_layers * n_blocks * 2 slabs, laid out [n_layers][n_blocks][K,V][slab]; ids is a host array of n_blocks
 * block ids.  n_layers > 1 is the shape of a reload's layer chunk under a small copy budget. */
int32_t ps_copy_blocks(ps_ctx* ctx, int32_t layer, int32_t n_layers, const int32_t* ids, int32_t n_blocks,
                       void* staging, int32_t direction);

/* Test hook: writes `value` into the context's kernel status word as a kernel would (1 = a copy kernel met a
 * bad block id, 2 = an attention kernel did, 3 = a bounded wait inside the attention kernel ran out; on a device
 * context 3 also leaves the kernel's chunk and arrival counters dirty, as CTAs that gave up would).  The next
 * ps_poll / ps_step / ps_sync then reports it.  Lets the error path be exercised without making a kernel fail. */
int32_t ps_inject_status(ps_ctx* ctx, int32_t value);

#ifdef __cplusplus
}
#endif
#endif /* PS_KVSWAP_H */
