// Paged grouped-query decode attention: the per-layer computation that the pipelined reload
// hides under (Section 4.3, "Pipelined Reloading": layer i computes while layer i+1 loads).
//
//   out[b][h] = softmax_t( q[b][h] . K[t][h/G] / sqrt(D) ) . V[t][h/G],   t < ctx_len[b]
//
// bf16 inputs, fp32 accumulation, softmax in base 2 with log2(e)/sqrt(D) folded into q.  The
// work is split over the KV axis into items of a bounded token count; an item that is the only
// one of its row writes the final output, otherwise it writes an unnormalised partial (running
// max, running sum, D accumulators per head); partials are combined by the merge kernel (CUDA-core
// path) or inside the tensor-core kernel.
//
// The kernel is HBM-bound (G flop per KV byte), so the SIMT kernel below spends its effort on
// 16-byte coalesced loads with many of them in flight; softmax statistics are reduced with warp
// shuffles inside the group of lanes that shares a token.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cstring>
#include <math_constants.h>

#include "ps_internal.h"

namespace ps {
namespace {

constexpr float kNegBig = -1.0e30f;  // "no token seen yet": finite, so that differences stay finite
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ uint4 ld_nc16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ void bf16x8_to_f32(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x << 16);
    f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16);
    f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16);
    f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16);
    f[7] = __uint_as_float(v.w & 0xffff0000u);
}

// ------------------------------------------------------------------------------------------------
// SIMT kernel.  grid = (items, Hkv); 128 threads.  D/8 lanes share one token (each lane owns 8
// head dims); the 128/(D/8) lane groups of the CTA walk the item's tokens with stride, kUnroll
// tokens per trip, and are combined through shared memory at the end.
// ------------------------------------------------------------------------------------------------
constexpr int kSimtThreads = 128;
constexpr int kUnroll = 4;

template <int D, int G>
__global__ void __launch_bounds__(kSimtThreads)
decode_attn_simt_kernel(const __nv_bfloat16* __restrict__ kpool, const __nv_bfloat16* __restrict__ vpool,
                        const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out,
                        float* __restrict__ lse, AttnBatch batch, int32_t item_begin, int32_t num_kv_heads,
                        int32_t block_size, int32_t block_shift, int32_t num_blocks, float* __restrict__ partials,
                        float scale_log2e, int32_t* status) {
    constexpr int LPT = D / 8;                  // lanes per token
    constexpr int NG = kSimtThreads / LPT;      // lane groups per CTA
    __shared__ float sm_m[NG][G];
    __shared__ float sm_l[NG][G];
    __shared__ float sm_acc[NG][G][D];

    const AttnItem item = batch.items[item_begin + blockIdx.x];
    const int kvh = blockIdx.y;
    const int Hq = num_kv_heads * G;
    const int lig = threadIdx.x % LPT;          // lane in group: owns dims [8 lig, 8 lig + 8)
    const int group = threadIdx.x / LPT;
    const int32_t* table = batch.block_tables + (int64_t)item.b * batch.table_stride;
    const int64_t tok_stride = (int64_t)num_kv_heads * D;   // elements between consecutive tokens of a block
    const int64_t head_off = (int64_t)kvh * D + 8 * lig;

    float qf[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint4 raw = *reinterpret_cast<const uint4*>(q + ((int64_t)item.b * Hq + kvh * G + g) * D + 8 * lig);
        bf16x8_to_f32(raw, qf[g]);
#pragma unroll
        for (int i = 0; i < 8; ++i) qf[g][i] *= scale_log2e;
    }

    float m[G], l[G], acc[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = kNegBig;
        l[g] = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[g][i] = 0.f;
    }

    // the trip count is uniform over the CTA (full-mask shuffles below); lanes past the end are masked
    for (int tb = item.t_begin; tb < item.t_end; tb += NG * kUnroll) {
        const int t0 = tb + group;
        uint4 kraw[kUnroll], vraw[kUnroll];
        bool valid[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int t = t0 + u * NG;
            valid[u] = t < item.t_end;
            kraw[u] = make_uint4(0, 0, 0, 0);
            vraw[u] = make_uint4(0, 0, 0, 0);
            if (valid[u]) {
                const int blk = block_shift >= 0 ? (t >> block_shift) : (t / block_size);
                const int slot = t - blk * block_size;
                const int id = __ldg(table + blk);
                if ((unsigned)id >= (unsigned)num_blocks) {
                    *(volatile int32_t*)status = 2;
                    valid[u] = false;
                } else {
                    const int64_t off = ((int64_t)id * block_size + slot) * tok_stride + head_off;
                    kraw[u] = ld_nc16(kpool + off);
                    vraw[u] = ld_nc16(vpool + off);
                }
            }
        }
        float s[kUnroll][G];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float kf[8];
            bf16x8_to_f32(kraw[u], kf);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float d = 0.f;
#pragma unroll
                for (int i = 0; i < 8; ++i) d = fmaf(qf[g][i], kf[i], d);
                s[u][g] = d;
            }
        }
#pragma unroll
        for (int off = LPT / 2; off > 0; off >>= 1)
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int g = 0; g < G; ++g) s[u][g] += __shfl_xor_sync(0xffffffffu, s[u][g], off);

        float p[kUnroll][G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float mx = m[g];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (valid[u]) mx = fmaxf(mx, s[u][g]);
            const float alpha = exp2f(m[g] - mx);
            m[g] = mx;
            float ps = 0.f;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                p[u][g] = valid[u] ? exp2f(s[u][g] - mx) : 0.f;
                ps += p[u][g];
            }
            l[g] = l[g] * alpha + ps;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[g][i] *= alpha;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float vf[8];
            bf16x8_to_f32(vraw[u], vf);
#pragma unroll
            for (int g = 0; g < G; ++g)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[g][i] = fmaf(p[u][g], vf[i], acc[g][i]);
        }
    }

    // combine the lane groups
#pragma unroll
    for (int g = 0; g < G; ++g) {
        if (lig == 0) {
            sm_m[group][g] = m[g];
            sm_l[group][g] = l[g];
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) sm_acc[group][g][8 * lig + i] = acc[g][i];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < G * D; e += kSimtThreads) {
        const int g = e / D;
        const int d = e - g * D;
        float M = kNegBig;
#pragma unroll
        for (int i = 0; i < NG; ++i) M = fmaxf(M, sm_m[i][g]);
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int i = 0; i < NG; ++i) {
            const float w = exp2f(sm_m[i][g] - M);
            L = fmaf(sm_l[i][g], w, L);
            O = fmaf(sm_acc[i][g][d], w, O);
        }
        const int h = kvh * G + g;
        if (item.n_parts == 1) {
            const float o = L > 0.f ? O / L : 0.f;
            out[((int64_t)item.b * Hq + h) * D + d] = __float2bfloat16_rn(o);
            if (lse != nullptr && d == 0)
                lse[(int64_t)item.b * Hq + h] = L > 0.f ? (M + log2f(L)) * kLn2 : -CUDART_INF_F;
        } else {
            float* pr = partials + ((int64_t)item.part * Hq + h) * (D + 2);
            pr[d] = O;
            if (d == 0) {
                pr[D] = M;
                pr[D + 1] = L;
            }
        }
    }
}

// Merge: grid = (B, Hq), D threads.  Rows with a single part were finished by the attention kernel.
template <int D>
__global__ void __launch_bounds__(D)
attn_merge_kernel(__nv_bfloat16* __restrict__ out, float* __restrict__ lse, AttnBatch batch, int32_t Hq,
                  const float* __restrict__ partials, int32_t lane) {
    const int b = blockIdx.x;
    const int n = batch.row_parts[b];
    if (n <= 1) return;
    if (lane >= 0 && batch.row_lane[b] != lane) return;
    const int h = blockIdx.y;
    const int d = threadIdx.x;
    const float* base = partials + ((int64_t)batch.row_first_part[b] * Hq + h) * (D + 2);
    const int64_t stride = (int64_t)Hq * (D + 2);
    float M = kNegBig;
    for (int i = 0; i < n; ++i) M = fmaxf(M, base[i * stride + D]);
    float L = 0.f, O = 0.f;
    for (int i = 0; i < n; ++i) {
        const float w = exp2f(base[i * stride + D] - M);
        L = fmaf(base[i * stride + D + 1], w, L);
        O = fmaf(base[i * stride + d], w, O);
    }
    out[((int64_t)b * Hq + h) * D + d] = __float2bfloat16_rn(L > 0.f ? O / L : 0.f);
    if (lse != nullptr && d == 0) lse[(int64_t)b * Hq + h] = L > 0.f ? (M + log2f(L)) * kLn2 : -CUDART_INF_F;
}

int shift_of(int32_t v) {
    if (v <= 0 || (v & (v - 1))) return -1;
    int s = 0;
    while ((1 << s) < v) ++s;
    return s;
}

template <int D, int G>
cudaError_t launch_simt(const AttnShape& sh, const void* kpool, const void* vpool, const void* q, void* out, float* lse,
                        const AttnBatch& batch, int32_t item_begin, int32_t n_items, float* partials,
                        int32_t* d_status, cudaStream_t stream) {
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)D);
    dim3 grid((unsigned)n_items, (unsigned)sh.num_kv_heads);
    decode_attn_simt_kernel<D, G><<<grid, kSimtThreads, 0, stream>>>(
        (const __nv_bfloat16*)kpool, (const __nv_bfloat16*)vpool, (const __nv_bfloat16*)q, (__nv_bfloat16*)out, lse,
        batch, item_begin, sh.num_kv_heads, sh.block_size, shift_of(sh.block_size), sh.num_blocks, partials,
        scale_log2e, d_status);
    return cudaGetLastError();
}


// ------------------------------------------------------------------------------------------------
// Tensor-core kernel (head_dim 128, 8 KV heads, block size a multiple of 16).
//
// Work: the batch's contexts are cut into 16-token tiles forming one sequence, which the host divides
// into equal static shares, one per CTA (one CTA per SM): every CTA streams the same number of bytes
// whatever the context-length mix.  Optionally the sequence's tail is cut into chunks handed out through
// an atomic counter to whichever CTA finishes first (the host asks for that when reload traffic makes
// SMs unevenly fast).  An item is a (row, token range); each item produces one result: final if it
// covers the whole row, else a partial.  The warp that delivers the last partial of a (row, KV head),
// found through an arrival counter, combines the row's partials after its CTA's last tile.
//
// Data path: a tile is 16 token rows of K and 16 of V; a token row holds all 8 KV heads (2 KiB,
// contiguous in the pool).  Stages of a 3-deep shared-memory ring are signalled through mbarriers; next to
// each stage the producer warp publishes which item and tile it holds, and the consumers follow that
// stream.  Tensor-map mode: per stage two box copies (cp.async.bulk.tensor) of 32 KiB through maps that
// view a pool as (64 elements, token row, 128-byte chunk of the row) with the 128-byte swizzle, so a tile
// lands as [chunk][token][128 B] with 16-byte units XORed by the token index and ldmatrix over 8 tokens
// of one head touches 8 different bank groups; token rows past a context's end arrive too and are
// cleared (V) or masked (scores) by the consumers.  Row mode: one 2 KiB bulk copy per token row at a
// 2064-byte pitch (same bank property by padding); rows past the end are never copied, and the ring is
// zeroed once so that a stale row is always finite.  Row mode is limited by the rate at which the copy
// unit retires 2 KiB copies (about 6.5 TB/s over the chip), box copies by HBM.
//
// Math: warp w owns KV head w.  Scores: mma.m16n8k16 with the G query heads of the group as the M
// rows (padded to 16; the padding rows of every product are dropped) and 8 tokens as N; softmax
// statistics per query head are reduced over the 4 lanes of a quad with shuffles; P is re-packed in
// registers as the A operand of P.V with V read through ldmatrix.trans.  (Two warps per head were
// tried: at 17 warps the register budget drops to 96 per thread and the inner loop spills.)
// Tensor cores keep the FMA work off the ALUs: the kernel is bound by HBM (G flop per KV byte).
//
// Every wait is bounded: after kSpinLimit polls a thread raises the CTA's abort word, reports
// through the status word and everybody leaves.
// ------------------------------------------------------------------------------------------------
constexpr int kMmaD = 128;
constexpr int kMmaHkv = 8;
constexpr int kMmaStages = 3;
constexpr int kMmaRowBytes = kMmaHkv * kMmaD * 2;         // 2048: one token, all KV heads
constexpr int kMmaPitch = kMmaRowBytes + 16;              // 2064: breaks the 2 KiB bank alignment
constexpr int kMmaSlabBytes = kMmaTileTokens * kMmaPitch; // one K (or V) tile in shared memory
constexpr int kMmaStageBytes = 2 * kMmaSlabBytes;
constexpr int kMmaRingBytes = kMmaStages * kMmaStageBytes;
constexpr int kMmaMaxPending = 14;                        // rows a warp may note for combining after its last tile
constexpr int kMmaCtrlBytes = 128 + 8 * 16 * 4 + 128;     // barriers, stage descriptors, abort word; pending-row lists;
                                                          // exchange barriers
constexpr int kMmaConsumerWarps = kMmaHkv;
constexpr int kMmaThreads = (kMmaConsumerWarps + 1) * 32;
constexpr int kMmaPartStride = kMmaD + 4;                 // floats per (part, query head): 16-byte aligned rows
constexpr int kSpinLimit = 1 << 22;
constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagEnd = 4;

// Tensor-map mode: a K (or V) tile is one 32 KiB box copy, laid out [16 chunks of 128 B][16 tokens][128 B] with
// the 128-byte swizzle (16-byte units XORed with the token index mod 8), so no row padding is needed.
constexpr int kTmaTileBytes = kMmaTileTokens * kMmaRowBytes;   // 32768
constexpr int kTmaStageBytes = 2 * kTmaTileBytes;              // 65536
constexpr int kTmaRingBytes = kMmaStages * kTmaStageBytes;
constexpr int kTmaAlign = 1024;                                // the swizzle pattern repeats every 1 KiB

// Fewer than 8 KV heads (tensor-map mode only): a stage still holds 64 KiB, now 8 / HKV sub-tiles of 16 tokens
// each (one K and one V box per sub-tile, possibly from different blocks), and the 8 consumer warps are
// (head, sub-tile) pairs: warp w works on head w % HKV, sub-tile w / HKV.  The warps of one head each keep their
// own softmax state over every (8 / HKV)-th 16-token slice of the row and combine the states at the end of an
// item through a small exchange area (34 floats per lane of every warp with a sub-tile index above 0).
constexpr int mma_subs(int hkv) { return kMmaHkv / hkv; }
constexpr int mma_xchg_bytes(int hkv) { return (kMmaHkv - hkv) * 32 * 34 * 4; }
constexpr int mma_smem_bytes(bool tma, int hkv) {
    return tma ? kTmaRingBytes + kTmaAlign + kMmaCtrlBytes + mma_xchg_bytes(hkv) : kMmaRingBytes + kMmaCtrlBytes;
}

struct StageDesc {  // published by the producer next to every ring stage
    int32_t item;   // index into batch.items
    int32_t t0;     // first token of the tile
    int32_t rows;   // valid token rows (0 for the pseudo-tile of an empty context)
    int32_t flags;  // kFlagFirst | kFlagLast | kFlagEnd
};

// Release / acquire fence at device scope: what publishing a partial result before announcing it, and reading
// the other parts after finding them all announced, need.  (__threadfence() is the sequentially consistent
// fence, which costs more and orders nothing more that this kernel relies on.)
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded, warp-uniform wait.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int32_t* abort_word,
                                          int32_t* status) {
    bool ok = false;
    for (int i = 0; i < kSpinLimit; ++i) {
        if (mbar_test(bar, parity)) {
            ok = true;
            break;
        }
        if (*abort_word) break;
        if (i > 32) __nanosleep(40);
    }
    if (!ok && !*abort_word) {
        *abort_word = 1;
        *(volatile int32_t*)status = 3;
    }
    return __all_sync(0xffffffffu, ok);
}
// KV rows are read once per launch: they are marked evict-first in L2 so that the split-KV partials (written and
// re-read within the launch) and the batch metadata stay resident under the stream.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
// One box of a rank-3 tensor map (element, token row, 128-byte chunk) into shared memory.
__device__ __forceinline__ void tensor_g2s(uint32_t dst, const void* map, int32_t token_row, uint32_t bar,
                                           uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;" ::"r"(dst),
        "l"(map), "r"(0), "r"(token_row), "r"(0), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
// D = A(16x16) B(16x8) + C; only rows 0-7 of A are populated (a1 = a3 = 0), rows 8-15 of D are dropped.
__device__ __forceinline__ void mma_k16(float& d0, float& d1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1,
                                        float c0, float c1) {
    float x2, x3;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d0), "=f"(d1), "=f"(x2), "=f"(x3)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(c0), "f"(c1), "f"(0.f), "f"(0.f));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// Combines the parts of batch row b for the G query heads of KV head h (one warp; every part has been
// delivered and fenced).  Parts are combined in part order, whoever calls.  The loads of all G heads
// are issued together, two parts at a time.  Re-arms the row's arrival counter.
template <int G, int HKV>
__device__ __forceinline__ void merge_row(int b, int h, int lane, const AttnBatch& batch,
                                          const float* __restrict__ partials, __nv_bfloat16* __restrict__ out,
                                          float* __restrict__ lse, int32_t* __restrict__ row_done) {
    constexpr int Hq = HKV * G;
    fence_acq_rel_gpu();
    const int n = batch.row_parts[b];
    const float* base = partials + ((int64_t)batch.row_first_part[b] * Hq + h * G) * kMmaPartStride;
    const int64_t stride = (int64_t)Hq * kMmaPartStride;   // floats between parts
    // One pass over the parts, two at a time, with a running maximum per head (sums and accumulators are
    // rescaled when it grows): every part is loaded once, the loads of a pair are issued together, and the
    // chain of dependent round trips to L2 is half as long as with a separate pass for the maximum.  Lane owns
    // dims [4 lane, 4 lane + 4) of every head.
    float M[G];
    float4 acc[G];
    float Ls[G];
#pragma unroll
    for (int gg = 0; gg < G; ++gg) {
        M[gg] = kNegBig;
        acc[gg] = make_float4(0.f, 0.f, 0.f, 0.f);
        Ls[gg] = 0.f;
    }
    for (int i0 = 0; i0 < n; i0 += 2) {
        const bool two = i0 + 1 < n;
        float4 va[G], vb[G];
        float ma[G], la[G], mb[G], lb[G];
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            const float* pa = base + i0 * stride + gg * kMmaPartStride;
            va[gg] = __ldcg(reinterpret_cast<const float4*>(pa) + lane);
            ma[gg] = __ldcg(pa + kMmaD);
            la[gg] = __ldcg(pa + kMmaD + 1);
            vb[gg] = make_float4(0.f, 0.f, 0.f, 0.f);
            mb[gg] = kNegBig;
            lb[gg] = 0.f;
            if (two) {
                vb[gg] = __ldcg(reinterpret_cast<const float4*>(pa + stride) + lane);
                mb[gg] = __ldcg(pa + stride + kMmaD);
                lb[gg] = __ldcg(pa + stride + kMmaD + 1);
            }
        }
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            const float m_new = fmaxf(M[gg], fmaxf(ma[gg], mb[gg]));
            const float sc = exp2f(M[gg] - m_new);
            const float wa = exp2f(ma[gg] - m_new);
            const float wb = two ? exp2f(mb[gg] - m_new) : 0.f;
            M[gg] = m_new;
            Ls[gg] = fmaf(lb[gg], wb, fmaf(la[gg], wa, Ls[gg] * sc));
            acc[gg].x = fmaf(vb[gg].x, wb, fmaf(va[gg].x, wa, acc[gg].x * sc));
            acc[gg].y = fmaf(vb[gg].y, wb, fmaf(va[gg].y, wa, acc[gg].y * sc));
            acc[gg].z = fmaf(vb[gg].z, wb, fmaf(va[gg].z, wa, acc[gg].z * sc));
            acc[gg].w = fmaf(vb[gg].w, wb, fmaf(va[gg].w, wa, acc[gg].w * sc));
        }
    }
#pragma unroll
    for (int gg = 0; gg < G; ++gg) {
        const int hq = h * G + gg;
        const float inv = Ls[gg] > 0.f ? 1.f / Ls[gg] : 0.f;
        __nv_bfloat16* orow = out + ((int64_t)b * Hq + hq) * kMmaD;
        uint2 packed;
        packed.x = pack_bf16(acc[gg].x * inv, acc[gg].y * inv);
        packed.y = pack_bf16(acc[gg].z * inv, acc[gg].w * inv);
        *reinterpret_cast<uint2*>(orow + 4 * lane) = packed;
        if (lse != nullptr && lane == 0)
            lse[(int64_t)b * Hq + hq] = Ls[gg] > 0.f ? (M[gg] + log2f(Ls[gg])) * kLn2 : -CUDART_INF_F;
    }
    if (lane == 0) row_done[b * HKV + h] = 0;  // every part has arrived: re-arm for the next launch
}

template <int G, int HKV, bool kTma>
__global__ void __launch_bounds__(kMmaThreads, 1)
decode_attn_mma_kernel(const __nv_bfloat16* __restrict__ kpool, const __nv_bfloat16* __restrict__ vpool,
                       const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap,
                       const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out, float* __restrict__ lse,
                       AttnBatch batch, int32_t sched_lane, int32_t block_size, int32_t block_shift,
                       int32_t num_blocks, float* __restrict__ partials, int32_t* __restrict__ sched,
                       int32_t* __restrict__ row_done, float scale_log2e, int32_t* status, int32_t wait_first) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    static_assert(HKV == kMmaHkv || kTma, "fewer than 8 KV heads need the tensor-map mode");
    constexpr int Hq = HKV * G;
    constexpr int kSubs = kMmaHkv / HKV;                         // 16-token sub-tiles per stage
    constexpr int kSubBytes = kMmaTileTokens * HKV * kMmaD * 2;   // one K (or V) sub-tile in tensor-map mode
    constexpr int kStageTokens = kMmaTileTokens * kSubs;
    constexpr int kStageBytes = kTma ? kTmaStageBytes : kMmaStageBytes;
    constexpr int kRingBytes = kTma ? kTmaRingBytes : kMmaRingBytes;
    constexpr int kVOff = kTma ? kTmaTileBytes : kMmaSlabBytes;   // V tiles inside a stage
    // the swizzled layout needs the ring on a 1 KiB boundary of the shared address space
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = kTma ? (raw + kTmaAlign - 1) & ~(uint32_t)(kTmaAlign - 1) : raw;
    unsigned char* smem = smem_raw + (ring - raw);
    unsigned char* ctrl = smem + kRingBytes;
    const uint32_t bar_full = ring + kRingBytes;            // [kMmaStages]
    const uint32_t bar_empty = bar_full + 8 * kMmaStages;   // [kMmaStages]
    // 48 bytes of barriers, then the stage descriptors and the abort word
    volatile StageDesc* sdesc = reinterpret_cast<volatile StageDesc*>(ctrl + 64);
    volatile int32_t* abort_word = reinterpret_cast<volatile int32_t*>(ctrl + 64 + 16 * kMmaStages);
    const uint32_t bar_xfull = bar_full + 640;              // [HKV] exchange: states of a head's other warps are in
    const uint32_t bar_xempty = bar_xfull + 8 * kMmaHkv;    // [HKV] exchange: the combining warp has read them
    float* xchg = reinterpret_cast<float*>(ctrl + kMmaCtrlBytes);
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // Programmatic dependent launch: the next layer's launch (same kernel, independent inputs) may start filling
    // SMs as the CTAs of this one retire, which hides its launch latency and prologue under this launch's tail.
    // What consecutive launches do share is the split-KV scratch (partials, arrival counters, chunk counters):
    // a thread executes griddepcontrol.wait (dep_wait below) before it first touches any of it, i.e. it waits
    // until the launch this one depends on has completed and its memory operations are visible; as every
    // launch also executes it before it ends, launches complete in order, so no earlier launch is still
    // running either.  The first such access comes at the end of a CTA's first row part, long after the
    // predecessor's tail.  All of it is a no-op for ordinary launches.
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    auto dep_wait = []() { asm volatile("griddepcontrol.wait;" ::: "memory"); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < kMmaStages; ++s) {
            mbar_init(bar_full + 8 * s, 1);
            mbar_init(bar_empty + 8 * s, kMmaConsumerWarps);
        }
        if (kSubs > 1)
            for (int hh = 0; hh < HKV; ++hh) {
                mbar_init(bar_xfull + 8 * hh, kSubs - 1);
                mbar_init(bar_xempty + 8 * hh, 1);
            }
        *abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (!kTma) {  // row copies skip the rows past a context's end: a stale row must at least be finite
        for (int i = threadIdx.x; i < kRingBytes / 16; i += kMmaThreads)
            reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy zeroes before async-proxy writes
    }
    __syncthreads();
    // A launch whose inputs (queries, KV, batch metadata) may come from the kernel before it on the stream is
    // still made programmatically dependent on that kernel: block scheduling, the shared-memory set-up and the
    // barrier initialisation above then run under the predecessor's tail, and every thread waits here, before
    // the first read of anything the predecessor may have written.
    if (wait_first) dep_wait();

    const int32_t* cta_begin = batch.cta_begin[sched_lane];
    const int item0 = cta_begin[blockIdx.x];
    const int item1 = cta_begin[blockIdx.x + 1];
    const int dyn_begin = cta_begin[gridDim.x];         // the lane's dynamic chunks follow the static shares
    const int dyn_end = batch.lane_items[sched_lane + 1];

    if (warp == kMmaConsumerWarps) {
        // ------------------------------------------------ producer warp
        const uint64_t kv_policy = l2_evict_first_policy();
        int n = 0;
        bool ok = true;
        int32_t* counter = sched + 2 * sched_lane;
        int it = item0;
        bool dynamic = false;
        AttnItem pre_item{};   // descriptor and id windows of the CTA's next static item, fetched ahead
        int pre_it = -1, pre_ids = 0, pre_ids_next = 0;
        while (ok) {
            if (!dynamic && it >= item1) dynamic = true;
            if (dynamic) {
                int c = 0;
                dep_wait();
                if (lane == 0) c = atomicAdd(counter, 1);
                c = __shfl_sync(0xffffffffu, c, 0);
                it = dyn_begin + c;
                if (it >= dyn_end) break;
            }
            // A static item's descriptor and first block-id windows were fetched while the item before it was
            // being streamed (below); otherwise they are fetched now, three dependent loads during which no
            // copy is issued.
            const bool primed = pre_it == it;
            const AttnItem item = primed ? pre_item : batch.items[it];
            const int32_t* table = batch.block_tables + (int64_t)item.b * batch.table_stride;
            const int ntiles = max(1, (item.t_end - item.t_begin + kStageTokens - 1) / kStageTokens);
            // Block ids are read 32 at a time, one per lane, a window ahead of their use: the table read
            // never sits between a freed stage and the copies that refill it.
            const int last_blk = (max(item.t_end, 1) - 1) / block_size;
            int win = block_shift >= 0 ? (item.t_begin >> block_shift) : (item.t_begin / block_size);
            int ids = primed ? pre_ids : (win + lane <= last_blk ? __ldg(table + win + lane) : 0);
            int ids_next = primed ? pre_ids_next : (win + 32 + lane <= last_blk ? __ldg(table + win + 32 + lane) : 0);
            pre_it = -1;
            const bool prime_next = !dynamic && it + 1 < item1;
            if (prime_next) pre_item = batch.items[it + 1];  // issued now, needed after this item's first copies
            for (int ti = 0; ti < ntiles; ++ti, ++n) {
                const int s = n % kMmaStages;
                const int t0 = item.t_begin + ti * kStageTokens;
                const int rows = max(0, min(kStageTokens, item.t_end - t0));
                const int blk = block_shift >= 0 ? (t0 >> block_shift) : (t0 / block_size);
                if (blk >= win + 32) {  // a stage starts at most 8 blocks after the last: the next window is the one ahead
                    win += 32;
                    ids = ids_next;
                    ids_next = win + 32 + lane <= last_blk ? __ldg(table + win + 32 + lane) : 0;
                }
                if (n >= kMmaStages) ok = mbar_wait(bar_empty + 8 * s, ((n / kMmaStages) - 1) & 1, abort_word, status);
                if (!ok) break;
                const uint32_t full = bar_full + 8 * s;
                // this lane's sub-tile (tensor-map mode: lanes 2 s and 2 s + 1 copy K and V of sub-tile s; row mode:
                // every lane looks at the stage's only sub-tile) and its block: ids of the current or next window
                const int my_sub = kTma ? (lane >> 1) : 0;
                const int my_t = t0 + kMmaTileTokens * my_sub;
                const bool my_valid = my_sub < kSubs && kMmaTileTokens * my_sub < rows;
                const int my_blk = my_valid ? (block_shift >= 0 ? (my_t >> block_shift) : (my_t / block_size)) : blk;
                const int id_a = __shfl_sync(0xffffffffu, ids, (my_blk - win) & 31);
                const int id_b = __shfl_sync(0xffffffffu, ids_next, (my_blk - win) & 31);
                const int id = my_blk - win < 32 ? id_a : id_b;
                const int slot = my_t - my_blk * block_size;
                const bool bad = my_valid && (unsigned)id >= (unsigned)num_blocks;
                bool copy = rows > 0;
                if (__any_sync(0xffffffffu, bad)) {  // nothing is copied and the tile is skipped
                    *(volatile int32_t*)status = 2;
                    copy = false;
                }
                const int n_subs = (rows + kMmaTileTokens - 1) / kMmaTileTokens;
                if (lane == 0) {
                    sdesc[s].item = it;
                    sdesc[s].t0 = t0;
                    sdesc[s].rows = copy ? rows : 0;
                    sdesc[s].flags = (ti == 0 ? kFlagFirst : 0) | (ti == ntiles - 1 ? kFlagLast : 0);
                    if (copy)
                        mbar_expect_tx(full, kTma ? (uint32_t)(n_subs * 2 * kSubBytes) : (uint32_t)rows * 2u * kMmaRowBytes);
                    else
                        mbar_arrive(full);
                }
                __syncwarp();  // descriptor and expected byte count are posted before any copy can complete
                if (copy) {
                    if (kTma) {
                        // whole boxes of 16 token rows: a sub-tile lies inside one block, so rows past the context's
                        // end are in bounds (the consumers clear them in V and mask them in the scores)
                        if (my_valid)
                            tensor_g2s(ring + s * kStageBytes + (lane & 1) * kVOff + my_sub * kSubBytes,
                                       (lane & 1) ? &vmap : &kmap, id * block_size + slot, full, kv_policy);
                    } else {
                        const int r = lane & 15;
                        if (r < rows) {
                            const int64_t off = ((int64_t)id * block_size + slot + r) * (kMmaRowBytes / 2);  // elements
                            const uint32_t dst = ring + s * kStageBytes + (lane < 16 ? 0 : kVOff) + r * kMmaPitch;
                            bulk_g2s(dst, (lane < 16 ? kpool : vpool) + off, kMmaRowBytes, full, kv_policy);
                        }
                    }
                }
                if (prime_next && ti == min(1, ntiles - 1)) {
                    // the next item's first two block-id windows, under the copies just issued
                    const int32_t* ntable = batch.block_tables + (int64_t)pre_item.b * batch.table_stride;
                    const int nlast = (max(pre_item.t_end, 1) - 1) / block_size;
                    const int nwin = block_shift >= 0 ? (pre_item.t_begin >> block_shift) : (pre_item.t_begin / block_size);
                    pre_ids = nwin + lane <= nlast ? __ldg(ntable + nwin + lane) : 0;
                    pre_ids_next = nwin + 32 + lane <= nlast ? __ldg(ntable + nwin + 32 + lane) : 0;
                    pre_it = it + 1;
                }
            }
            if (!dynamic) ++it;
        }
        if (ok) {  // end-of-stream marker
            const int s = n % kMmaStages;
            if (n >= kMmaStages) ok = mbar_wait(bar_empty + 8 * s, ((n / kMmaStages) - 1) & 1, abort_word, status);
            if (ok && lane == 0) {
                sdesc[s].flags = kFlagEnd;
                mbar_arrive(bar_full + 8 * s);
            }
        }
        // the last CTA to finish fetching re-arms the chunk counter for the lane's next launch
        dep_wait();
        if (lane == 0) {
            __threadfence();
            if (atomicAdd(counter + 1, 1) == (int)gridDim.x - 1) {
                atomicExch(counter, 0);
                atomicExch(counter + 1, 0);
            }
        }
    } else {
        // ------------------------------------------------ consumers: warp = (KV head, 16-token sub-tile of the stage)
        const int h = warp % HKV;
        const int sub = warp / HKV;
        const int g = lane >> 2;  // mma row = query head inside the group (real if g < G)
        const int t = lane & 3;
        const int ld_row = lane & 7;
        const int ld_mat = lane >> 3;
        // K, no transpose: matrices {tok 0-7, d lo}, {tok 0-7, d hi}, {tok 8-15, d lo}, {tok 8-15, d hi}
        // V, transposed on load: matrices {tok 0-7, d lo}, {tok 8-15, d lo}, {tok 0-7, d hi}, {tok 8-15, d hi}
        const int k_tok = ld_row + ((ld_mat & 2) ? 8 : 0), k_half = ld_mat & 1;
        const int v_tok = ld_row + ((ld_mat & 1) ? 8 : 0), v_half = (ld_mat & 2) ? 1 : 0;
        // Row-copy mode: token rows at a 2064-byte pitch, head h at byte 256 h.  Tensor-map mode: head h is the
        // 128-byte chunks 2h and 2h + 1, each [16 tokens][128 B]; the 16-byte unit u of a token row sits at
        // unit u ^ (token mod 8).  k_x[u] / v_x[u]: byte offset of the lane's unit for dims 32 u .. 32 u + 15.
        const uint32_t k_lane_off = kTma ? (uint32_t)(sub * kSubBytes + 2 * h * 2048 + k_tok * 128)
                                         : (uint32_t)(k_tok * kMmaPitch + h * 256 + k_half * 16);
        const uint32_t v_lane_off = kTma ? (uint32_t)(kVOff + sub * kSubBytes + 2 * h * 2048 + v_tok * 128)
                                         : (uint32_t)(kVOff + v_tok * kMmaPitch + h * 256 + v_half * 16);
        uint32_t k_x[4], v_x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            k_x[u] = kTma ? (uint32_t)(((2 * u + k_half) ^ ld_row) << 4) : (uint32_t)(64 * u);
            v_x[u] = kTma ? (uint32_t)(((2 * u + v_half) ^ ld_row) << 4) : (uint32_t)(64 * u);
        }
        uint32_t qa[8][2];
        float o[16][2];
        float m_run = kNegBig, l_run = 0.f;
        int item_b = 0, item_part = 0, item_nparts = 1;
        volatile int32_t* pending = reinterpret_cast<volatile int32_t*>(ctrl + 128) + warp * 16;
        int n_pend = 0;
        int xphase = 0;  // item ends seen so far: phase of the exchange barriers
        bool ok = true;
#pragma unroll
        for (int j = 0; j < 8; ++j) qa[j][0] = qa[j][1] = 0u;
#pragma unroll
        for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = 0.f;

        for (int n = 0;; ++n) {
            const int s = n % kMmaStages;
            ok = mbar_wait(bar_full + 8 * s, (n / kMmaStages) & 1, abort_word, status);
            if (!ok) break;
            const int flags = sdesc[s].flags;
            if (flags & kFlagEnd) break;
            const int rows = max(0, min(kMmaTileTokens, sdesc[s].rows - kMmaTileTokens * sub));  // of this warp's sub-tile
            if (flags & kFlagFirst) {
                const AttnItem* ip = batch.items + sdesc[s].item;
                item_b = ip->b;
                item_part = ip->part;
                item_nparts = ip->n_parts;
                const __nv_bfloat16* qrow = q + ((int64_t)item_b * Hq + h * G + g) * kMmaD;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    qa[j][0] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 2 * t) : 0u;
                    qa[j][1] = g < G ? *reinterpret_cast<const uint32_t*>(qrow + 16 * j + 8 + 2 * t) : 0u;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) o[i][0] = o[i][1] = 0.f;
                m_run = kNegBig;
                l_run = 0.f;
            }
            if (rows > 0) {
                const uint32_t base = ring + s * kStageBytes;
                if (kTma && rows < kMmaTileTokens) {
                    // the box brought whole token rows past the context's end: clear this head's part of them in V
                    // (a zero weight times a non-finite leftover would poison the row's output)
                    if (lane < 16)
                        for (int r = rows; r < kMmaTileTokens; ++r)
                            *reinterpret_cast<uint4*>(smem + s * kStageBytes + kVOff + sub * kSubBytes +
                                                      (2 * h + (lane >> 3)) * 2048 + r * 128 + (lane & 7) * 16) =
                                make_uint4(0, 0, 0, 0);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // before the stage is refilled
                    __syncwarp();
                }
                // scores of row g: s0 -> tokens 2t, 2t+1; s1 -> tokens 8+2t, 9+2t
                float s00 = 0.f, s01 = 0.f, s10 = 0.f, s11 = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(base + k_lane_off + (kTma ? (j >> 2) * 2048 : (j >> 2) * 128) + (kTma ? k_x[j & 3] : 32 * (j & 3)),
                            b0, b1, b2, b3);
                    mma_k16(s00, s01, qa[j][0], qa[j][1], b0, b1, s00, s01);
                    mma_k16(s10, s11, qa[j][0], qa[j][1], b2, b3, s10, s11);
                }
                const float x0 = s00 * scale_log2e, x1 = s01 * scale_log2e;
                const float x2 = s10 * scale_log2e, x3 = s11 * scale_log2e;
                const bool v0 = 2 * t < rows, v1 = 2 * t + 1 < rows, v2 = 8 + 2 * t < rows, v3 = 9 + 2 * t < rows;
                float mx = kNegBig;
                if (v0) mx = x0;
                if (v1) mx = fmaxf(mx, x1);
                if (v2) mx = fmaxf(mx, x2);
                if (v3) mx = fmaxf(mx, x3);
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                const float m_new = fmaxf(m_run, mx);
                const float alpha = exp2f(m_run - m_new);
                m_run = m_new;
                const float p0 = v0 ? exp2f(x0 - m_new) : 0.f;
                const float p1 = v1 ? exp2f(x1 - m_new) : 0.f;
                const float p2 = v2 ? exp2f(x2 - m_new) : 0.f;
                const float p3 = v3 ? exp2f(x3 - m_new) : 0.f;
                l_run = l_run * alpha + (p0 + p1 + p2 + p3);
                const uint32_t pa0 = pack_bf16(p0, p1);  // A operand: row g, tokens 2t, 2t+1
                const uint32_t pa2 = pack_bf16(p2, p3);  // row g, tokens 8+2t, 9+2t
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(base + v_lane_off + (kTma ? (c >> 2) * 2048 : (c >> 2) * 128) + (kTma ? v_x[c & 3] : 32 * (c & 3)),
                              b0, b1, b2, b3);
                    mma_k16(o[2 * c][0], o[2 * c][1], pa0, pa2, b0, b1, o[2 * c][0] * alpha, o[2 * c][1] * alpha);
                    mma_k16(o[2 * c + 1][0], o[2 * c + 1][1], pa0, pa2, b2, b3, o[2 * c + 1][0] * alpha,
                            o[2 * c + 1][1] * alpha);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * s);

            if ((flags & kFlagLast) && kSubs > 1) {
                // the warps of a head combine their softmax states: the others hand theirs to the warp of sub-tile 0
                // (same fragment layout in every warp, so lane i combines with lane i)
                if (sub > 0) {
                    if (xphase > 0) ok = mbar_wait(bar_xempty + 8 * h, (xphase - 1) & 1, abort_word, status);
                    if (!ok) break;
                    float* mine = xchg + ((size_t)((sub - 1) * HKV + h) * 32 + lane) * 34;
                    mine[0] = m_run;
                    mine[1] = l_run;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        mine[2 + 2 * i] = o[i][0];
                        mine[3 + 2 * i] = o[i][1];
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_xfull + 8 * h);
                } else {
                    ok = mbar_wait(bar_xfull + 8 * h, xphase & 1, abort_word, status);
                    if (!ok) break;
#pragma unroll 1
                    for (int ss = 1; ss < kSubs; ++ss) {
                        const float* other = xchg + ((size_t)((ss - 1) * HKV + h) * 32 + lane) * 34;
                        const float m_o = other[0];
                        const float m_new = fmaxf(m_run, m_o);
                        const float a = exp2f(m_run - m_new), b = exp2f(m_o - m_new);
                        m_run = m_new;
                        l_run = l_run * a + other[1] * b;
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            o[i][0] = o[i][0] * a + other[2 + 2 * i] * b;
                            o[i][1] = o[i][1] * a + other[3 + 2 * i] * b;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_xempty + 8 * h);
                }
                ++xphase;
            }
            if ((flags & kFlagLast) && sub == 0) {
                float L = l_run;
                L += __shfl_xor_sync(0xffffffffu, L, 1);
                L += __shfl_xor_sync(0xffffffffu, L, 2);
                if (g < G) {
                    const int hq = h * G + g;
                    if (item_nparts == 1) {
                        const float inv = L > 0.f ? 1.f / L : 0.f;
                        __nv_bfloat16* orow = out + ((int64_t)item_b * Hq + hq) * kMmaD;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            *reinterpret_cast<uint32_t*>(orow + 8 * i + 2 * t) = pack_bf16(o[i][0] * inv, o[i][1] * inv);
                        if (lse != nullptr && t == 0)
                            lse[(int64_t)item_b * Hq + hq] = L > 0.f ? (m_run + log2f(L)) * kLn2 : -CUDART_INF_F;
                    } else {
                        dep_wait();
                        float* pr = partials + ((int64_t)item_part * Hq + hq) * kMmaPartStride;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            *reinterpret_cast<float2*>(pr + 8 * i + 2 * t) = make_float2(o[i][0], o[i][1]);
                        if (t == 0) {
                            pr[kMmaD] = m_run;
                            pr[kMmaD + 1] = L;
                        }
                    }
                }
                if (item_nparts > 1) {
                    dep_wait();
                    // Split-KV fix-up: the warp that delivers the last part of a (row, KV head) combines the
                    // parts.  Combining costs a few round trips to L2 during which this warp would hold up the
                    // CTA's ring, so the row is only noted here and combined after the CTA's last tile.
                    // (Publishing and announcing the part right here costs two such round trips already, about
                    // 3.5 us under full memory load; putting them off to the CTA's end as well was measured and is
                    // worse: every row is then completed, and combined, in the launch's last microseconds.)
                    fence_acq_rel_gpu();
                    __syncwarp();
                    int prev = 0;
                    if (lane == 0) prev = atomicAdd(row_done + item_b * HKV + h, 1);
                    prev = __shfl_sync(0xffffffffu, prev, 0);
                    if (prev == item_nparts - 1) {
                        if (n_pend < kMmaMaxPending) {
                            if (lane == 0) pending[n_pend] = item_b;
                            ++n_pend;
                        } else {
                            merge_row<G, HKV>(item_b, h, lane, batch, partials, out, lse, row_done);
                        }
                    }
                }
            }
        }
        if (ok) {
            __syncwarp();
            for (int p = 0; p < n_pend; ++p) merge_row<G, HKV>(pending[p], h, lane, batch, partials, out, lse, row_done);
        }
    }
    // A launch does not complete before the launch it was made programmatically dependent on has completed:
    // work enqueued after this launch may rely on both.  (Returns at once for ordinary launches.)
    dep_wait();
}

template <int G, int HKV>
cudaError_t launch_mma(const AttnShape& sh, const void* kpool, const void* vpool, const AttnTensorMaps* maps, const void* q,
                       void* out, float* lse, const AttnBatch& batch, int32_t lane, float* partials, int32_t* sched,
                       int32_t* row_done, int32_t* d_status, int dep_mode, cudaStream_t stream) {
    const float scale_log2e = 1.4426950408889634f / sqrtf((float)kMmaD);
    static_assert(sizeof(CUtensorMap) == sizeof(maps->k), "AttnTensorMaps must hold driver tensor maps");
    if (HKV != kMmaHkv && maps == nullptr) return cudaErrorNotSupported;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)batch.n_cta[lane]);
    cfg.blockDim = dim3(kMmaThreads);
    cfg.dynamicSmemBytes = (size_t)mma_smem_bytes(maps != nullptr, HKV);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dep_mode != 0 ? 1 : 0;
    const int32_t wait_first = dep_mode == 2 ? 1 : 0;
    CUtensorMap km, vm;
    if (maps != nullptr) {
        memcpy(&km, maps->k, sizeof km);
        memcpy(&vm, maps->v, sizeof vm);
    } else {
        memset(&km, 0, sizeof km);
        memset(&vm, 0, sizeof vm);
    }
    const __nv_bfloat16* kp = (const __nv_bfloat16*)kpool;
    const __nv_bfloat16* vp = (const __nv_bfloat16*)vpool;
    const __nv_bfloat16* qp = (const __nv_bfloat16*)q;
    __nv_bfloat16* op = (__nv_bfloat16*)out;
    const int32_t shift = shift_of(sh.block_size);
    if (maps != nullptr)
        return cudaLaunchKernelEx(&cfg, decode_attn_mma_kernel<G, HKV, true>, kp, vp, km, vm, qp, op, lse, batch, lane,
                                  sh.block_size, shift, sh.num_blocks, partials, sched, row_done, scale_log2e, d_status, wait_first);
    if constexpr (HKV == kMmaHkv)
        return cudaLaunchKernelEx(&cfg, decode_attn_mma_kernel<G, HKV, false>, kp, vp, km, vm, qp, op, lse, batch, lane,
                                  sh.block_size, shift, sh.num_blocks, partials, sched, row_done, scale_log2e, d_status, wait_first);
    return cudaErrorNotSupported;
}

template <int G>
cudaError_t launch_mma_hkv(const AttnShape& sh, const void* kpool, const void* vpool, const AttnTensorMaps* maps,
                           const void* q, void* out, float* lse, const AttnBatch& batch, int32_t lane, float* partials,
                           int32_t* sched, int32_t* row_done, int32_t* d_status, int dep_mode,
                           cudaStream_t stream) {
    switch (sh.num_kv_heads) {
#define PS_HKV_CASE(HH)                                                                                              \
    case HH:                                                                                                         \
        return launch_mma<G, HH>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status, \
                                 dep_mode, stream);
        PS_HKV_CASE(1) PS_HKV_CASE(2) PS_HKV_CASE(4) PS_HKV_CASE(8)
#undef PS_HKV_CASE
    }
    return cudaErrorNotSupported;
}

}  // namespace

size_t attn_partial_bytes(const AttnShape& sh, int32_t max_parts) {
    return (size_t)max_parts * sh.num_q_heads * (sh.head_dim + 4) * sizeof(float);
}

bool attn_mma_supported(const AttnShape& sh) {
    const int G = sh.num_q_heads / sh.num_kv_heads;
    const int hkv = sh.num_kv_heads;
    return sh.head_dim == kMmaD && (hkv == 1 || hkv == 2 || hkv == 4 || hkv == 8) && G >= 1 && G <= 8 &&
           sh.block_size % kMmaTileTokens == 0;
}

int32_t attn_mma_tile_tokens(const AttnShape& sh) { return kMmaTileTokens * mma_subs(sh.num_kv_heads); }

cudaError_t attn_init() {
    cudaError_t e;
#define PS_MMA_ATTR_ONE(GG, HH, TT)                                                                                   \
    e = cudaFuncSetAttribute(decode_attn_mma_kernel<GG, HH, TT>, cudaFuncAttributeMaxDynamicSharedMemorySize,         \
                             mma_smem_bytes(TT, HH));                                                                 \
    if (e != cudaSuccess) return e;
#define PS_MMA_ATTR(GG)                                                                                               \
    PS_MMA_ATTR_ONE(GG, 8, false) PS_MMA_ATTR_ONE(GG, 8, true) PS_MMA_ATTR_ONE(GG, 4, true) PS_MMA_ATTR_ONE(GG, 2, true) \
        PS_MMA_ATTR_ONE(GG, 1, true)
    PS_MMA_ATTR(1) PS_MMA_ATTR(2) PS_MMA_ATTR(3) PS_MMA_ATTR(4) PS_MMA_ATTR(5) PS_MMA_ATTR(6) PS_MMA_ATTR(7) PS_MMA_ATTR(8)
#undef PS_MMA_ATTR
#undef PS_MMA_ATTR_ONE
    return cudaSuccess;
}

// Tensor maps over one layer's pools, seen as rank-3 tensors (64 elements = 128 bytes, token row, 128-byte chunk
// of the row): strides one token row (256 bytes per KV head) and 128 bytes per chunk, box 64 x 16 token rows x all
// chunks of a row, 128-byte swizzle.  The driver entry point is looked up at run time (the library does not link against the driver).
cudaError_t attn_make_tensor_maps(const AttnShape& sh, const void* kpool, const void* vpool, AttnTensorMaps* out) {
    if (!attn_mma_supported(sh)) return cudaErrorNotSupported;
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (encode == nullptr) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || fn == nullptr) return cudaErrorNotSupported;
        encode = (EncodeFn)fn;
    }
    const cuuint64_t row_bytes = (cuuint64_t)sh.num_kv_heads * kMmaD * 2;
    const cuuint64_t dims[3] = {64, (cuuint64_t)sh.num_blocks * (cuuint64_t)sh.block_size, row_bytes / 128};
    const cuuint64_t strides[2] = {row_bytes, 128};   // bytes: token row, then chunk of the row
    const cuuint32_t box[3] = {64, (cuuint32_t)kMmaTileTokens, (cuuint32_t)(row_bytes / 128)};
    const cuuint32_t estr[3] = {1, 1, 1};
    const void* pools[2] = {kpool, vpool};
    unsigned char* dst[2] = {out->k, out->v};
    for (int t = 0; t < 2; ++t) {
        CUtensorMap m;
        const CUresult r = encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(pools[t]), dims, strides, box,
                                  estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
        memcpy(dst[t], &m, sizeof m);
    }
    return cudaSuccess;
}

cudaError_t launch_decode_attn(int kernel, const AttnShape& sh, const void* kpool, const void* vpool,
                               const AttnTensorMaps* maps, const void* q, void* out, float* lse, const AttnBatch& batch,
                               int32_t lane, float* partials, int32_t* sched, int32_t* row_done, int32_t* d_status,
                               int dep_mode, cudaStream_t stream) {
    if (lane < 0 || lane > 1) return cudaErrorInvalidValue;
    const int item_begin = batch.lane_items[lane];
    const int n_items = batch.lane_items[lane + 1] - item_begin;
    if (n_items <= 0) return cudaSuccess;
    const int G = sh.num_q_heads / sh.num_kv_heads;
    if (kernel == 2) {
        if (!attn_mma_supported(sh) || batch.n_cta[lane] <= 0 || sched == nullptr || row_done == nullptr)
            return cudaErrorNotSupported;
        switch (G) {
            case 1: return launch_mma_hkv<1>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 2: return launch_mma_hkv<2>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 3: return launch_mma_hkv<3>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 4: return launch_mma_hkv<4>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 5: return launch_mma_hkv<5>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 6: return launch_mma_hkv<6>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 7: return launch_mma_hkv<7>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
            case 8: return launch_mma_hkv<8>(sh, kpool, vpool, maps, q, out, lse, batch, lane, partials, sched, row_done, d_status,
                                       dep_mode, stream);
        }
        return cudaErrorNotSupported;
    }
    if (kernel != 1) return cudaErrorNotSupported;
#define PS_SIMT_CASE(DD, GG)                                                                                       \
    if (sh.head_dim == DD && G == GG)                                                                              \
        return launch_simt<DD, GG>(sh, kpool, vpool, q, out, lse, batch, item_begin, n_items, partials, d_status, \
                                   stream);
    PS_SIMT_CASE(128, 1) PS_SIMT_CASE(128, 2) PS_SIMT_CASE(128, 3) PS_SIMT_CASE(128, 4)
    PS_SIMT_CASE(128, 5) PS_SIMT_CASE(128, 6) PS_SIMT_CASE(128, 7) PS_SIMT_CASE(128, 8)
    PS_SIMT_CASE(64, 1) PS_SIMT_CASE(64, 2) PS_SIMT_CASE(64, 3) PS_SIMT_CASE(64, 4)
    PS_SIMT_CASE(64, 5) PS_SIMT_CASE(64, 6) PS_SIMT_CASE(64, 7) PS_SIMT_CASE(64, 8)
#undef PS_SIMT_CASE
    return cudaErrorNotSupported;
}

cudaError_t launch_attn_merge(const AttnShape& sh, void* out, float* lse, const AttnBatch& batch,
                              const float* partials, int32_t lane, cudaStream_t stream) {
    if (batch.batch <= 0) return cudaSuccess;
    dim3 grid((unsigned)batch.batch, (unsigned)sh.num_q_heads);
    if (sh.head_dim == 128)
        attn_merge_kernel<128><<<grid, 128, 0, stream>>>((__nv_bfloat16*)out, lse, batch, sh.num_q_heads, partials, lane);
    else if (sh.head_dim == 64)
        attn_merge_kernel<64><<<grid, 64, 0, stream>>>((__nv_bfloat16*)out, lse, batch, sh.num_q_heads, partials, lane);
    else
        return cudaErrorNotSupported;
    return cudaGetLastError();
}

}  // namespace ps
