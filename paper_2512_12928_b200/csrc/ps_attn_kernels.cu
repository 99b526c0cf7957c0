// Paged grouped-query decode attention: the per-layer computation that the pipelined reload
// hides under (Section 4.3, "Pipelined Reloading": layer i computes while layer i+1 loads).
//
//   out[b][h] = softmax_t( q[b][h] . K[t][h/G] / sqrt(D) ) . V[t][h/G],   t < ctx_len[b]
//
// bf16 inputs, fp32 accumulation, softmax in base 2 with log2(e)/sqrt(D) folded into q.  The
// work is split over the KV axis into items of a bounded token count; an item that is the only
// one of its row writes the final output, otherwise it writes an unnormalised partial (running
// max, running sum, D accumulators per head) that the merge kernel combines.
//
// The kernel is HBM-bound (G flop per KV byte), so the SIMT kernel below spends its effort on
// 16-byte coalesced loads with many of them in flight; softmax statistics are reduced with warp
// shuffles inside the group of lanes that shares a token.
#include <cuda_bf16.h>
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

}  // namespace

size_t attn_partial_bytes(const AttnShape& sh, int32_t max_parts) {
    return (size_t)max_parts * sh.num_q_heads * (sh.head_dim + 2) * sizeof(float);
}

bool attn_mma_supported(const AttnShape&) { return false; }

cudaError_t attn_init() { return cudaSuccess; }

cudaError_t launch_decode_attn(int kernel, const AttnShape& sh, const void* kpool, const void* vpool, const void* q,
                               void* out, float* lse, const AttnBatch& batch, int32_t item_begin, int32_t item_end,
                               float* partials, int32_t* d_status, cudaStream_t stream) {
    const int n_items = item_end - item_begin;
    if (n_items <= 0) return cudaSuccess;
    if (kernel != 1) return cudaErrorNotSupported;
    const int G = sh.num_q_heads / sh.num_kv_heads;
#define PS_SIMT_CASE(DD, GG)                                                                                       \
    if (sh.head_dim == DD && G == GG)                                                                              \
        return launch_simt<DD, GG>(sh, kpool, vpool, q, out, lse, batch, item_begin, n_items, partials, d_status, \
                                   stream);
    PS_SIMT_CASE(128, 1) PS_SIMT_CASE(128, 2) PS_SIMT_CASE(128, 4) PS_SIMT_CASE(128, 8)
    PS_SIMT_CASE(64, 1) PS_SIMT_CASE(64, 2) PS_SIMT_CASE(64, 4) PS_SIMT_CASE(64, 8)
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
