// Weighted combine back to token order: the sum of Eq. 1,
//   y[t] = sum over the slots k of token t that hold a normal expert of g~[t,k] * O[inv[t,k]],
// taken in slot order in fp32 and rounded once to bf16.  It is a gather, not a scatter with
// atomics, so the result is the same bits on every run, and a token with no surviving slot gets
// +0 in every element.  The copy-expert variant (Appendix B) adds (sum of zero-slot weights) * x[t].
#include "zeda_internal.h"

namespace zeda {

namespace {

__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], float w, const uint4 &v) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
        acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xffff0000u), acc[2 * i + 1]);
    }
}

// One CTA per token, kCombineThreads threads, each owning every kCombineThreads-th 16-byte chunk of
// the row (small CTAs: many tokens in flight per SM hide the dependent slot-table and row loads).
constexpr int kCombineThreads = 64;

// The token's slot table: positions of its surviving slots in the expert outputs (-1 for a zero slot),
// the gate weights, and the summed weight of the zero slots.
struct SlotTable {
    int32_t pos[kMaxTopK];
    float w[kMaxTopK];
    float zero_mass;
};

__device__ __forceinline__ void load_slot_table(SlotTable &st, const int32_t *__restrict__ inv,
                                                const float *__restrict__ topk_w, int t, int K) {
    // every thread reads the table itself (K <= 16 entries, one cache line each way)
    st.zero_mass = 0.f;
#pragma unroll
    for (int k = 0; k < kMaxTopK; ++k) {
        st.pos[k] = -1;
        st.w[k] = 0.f;
        if (k < K) {
            st.pos[k] = __ldg(inv + (size_t)t * K + k);
            st.w[k] = __ldg(topk_w + (size_t)t * K + k);
            if (st.pos[k] < 0) st.zero_mass += st.w[k];
        }
    }
}

// 16-byte chunk c of y[t] in fp32: the sum of Eq. 1 in slot order.
__device__ __forceinline__ void combine_chunk(float (&acc)[8], const SlotTable &st, const __nv_bfloat16 *__restrict__ obuf,
                                              const __nv_bfloat16 *__restrict__ x, int t, int c, int K, int d,
                                              int copy_experts) {
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
    for (int k0 = 0; k0 < kMaxTopK; k0 += 8) {  // eight row loads are issued before the first use
        if (k0 >= K) break;
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (k0 + k < K && st.pos[k0 + k] >= 0)
                v[k] = __ldg(reinterpret_cast<const uint4 *>(obuf + (size_t)st.pos[k0 + k] * d) + c);
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (k0 + k < K && st.pos[k0 + k] >= 0) fma_bf16x8(acc, st.w[k0 + k], v[k]);
    }
    if (copy_experts && st.zero_mass != 0.f)
        fma_bf16x8(acc, st.zero_mass, __ldg(reinterpret_cast<const uint4 *>(x + (size_t)t * d) + c));
}

__global__ void __launch_bounds__(kCombineThreads, 16)
combine_kernel(const __nv_bfloat16 *__restrict__ obuf, const int32_t *__restrict__ inv,
               const float *__restrict__ topk_w, const __nv_bfloat16 *__restrict__ x, int K, int d,
               int copy_experts, __nv_bfloat16 *__restrict__ y) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    SlotTable st;
    load_slot_table(st, inv, topk_w, t, K);
    for (int c = blockIdx.y * kCombineThreads + threadIdx.x; c < d / 8; c += gridDim.y * kCombineThreads) {
        float acc[8];
        combine_chunk(acc, st, obuf, x, t, c, K, d, copy_experts);
        uint4 o;
        uint32_t *ou = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 b = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
            ou[i] = *reinterpret_cast<const uint32_t *>(&b);
        }
        reinterpret_cast<uint4 *>(y + (size_t)t * d)[c] = o;
    }
}

// The combine fused with the glue between stacked layers: instead of storing y the CTA forms
// r <- bf16(r + bf16(y)) and h = r / sqrt(mean(r^2) + eps) -- the bits a combine followed by the
// residual + norm kernel produces, without the round trip of y through memory and without the
// second launch.  The whole row sits in one CTA: rows of up to 64 * 4 * 8 = 2048 elements.
//
// Same bits: the residual + norm kernel runs 256 threads with one chunk each for such rows, reduces
// the squares over the 32 lanes of a warp by xor shuffles and adds the eight warp sums in order.
// Chunk c = thread + 64 * i here is lane (thread & 31) of warp (thread >> 5) + 2 * i there, so the
// per-iteration sums are reduced separately and stored as that warp's sum.
constexpr int kFuseChunks = 4;

__global__ void __launch_bounds__(kCombineThreads, 12)
combine_glue_kernel(const __nv_bfloat16 *__restrict__ obuf, const int32_t *__restrict__ inv,
                    const float *__restrict__ topk_w, const __nv_bfloat16 *__restrict__ x, int K, int d,
                    int copy_experts, __nv_bfloat16 *__restrict__ resid, __nv_bfloat16 *__restrict__ h_next, float eps) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    const int chunks = d / 8;
    SlotTable st;
    load_slot_table(st, inv, topk_w, t, K);
    uint32_t keep[kFuseChunks][4];  // the updated residual of this thread's chunks (bf16 pairs)
    float ss[kFuseChunks];
#pragma unroll
    for (int i = 0; i < kFuseChunks; ++i) {
        ss[i] = 0.f;
        const int c = threadIdx.x + i * kCombineThreads;
        if (c < chunks) {
            float acc[8];
            combine_chunk(acc, st, obuf, x, t, c, K, d, copy_experts);
            const uint4 rv = *(reinterpret_cast<const uint4 *>(resid + (size_t)t * d) + c);
            const uint32_t ru[4] = {rv.x, rv.y, rv.z, rv.w};
            uint4 o;
            uint32_t *ou = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 yb = __floats2bfloat162_rn(acc[2 * j], acc[2 * j + 1]);  // y as it would be stored
                const float s0 = __uint_as_float(ru[j] << 16) + __low2float(yb);
                const float s1 = __uint_as_float(ru[j] & 0xffff0000u) + __high2float(yb);
                const __nv_bfloat162 rb = __floats2bfloat162_rn(s0, s1);
                ou[j] = keep[i][j] = *reinterpret_cast<const uint32_t *>(&rb);
                const float r0 = __low2float(rb), r1 = __high2float(rb);  // the normalisation sees the stored residual
                ss[i] = fmaf(r0, r0, ss[i]);
                ss[i] = fmaf(r1, r1, ss[i]);
            }
            reinterpret_cast<uint4 *>(resid + (size_t)t * d)[c] = o;
        }
    }
    __shared__ float warp_ss[kFuseChunks * kCombineThreads / 32];
#pragma unroll
    for (int i = 0; i < kFuseChunks; ++i) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss[i] += __shfl_xor_sync(0xffffffffu, ss[i], o);
        if ((threadIdx.x & 31) == 0) warp_ss[(threadIdx.x >> 5) + (kCombineThreads / 32) * i] = ss[i];
    }
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < kFuseChunks * kCombineThreads / 32; ++w) tot += warp_ss[w];
    const float scale = rsqrtf(tot / (float)d + eps);
#pragma unroll
    for (int i = 0; i < kFuseChunks; ++i) {
        const int c = threadIdx.x + i * kCombineThreads;
        if (c < chunks) {
            uint4 o;
            uint32_t *ou = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 p = __floats2bfloat162_rn(__uint_as_float(keep[i][j] << 16) * scale,
                                                               __uint_as_float(keep[i][j] & 0xffff0000u) * scale);
                ou[j] = *reinterpret_cast<const uint32_t *>(&p);
            }
            reinterpret_cast<uint4 *>(h_next + (size_t)t * d)[c] = o;
        }
    }
}

}  // namespace

int launch_combine(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *y, cudaStream_t s) {
    return launch_combine_rows(h, h->ws.obuf, x, T, y, s);
}

// rows: the expert outputs of the call's surviving pairs in (expert, token) order
int launch_combine_rows(const zeda_moe *h, const __nv_bfloat16 *rows, const __nv_bfloat16 *x, int T, __nv_bfloat16 *y,
                        cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    // small batches spread a row over several CTAs so that the grid still covers the SMs
    const int chunks = c.d_model / 8;
    int gy = 1;
    while (T * gy < 4 * h->sm_count && gy * kCombineThreads < chunks) gy *= 2;
    const cudaError_t e = launch_kernel(h->pdl, combine_kernel, dim3(T, gy), dim3(kCombineThreads), 0, s, rows, (const int32_t *)h->ws.inv,
                                        (const float *)h->ws.topk_w, x, c.top_k, c.d_model, (int)(c.expert_kind == ZEDA_EXPERT_COPY), y);
    return e == cudaSuccess ? 1 : -1;
}

bool combine_glue_supported(const zeda_moe *h) { return h->cfg.d_model <= kCombineThreads * kFuseChunks * 8; }

// resid <- bf16(resid + y), h_next = RMSNorm(resid) with y never stored; h_next must not overlap x
// (the copy-expert variant reads x[t] while other CTAs already write their h_next rows).
int launch_combine_glue(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *resid, __nv_bfloat16 *h_next, float eps,
                        cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const cudaError_t e = launch_kernel(h->pdl, combine_glue_kernel, dim3(T), dim3(kCombineThreads), 0, s,
                                        (const __nv_bfloat16 *)h->ws.obuf, (const int32_t *)h->ws.inv, (const float *)h->ws.topk_w,
                                        x, c.top_k, c.d_model, (int)(c.expert_kind == ZEDA_EXPERT_COPY), resid, h_next, eps);
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
