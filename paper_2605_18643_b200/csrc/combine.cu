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

__global__ void __launch_bounds__(kCombineThreads, 16)
combine_kernel(const __nv_bfloat16 *__restrict__ obuf, const int32_t *__restrict__ inv,
               const float *__restrict__ topk_w, const __nv_bfloat16 *__restrict__ x, int K, int d,
               int copy_experts, __nv_bfloat16 *__restrict__ y) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    // every thread reads the token's slot table itself (K <= 16 entries, one cache line each way)
    int32_t pos[kMaxTopK];
    float w[kMaxTopK];
    float zero_mass = 0.f;
#pragma unroll
    for (int k = 0; k < kMaxTopK; ++k) {
        pos[k] = -1;
        w[k] = 0.f;
        if (k < K) {
            pos[k] = __ldg(inv + (size_t)t * K + k);
            w[k] = __ldg(topk_w + (size_t)t * K + k);
            if (pos[k] < 0) zero_mass += w[k];
        }
    }
    for (int c = blockIdx.y * kCombineThreads + threadIdx.x; c < d / 8; c += gridDim.y * kCombineThreads) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll
        for (int k0 = 0; k0 < kMaxTopK; k0 += 8) {  // eight row loads are issued before the first use
            if (k0 >= K) break;
            uint4 v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k0 + k < K && pos[k0 + k] >= 0)
                    v[k] = __ldg(reinterpret_cast<const uint4 *>(obuf + (size_t)pos[k0 + k] * d) + c);
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k0 + k < K && pos[k0 + k] >= 0) fma_bf16x8(acc, w[k0 + k], v[k]);
        }
        if (copy_experts && zero_mass != 0.f)
            fma_bf16x8(acc, zero_mass, __ldg(reinterpret_cast<const uint4 *>(x + (size_t)t * d) + c));
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

}  // namespace zeda
