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

__global__ void __launch_bounds__(256)
combine_kernel(const __nv_bfloat16 *__restrict__ obuf, const int32_t *__restrict__ inv,
               const float *__restrict__ topk_w, const __nv_bfloat16 *__restrict__ x, int K, int d,
               int copy_experts, __nv_bfloat16 *__restrict__ y) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    __shared__ int32_t s_pos[kMaxTopK];
    __shared__ float s_w[kMaxTopK];
    __shared__ float s_zero_mass;
    if (threadIdx.x < K) {
        s_pos[threadIdx.x] = inv[(size_t)t * K + threadIdx.x];
        s_w[threadIdx.x] = topk_w[(size_t)t * K + threadIdx.x];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float zm = 0.f;
        for (int k = 0; k < K; ++k) if (s_pos[k] < 0) zm += s_w[k];
        s_zero_mass = zm;
    }
    __syncthreads();
    for (int c = blockIdx.y * blockDim.x + threadIdx.x; c < d / 8; c += gridDim.y * blockDim.x) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.f;
#pragma unroll 4
        for (int k = 0; k < K; ++k) {
            const int p = s_pos[k];
            if (p >= 0) fma_bf16x8(acc, s_w[k], __ldg(reinterpret_cast<const uint4 *>(obuf + (size_t)p * d) + c));
        }
        if (copy_experts && s_zero_mass != 0.f)
            fma_bf16x8(acc, s_zero_mass, __ldg(reinterpret_cast<const uint4 *>(x + (size_t)t * d) + c));
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
    const zeda_moe_config_t &c = h->cfg;
    // one 16-byte chunk per thread; small batches spread a row over several CTAs to fill the SMs
    const int chunks = c.d_model / 8;
    const int threads = (T >= 1024 && chunks >= 256) ? 256 : (T >= 256 && chunks >= 128 ? 128 : 64);
    const int gy = (chunks + threads - 1) / threads;
    const cudaError_t e = launch_kernel(h->pdl, combine_kernel, dim3(T, gy), dim3(threads), 0, s, h->ws.obuf, h->ws.inv,
                                        h->ws.topk_w, x, c.top_k, c.d_model, (int)(c.expert_kind == ZEDA_EXPERT_COPY), y);
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
