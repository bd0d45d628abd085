// Glue between stacked MoE blocks: residual update and gain-free RMS normalisation in one pass.
//
// The paper's layer ends at Eq. 1; a stack of such layers (its models have 48 MoE layers,
// Section 4.2) needs something between them.  This kernel is that something for the layer-stack
// workload: r <- bf16(r + y) (y = the previous layer's output, absent before the first layer) and
// h = r / sqrt(mean(r^2) + eps), the next layer's input.  One CTA per token row, 16-byte accesses,
// the row held in registers between the two passes, fp32 arithmetic, a fixed-order reduction.
#include "zeda_internal.h"

namespace zeda {

namespace {

constexpr int kGlueThreads = 256;
constexpr int kGlueChunks = 4;  // 16-byte chunks per thread: rows of up to 256 * 4 * 8 = 8192 elements

__global__ void __launch_bounds__(kGlueThreads)
residual_rmsnorm_kernel(__nv_bfloat16 *__restrict__ r, const __nv_bfloat16 *__restrict__ y,
                        __nv_bfloat16 *__restrict__ h, int d, float eps) {
    pdl_launch_dependents();
    pdl_wait();
    const size_t row = (size_t)blockIdx.x * d;
    const int chunks = d / 8;
    float v[kGlueChunks][8];
    float ss = 0.f;
#pragma unroll
    for (int i = 0; i < kGlueChunks; ++i) {
        const int c = threadIdx.x + i * kGlueThreads;
        if (c < chunks) {
            const uint4 a = *reinterpret_cast<const uint4 *>(r + row + 8 * c);
            const uint32_t au[4] = {a.x, a.y, a.z, a.w};
            uint32_t bu[4] = {0, 0, 0, 0};
            if (y) {
                const uint4 b = __ldg(reinterpret_cast<const uint4 *>(y + row + 8 * c));
                bu[0] = b.x; bu[1] = b.y; bu[2] = b.z; bu[3] = b.w;
            }
            uint4 o;
            uint32_t *ou = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float s0 = __uint_as_float(au[j] << 16) + __uint_as_float(bu[j] << 16);
                const float s1 = __uint_as_float(au[j] & 0xffff0000u) + __uint_as_float(bu[j] & 0xffff0000u);
                const __nv_bfloat162 p = __floats2bfloat162_rn(s0, s1);
                ou[j] = *reinterpret_cast<const uint32_t *>(&p);
                v[i][2 * j] = __low2float(p);       // the normalisation sees the stored (rounded) residual
                v[i][2 * j + 1] = __high2float(p);
                ss = fmaf(v[i][2 * j], v[i][2 * j], ss);
                ss = fmaf(v[i][2 * j + 1], v[i][2 * j + 1], ss);
            }
            if (y) *reinterpret_cast<uint4 *>(r + row + 8 * c) = o;
        }
    }
    __shared__ float warp_ss[kGlueThreads / 32];
    __shared__ float s_scale;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((threadIdx.x & 31) == 0) warp_ss[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < kGlueThreads / 32; ++w) t += warp_ss[w];
        s_scale = rsqrtf(t / (float)d + eps);
    }
    __syncthreads();
    const float scale = s_scale;
#pragma unroll
    for (int i = 0; i < kGlueChunks; ++i) {
        const int c = threadIdx.x + i * kGlueThreads;
        if (c < chunks) {
            uint4 o;
            uint32_t *ou = reinterpret_cast<uint32_t *>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const __nv_bfloat162 p = __floats2bfloat162_rn(v[i][2 * j] * scale, v[i][2 * j + 1] * scale);
                ou[j] = *reinterpret_cast<const uint32_t *>(&p);
            }
            *reinterpret_cast<uint4 *>(h + row + 8 * c) = o;
        }
    }
}

}  // namespace
}  // namespace zeda

extern "C" zeda_status_t zeda_residual_rmsnorm(void *r, const void *y, void *h, int32_t T, int32_t d_model, float eps,
                                               void *stream) {
    using namespace zeda;
    if (T == 0) return ZEDA_OK;
    if (T < 0) { set_error("T must be >= 0"); return ZEDA_ERR_INVALID_ARG; }
    if (d_model < 64 || d_model % 64 || d_model > 8192) {
        set_error("d_model must be a multiple of 64 in [64, 8192]");
        return ZEDA_ERR_UNSUPPORTED;
    }
    if (!r || !h) { set_error("r and h are required"); return ZEDA_ERR_INVALID_ARG; }
    if ((reinterpret_cast<uintptr_t>(r) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(h)) & 15u) {
        set_error("r, y and h must be 16-byte aligned");
        return ZEDA_ERR_INVALID_ARG;
    }
    if (!(eps >= 0.f)) { set_error("eps must be >= 0"); return ZEDA_ERR_INVALID_ARG; }
    const cudaError_t e = launch_kernel(true, residual_rmsnorm_kernel, dim3(T), dim3(kGlueThreads), 0,
                                        static_cast<cudaStream_t>(stream), static_cast<__nv_bfloat16 *>(r),
                                        static_cast<const __nv_bfloat16 *>(y), static_cast<__nv_bfloat16 *>(h),
                                        (int)d_model, eps);
    if (e != cudaSuccess) { set_error("zeda_residual_rmsnorm launch: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
    return ZEDA_OK;
}
