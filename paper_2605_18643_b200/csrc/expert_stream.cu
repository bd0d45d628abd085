// Weight-streaming expert kernels for small per-expert batches (decode shapes).
//
// Appendix D: each normal expert has gate, up and down projections.  With a handful of rows per
// active expert the work is bound by reading each active expert's weights once from HBM, so the
// weight rows take the 16-row side of a register-level bf16 MMA (m16n8k16, fp32 accumulate) and up
// to 8 tokens take the 8-column side.  Each lane loads 16 contiguous bytes of a weight row and the
// same 16 bytes of an activation row; both operands use the same permutation of the reduction
// axis inside a 32-element step, so no shared-memory staging or transposition is needed.
//
// Work item = (chunk of <= 32 pair rows of one expert, block of weight rows); items are strided
// over all resident warps.  Zero-expert slots never reach these kernels: they were dropped by the
// compaction, so they cost neither FLOPs nor weight traffic.
#include "zeda_internal.h"

namespace zeda {

namespace {

__device__ __forceinline__ uint4 ld_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// acc[j] += W[rows] . act[token group j] over a reduction of length kdim (multiple of 32).
// row_lo / row_hi: this lane's two weight rows (MMA rows g and g+8), already offset by 8*(lane&3).
// act[j]: this lane's activation row for token group j (same offset) or nullptr.
template <int NG, int UNROLL>
__device__ __forceinline__ void stream_dot(const __nv_bfloat16 *row_lo, const __nv_bfloat16 *row_hi,
                                           const __nv_bfloat16 *const (&act)[NG], int kdim, float (&acc)[NG][4]) {
    for (int k0 = 0; k0 < kdim; k0 += 32 * UNROLL) {
        uint4 wl[UNROLL], wh[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int k = k0 + 32 * u;
            if (k < kdim) {
                wl[u] = ld_stream(row_lo + k);
                wh[u] = ld_stream(row_hi + k);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int k = k0 + 32 * u;
            if (k < kdim) {
#pragma unroll
                for (int j = 0; j < NG; ++j) {
                    uint4 a = make_uint4(0, 0, 0, 0);
                    if (act[j]) a = __ldg(reinterpret_cast<const uint4 *>(act[j] + k));
                    mma_bf16(acc[j], wl[u].x, wh[u].x, wl[u].y, wh[u].y, a.x, a.y);
                    mma_bf16(acc[j], wl[u].z, wh[u].z, wl[u].w, wh[u].w, a.z, a.w);
                }
            }
        }
    }
}

__device__ __forceinline__ float silu(float a) { return a / (1.f + expf(-a)); }

// GEMM1 + SwiGLU: Hmid[pos, 8*rb + g] = silu(<Wgate[8rb+g], x_tok>) * <Wup[8rb+g], x_tok>.
// MMA rows 0..7 = eight gate rows, rows 8..15 = the matching eight up rows, so a lane's c0/c1 and
// c2/c3 are the gate and up values of the same (row, token).
template <int NG>
__device__ __noinline__ void gemm1_item(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ wgu_e,
                                           const int32_t *__restrict__ pair_token, int pos0, int rows, int rb,
                                           int d, int He, __nv_bfloat16 *__restrict__ hmid, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const __nv_bfloat16 *row_lo = wgu_e + (size_t)(8 * rb + g) * d + 8 * t;
    const __nv_bfloat16 *row_hi = wgu_e + (size_t)(He + 8 * rb + g) * d + 8 * t;
    const __nv_bfloat16 *act[NG];
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int r = 8 * j + g;
        act[j] = (r < rows) ? x + (size_t)pair_token[pos0 + r] * d + 8 * t : nullptr;
    }
    float acc[NG][4];
#pragma unroll
    for (int j = 0; j < NG; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
    stream_dot<NG, (NG == 1 ? 4 : 2)>(row_lo, row_hi, act, d, acc);
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int r0 = 8 * j + 2 * t;
        if (r0 < rows) hmid[(size_t)(pos0 + r0) * He + 8 * rb + g] = __float2bfloat16_rn(silu(acc[j][0]) * acc[j][2]);
        if (r0 + 1 < rows) hmid[(size_t)(pos0 + r0 + 1) * He + 8 * rb + g] = __float2bfloat16_rn(silu(acc[j][1]) * acc[j][3]);
    }
}

// GEMM2: O[pos, 16*rb + {g, g+8}] = <Wdown[16rb + {g, g+8}], Hmid[pos]>.
template <int NG>
__device__ __noinline__ void gemm2_item(const __nv_bfloat16 *__restrict__ hmid, const __nv_bfloat16 *__restrict__ wd_e,
                                           int pos0, int rows, int rb, int d, int He,
                                           __nv_bfloat16 *__restrict__ obuf, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const __nv_bfloat16 *row_lo = wd_e + (size_t)(16 * rb + g) * He + 8 * t;
    const __nv_bfloat16 *row_hi = wd_e + (size_t)(16 * rb + g + 8) * He + 8 * t;
    const __nv_bfloat16 *act[NG];
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int r = 8 * j + g;
        act[j] = (r < rows) ? hmid + (size_t)(pos0 + r) * He + 8 * t : nullptr;
    }
    float acc[NG][4];
#pragma unroll
    for (int j = 0; j < NG; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f;
    stream_dot<NG, (NG == 1 ? 4 : 2)>(row_lo, row_hi, act, He, acc);
#pragma unroll
    for (int j = 0; j < NG; ++j) {
        const int r0 = 8 * j + 2 * t;
        if (r0 < rows) {
            obuf[(size_t)(pos0 + r0) * d + 16 * rb + g] = __float2bfloat16_rn(acc[j][0]);
            obuf[(size_t)(pos0 + r0) * d + 16 * rb + g + 8] = __float2bfloat16_rn(acc[j][2]);
        }
        if (r0 + 1 < rows) {
            obuf[(size_t)(pos0 + r0 + 1) * d + 16 * rb + g] = __float2bfloat16_rn(acc[j][1]);
            obuf[(size_t)(pos0 + r0 + 1) * d + 16 * rb + g + 8] = __float2bfloat16_rn(acc[j][3]);
        }
    }
}

__global__ void __launch_bounds__(256, 2)
expert_gemm1_stream_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ w_gate_up,
                           const int32_t *__restrict__ pair_token, const int32_t *__restrict__ counts,
                           const int32_t *__restrict__ offsets, const int32_t *__restrict__ chunk_expert,
                           const int32_t *__restrict__ chunk_row0, const int32_t *__restrict__ meta,
                           int d, int He, __nv_bfloat16 *__restrict__ hmid) {
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * (blockDim.x >> 5);
    const int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int row_blocks = He / 8;
    const long long n_items = (long long)meta[kMetaChunks] * row_blocks;
    for (long long item = gw; item < n_items; item += warps_total) {
        const int ci = (int)(item / row_blocks), rb = (int)(item % row_blocks);
        const int e = chunk_expert[ci], r0 = chunk_row0[ci];
        const int rows = min(kChunkRows, counts[e] - r0);
        const int pos0 = offsets[e] + r0;
        const __nv_bfloat16 *wgu_e = w_gate_up + (size_t)e * 2 * He * d;
        if (rows <= 8) gemm1_item<1>(x, wgu_e, pair_token, pos0, rows, rb, d, He, hmid, lane);
        else if (rows <= 16) gemm1_item<2>(x, wgu_e, pair_token, pos0, rows, rb, d, He, hmid, lane);
        else gemm1_item<4>(x, wgu_e, pair_token, pos0, rows, rb, d, He, hmid, lane);
    }
}

__global__ void __launch_bounds__(256, 2)
expert_gemm2_stream_kernel(const __nv_bfloat16 *__restrict__ hmid, const __nv_bfloat16 *__restrict__ w_down,
                           const int32_t *__restrict__ counts, const int32_t *__restrict__ offsets,
                           const int32_t *__restrict__ chunk_expert, const int32_t *__restrict__ chunk_row0,
                           const int32_t *__restrict__ meta, int d, int He, __nv_bfloat16 *__restrict__ obuf) {
    const int lane = threadIdx.x & 31;
    const int warps_total = gridDim.x * (blockDim.x >> 5);
    const int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int row_blocks = d / 16;
    const long long n_items = (long long)meta[kMetaChunks] * row_blocks;
    for (long long item = gw; item < n_items; item += warps_total) {
        const int ci = (int)(item / row_blocks), rb = (int)(item % row_blocks);
        const int e = chunk_expert[ci], r0 = chunk_row0[ci];
        const int rows = min(kChunkRows, counts[e] - r0);
        const int pos0 = offsets[e] + r0;
        const __nv_bfloat16 *wd_e = w_down + (size_t)e * d * He;
        if (rows <= 8) gemm2_item<1>(hmid, wd_e, pos0, rows, rb, d, He, obuf, lane);
        else if (rows <= 16) gemm2_item<2>(hmid, wd_e, pos0, rows, rb, d, He, obuf, lane);
        else gemm2_item<4>(hmid, wd_e, pos0, rows, rb, d, He, obuf, lane);
    }
}

}  // namespace

int launch_experts_gemm1(const zeda_moe *h, const __nv_bfloat16 *x, int T, cudaStream_t s) {
    (void)T;
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    expert_gemm1_stream_kernel<<<h->sm_count * 2, 256, 0, s>>>(x, h->w_gate_up, ws.pair_token, ws.counts, ws.offsets,
                                                               ws.chunk_expert, ws.chunk_row0, ws.meta, c.d_model,
                                                               c.d_expert, ws.hmid);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_experts_gemm2(const zeda_moe *h, int T, cudaStream_t s) {
    (void)T;
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    expert_gemm2_stream_kernel<<<h->sm_count * 2, 256, 0, s>>>(ws.hmid, h->w_down, ws.counts, ws.offsets,
                                                               ws.chunk_expert, ws.chunk_row0, ws.meta, c.d_model,
                                                               c.d_expert, ws.obuf);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
