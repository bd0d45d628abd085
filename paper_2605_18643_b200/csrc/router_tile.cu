// Router logits on the tensor cores for large batches (prefill shapes).
//
// Section 2.1: the router scores N + N_Z candidates per token, 2 (N + N_Z) n H FLOPs (Appendix D).
// The fp32 router weights cannot go through a bf16 MMA as they are, and a TF32 product would put
// logit errors too close to the top-K tie margin.  Instead every fp32 weight is split once, at
// handle creation, into three bf16 pieces w = hi + mid + lo (8 + 8 + 8 mantissa bits, exact), so
// that with bf16 activations every product is exact in the fp32 accumulator.  The GEMM runs with
// the candidates as the 128-row M operand and 128 tokens as N; the three pieces accumulate into
// three TMEM accumulators and the epilogue adds them (small to large) and the bias.
#include "tc_common.cuh"

namespace zeda {

namespace {

using namespace tc;

constexpr int kBlockK = 64;
constexpr int kTileBytes = 128 * kBlockK * 2;  // 16 KB: [128 rows x 64] bf16
constexpr int kStages = 3;
constexpr int kStageBytes = 4 * kTileBytes;    // hi, mid, lo, x
constexpr int kThreads = 192;
constexpr int kTokTile = 128;

struct RouterMaps {
    CUtensorMap w_split;  // [3][NC_pad][d] bf16, box {64, 128, 1}
};

// hi/mid/lo split of the fp32 router rows; rows >= n_cand are zero.
__global__ void __launch_bounds__(256)
split_router_kernel(const float *__restrict__ w, int n_cand, int nc_pad, int d, __nv_bfloat16 *__restrict__ out) {
    const size_t total = (size_t)nc_pad * d;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int row = (int)(i / d);
        float v = row < n_cand ? w[i] : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(v);
        v -= __bfloat162float(hi);
        const __nv_bfloat16 mid = __float2bfloat16_rn(v);
        v -= __bfloat162float(mid);
        const __nv_bfloat16 lo = __float2bfloat16_rn(v);
        out[i] = hi;
        out[total + i] = mid;
        out[2 * total + i] = lo;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
router_logits_tile_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                          const float *__restrict__ bias, int T, int n_cand, int m_tiles, int k_steps, int split,
                          int32_t *__restrict__ meta, float *__restrict__ logits) {
    pdl_launch_dependents();
    extern __shared__ __align__(1024) unsigned char router_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * kStages + 2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    const uint32_t ring = (smem_u32(router_smem) + 1023u) & ~1023u;
    const uint32_t bar_full = smem_u32(&bars[0]);
    const uint32_t bar_empty = smem_u32(&bars[kStages]);
    const uint32_t bar_tfull = smem_u32(&bars[2 * kStages]);
    const uint32_t bar_tempty = smem_u32(&bars[2 * kStages + 1]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int i = 0; i < kStages; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
        mbar_init(bar_tfull, 1);
        mbar_init(bar_tempty, 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), 512);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;
    pdl_wait();
    // Work item = (token tile, candidate tile, slice of the reduction axis).  With few token tiles the
    // reduction axis is cut into `split` slices so that the grid still covers the SMs; slice p writes
    // its partial sums to logits + p * T * n_cand and the top-K kernel adds the slices in order.
    const int tok_tiles = (T + kTokTile - 1) / kTokTile;
    const int n_items = tok_tiles * m_tiles * split;
    k_steps /= split;  // per item

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it_count = 0;
            bool ok = true;
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const int sp = item % split, mt = (item / split) % m_tiles, tt = item / (split * m_tiles);
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    const uint32_t s = it_count % kStages, ph = (it_count / kStages) & 1u;
                    if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = bar_full + 8 * s, sa = ring + s * kStageBytes;
                    const int kc = (sp * k_steps + ks) * kBlockK;
                    mbar_expect_tx(full, kStageBytes);
                    for (int piece = 0; piece < 3; ++piece)
                        tma_load_3d(sa + piece * kTileBytes, &map_w, kc, mt * 128, piece, full);
                    tma_load_2d(sa + 3 * kTileBytes, &map_x, kc, tt * kTokTile, full);
                }
            }
            if (!ok) { if (!*abort_flag) atomicExch(&meta[kMetaError], 4); s_abort = 1; }
            for (uint32_t j = (it_count > (uint32_t)kStages ? it_count - kStages : 0); j < it_count; ++j)
                mbar_wait(bar_full + 8 * (j % kStages), (j / kStages) & 1u, abort_flag);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            uint32_t it_count = 0, tile_count = 0;
            bool ok = true;
            const uint32_t idesc = instr_desc(kTokTile);
            for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile_count) {
                if (!mbar_wait(bar_tempty, (tile_count & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    const uint32_t s = it_count % kStages, ph = (it_count / kStages) & 1u;
                    if (!mbar_wait(bar_full + 8 * s, ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = ring + s * kStageBytes;
                    const uint64_t b = smem_desc_sw128(sa + 3 * kTileBytes);
#pragma unroll
                    for (int piece = 0; piece < 3; ++piece) {
                        const uint64_t a = smem_desc_sw128(sa + piece * kTileBytes);
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)
                            umma_bf16(tmem_base + piece * kTokTile, a + 2 * k, b + 2 * k, idesc, (ks | k) ? 1u : 0u);
                    }
                    umma_commit(bar_empty + 8 * s);
                }
                if (!ok) break;
                umma_commit(bar_tfull);
            }
            if (!ok) { if (!*abort_flag) atomicExch(&meta[kMetaError], 5); s_abort = 1; }
        }
    } else {
        const int q = warp & 3;
        uint32_t tile_count = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile_count) {
            const int sp = item % split, mt = (item / split) % m_tiles, tt = item / (split * m_tiles);
            if (!mbar_wait(bar_tfull, tile_count & 1u, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int j = mt * 128 + 32 * q + lane;  // candidate of this lane
            const float b = (bias && j < n_cand && sp == 0) ? __ldg(bias + j) : 0.f;  // slice 0 carries the bias
            float *out = logits + (size_t)sp * T * n_cand;
            const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16);
            const int tok0 = tt * kTokTile;
            for (int c0 = 0; c0 < kTokTile; c0 += 32) {
                float hi[32], mid[32], lo[32];
                tmem_ld32(t0 + c0, hi);
                tmem_ld32(t0 + kTokTile + c0, mid);
                tmem_ld32(t0 + 2 * kTokTile + c0, lo);
                if (c0 + 32 >= kTokTile) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty);
                }
                if (j < n_cand) {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (tok0 + c0 + c < T)
                            out[(size_t)(tok0 + c0 + c) * n_cand + j] = ((lo[c] + mid[c]) + hi[c]) + b;
                }
            }
        }
        if (!ok && lane == 0) { if (!*abort_flag) atomicExch(&meta[kMetaError], 6); s_abort = 1; }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

constexpr int kSmemBytes = kStages * kStageBytes + 1024;

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing will ever arrive on,
// with a short limit, and records the expiry in the handle's error word exactly as the kernels do.
__global__ void wait_selftest_kernel(int32_t *__restrict__ meta, long long limit_cycles) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_for(smem_u32(&bar), 0, &s_abort, limit_cycles)) atomicExch(&meta[kMetaError], 99);
    }
}

}  // namespace

int launch_wait_selftest(const zeda_moe *h, long long limit_cycles, cudaStream_t s) {
    wait_selftest_kernel<<<1, 32, 0, s>>>(h->ws.meta, limit_cycles);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int router_split_pad(int n_cand) { return (n_cand + 127) / 128 * 128; }

int init_router_tile(zeda_moe *h) {
    const zeda_moe_config_t &c = h->cfg;
    const int n_cand = c.n_real + c.n_zero, nc_pad = router_split_pad(n_cand);
    RouterMaps *rm = static_cast<RouterMaps *>(aligned_alloc(64, sizeof(RouterMaps)));
    if (!rm) { set_error("out of host memory"); return -1; }
    const cuuint64_t dims[3] = {(cuuint64_t)c.d_model, (cuuint64_t)nc_pad, 3};
    const cuuint64_t strides[2] = {(cuuint64_t)c.d_model * 2, (cuuint64_t)nc_pad * c.d_model * 2};
    const cuuint32_t box[3] = {kBlockK, 128, 1};
    bool ok = encode_bf16_map(&rm->w_split, h->ws.router_split, 3, dims, strides, box);
    ok = ok && cudaFuncSetAttribute(router_logits_tile_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess;
    if (!ok) { free(rm); return -1; }
    split_router_kernel<<<h->sm_count * 2, 256>>>(h->router_w, n_cand, nc_pad, c.d_model, h->ws.router_split);
    if (cudaGetLastError() != cudaSuccess) { free(rm); return -1; }
    h->router_maps = rm;
    return 0;
}

int router_split_factor(const zeda_moe *h, int T) {
    const int nc_pad = router_split_pad(h->cfg.n_real + h->cfg.n_zero);
    const int items = (T + kTokTile - 1) / kTokTile * (nc_pad / 128);
    const int k_steps = h->cfg.d_model / kBlockK;
    int split = 1;
    while (split < kRouterMaxSplit && items * split * 2 <= h->sm_count && k_steps % (split * 2) == 0 &&
           (long long)T * split * 2 <= router_part_rows(h->cfg.max_tokens))
        split *= 2;
    return split;
}

int launch_router_logits_tile(const zeda_moe *h, const __nv_bfloat16 *x, int T, float *logits, int split, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const int n_cand = c.n_real + c.n_zero, nc_pad = router_split_pad(n_cand);
    // the activations are the caller's buffer of this call: their tensor map is made per call (host only)
    CUtensorMap map_x;
    const cuuint64_t dims[2] = {(cuuint64_t)c.d_model, (cuuint64_t)T};
    const cuuint64_t strides[1] = {(cuuint64_t)c.d_model * 2};
    const cuuint32_t box[2] = {kBlockK, kTokTile};
    if (!encode_bf16_map(&map_x, x, 2, dims, strides, box)) return -1;
    const RouterMaps *rm = static_cast<const RouterMaps *>(h->router_maps);
    const int m_tiles = nc_pad / 128;
    const int n_items = (T + kTokTile - 1) / kTokTile * m_tiles * split;
    const int grid = n_items < h->sm_count ? n_items : h->sm_count;
    const cudaError_t e = launch_kernel(h->pdl, router_logits_tile_kernel, dim3(grid), dim3(kThreads), kSmemBytes, s,
                                        rm->w_split, map_x, h->router_bias, T, n_cand, m_tiles, c.d_model / kBlockK,
                                        split, h->ws.meta, logits);
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
