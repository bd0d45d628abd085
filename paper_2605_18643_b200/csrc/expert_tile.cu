// Grouped expert GEMMs on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM),
// operands staged in shared memory by TMA.
//
// Appendix D: each normal expert has gate, up and down projections; per surviving (token, expert)
// pair that is 6*H*H_e FLOPs.  Both GEMMs are run "weights as the M operand": the MMA's 128 rows
// are weight rows, its N columns are the (<= 128) pair rows of one expert, so a ragged expert of n
// pairs costs ceil(n/16)*16 columns instead of a padded 128-row tile, and small decode batches
// stream each active expert's weights exactly once.
//
//   work item   = (expert e, block of <= 128 of its pair rows, block of 256 weight rows)
//   A operands  = two [128 x 64] K-major weight tiles per k-step (GEMM1: 128 gate rows and the
//                 matching 128 up rows; GEMM2: two consecutive blocks of 128 down rows)
//   B operand   = [n x 64] K-major activation rows (x rows gathered into pair order, or Hmid)
//   D           = two fp32 accumulators [128 lanes x n columns] in TMEM, double-buffered
//
// One CTA per SM, persistent over a device-side work list (no host knowledge of P, counts).
// Warp 0: TMA producer.  Warp 1: TMEM allocation + MMA issue.  Warps 2-5: epilogue (TMEM ->
// registers -> SwiGLU / store).  Every mbarrier wait is bounded; on expiry the CTA records an
// error word, lets its copies land, frees its TMEM and returns.
#include "tc_common.cuh"

namespace zeda {

namespace {

using namespace tc;

constexpr int kBlockK = 64;                  // bf16 elements per k-step = one 128-byte swizzle row
constexpr int kATileBytes = 128 * kBlockK * 2;  // 16 KB
constexpr int kBBoxRows = 16;
constexpr int kBBoxBytes = kBBoxRows * kBlockK * 2;  // 2 KB
constexpr int kAccCols = 128;                // TMEM columns per accumulator
constexpr int kTmemCols = 512;               // 2 buffers x 2 accumulators x 128 columns
constexpr int kThreads = 192;

struct TileMaps {
    CUtensorMap w_gate_up;  // [N][2He][d]  box {64, 128, 1}
    CUtensorMap w_down;     // [N][d][He]   box {64, 128, 1}
    CUtensorMap x_sorted;   // [rows][d]    box {64, 16}
    CUtensorMap hmid;       // [rows][He]   box {64, 16}
};

__device__ __forceinline__ float silu(float a) { return a / (1.f + expf(-a)); }

struct ItemInfo {
    int e, pos0, n, mb;
};

__device__ __forceinline__ ItemInfo load_item(long long item, int m_blocks, const int32_t *tile_expert,
                                              const int32_t *tile_row0, const int32_t *counts, const int32_t *offsets) {
    ItemInfo it;
    const int tile = (int)(item / m_blocks);
    it.mb = (int)(item % m_blocks);
    it.e = tile_expert[tile];
    const int r0 = tile_row0[tile];
    it.n = min(kTileM, counts[it.e] - r0);
    it.pos0 = offsets[it.e] + r0;
    return it;
}

// MODE 1: GEMM1 + SwiGLU.  A0 = gate rows [128mb, +128), A1 = up rows [He + 128mb, +128) of expert e,
//         B = x_sorted rows, K = d.  out = Hmid[pos, 128mb + lane_row] (bf16).
// MODE 2: GEMM2.            A0/A1 = down rows [256mb, +128) / [256mb + 128, +128), B = Hmid rows, K = He.
//         out = O[pos, row] (bf16).
template <int MODE, int TN_MAX, int STAGES>
__global__ void __launch_bounds__(kThreads, 1)
expert_gemm_tile_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                        const int32_t *__restrict__ counts, const int32_t *__restrict__ offsets,
                        const int32_t *__restrict__ tile_expert, const int32_t *__restrict__ tile_row0,
                        int32_t *__restrict__ meta, int kdim, int out_rows, int a1_row_offset, int m_blocks,
                        __nv_bfloat16 *__restrict__ out, int out_ld) {
    constexpr int kStageBytes = 2 * kATileBytes + TN_MAX * kBlockK * 2;
    extern __shared__ __align__(1024) unsigned char tile_smem[];
    __shared__ __align__(8) unsigned long long bars[2 * STAGES + 4];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    // 1024-byte alignment of the operand ring (the swizzle pattern is a function of the address)
    const uint32_t ring = (smem_u32(tile_smem) + 1023u) & ~1023u;
    const uint32_t bar_full = smem_u32(&bars[0]);
    const uint32_t bar_empty = smem_u32(&bars[STAGES]);
    const uint32_t bar_tfull = smem_u32(&bars[2 * STAGES]);
    const uint32_t bar_tempty = smem_u32(&bars[2 * STAGES + 2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int i = 0; i < STAGES; ++i) { mbar_init(bar_full + 8 * i, 1); mbar_init(bar_empty + 8 * i, 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;

    const long long n_items = (long long)meta[kMetaTiles] * m_blocks;
    const int k_steps = kdim / kBlockK;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t it_count = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
                const ItemInfo it = load_item(item, m_blocks, tile_expert, tile_row0, counts, offsets);
                const int nb = (it.n + kBBoxRows - 1) / kBBoxRows;
                const int row_a0 = (MODE == 1 ? 128 : 256) * it.mb;
                const int row_a1 = row_a0 + a1_row_offset;
                const uint32_t bytes = 2 * kATileBytes + nb * kBBoxBytes;
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                    if (!mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag)) { ok = false; break; }
                    const uint32_t full = bar_full + 8 * s;
                    const uint32_t sa = ring + s * kStageBytes;
                    mbar_expect_tx(full, bytes);
                    tma_load_3d(sa, &map_a, ks * kBlockK, row_a0, it.e, full);
                    tma_load_3d(sa + kATileBytes, &map_a, ks * kBlockK, row_a1, it.e, full);
                    for (int b = 0; b < nb; ++b)
                        tma_load_2d(sa + 2 * kATileBytes + b * kBBoxBytes, &map_b, ks * kBlockK, it.pos0 + b * kBBoxRows, full);
                }
            }
            if (!ok) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 1);
                s_abort = 1;
            }
            // let the copies that were issued land before the CTA leaves (bounded)
            const uint32_t issued = it_count;
            for (uint32_t j = (issued > (uint32_t)STAGES ? issued - STAGES : 0); j < issued; ++j)
                mbar_wait(bar_full + 8 * (j % STAGES), (j / STAGES) & 1u, abort_flag);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            uint32_t it_count = 0, tile_count = 0;
            bool ok = true;
            for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile_count) {
                const ItemInfo it = load_item(item, m_blocks, tile_expert, tile_row0, counts, offsets);
                const int n_mma = ((it.n + 15) / 16) * 16;
                const uint32_t idesc = instr_desc(n_mma);
                const uint32_t buf = tile_count & 1u, tph = (tile_count >> 1) & 1u;
                if (!mbar_wait(bar_tempty + 8 * buf, tph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + buf * (2 * kAccCols);
                const uint32_t d1 = d0 + kAccCols;
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                    if (!mbar_wait(bar_full + 8 * s, ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = ring + s * kStageBytes;
                    const uint64_t a0 = smem_desc_sw128(sa);
                    const uint64_t a1 = smem_desc_sw128(sa + kATileBytes);
                    const uint64_t b = smem_desc_sw128(sa + 2 * kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) {
                        // +32 bytes per 16-element k slice inside the 128-byte swizzle row
                        const uint32_t acc = (ks | k) ? 1u : 0u;
                        umma_bf16(d0, a0 + 2 * k, b + 2 * k, idesc, acc);
                        umma_bf16(d1, a1 + 2 * k, b + 2 * k, idesc, acc);
                    }
                    umma_commit(bar_empty + 8 * s);   // stage free once these MMAs have read it
                }
                if (!ok) break;
                umma_commit(bar_tfull + 8 * buf);     // accumulators complete
            }
            if (!ok) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 2);
                s_abort = 1;
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;  // TMEM lane quarter this warp may read
        uint32_t tile_count = 0;
        bool ok = true;
        for (long long item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++tile_count) {
            const ItemInfo it = load_item(item, m_blocks, tile_expert, tile_row0, counts, offsets);
            const uint32_t buf = tile_count & 1u, tph = (tile_count >> 1) & 1u;
            if (!mbar_wait(bar_tfull + 8 * buf, tph, abort_flag)) ok = false;
            ok = __all_sync(0xffffffffu, ok);   // also reconverges the warp before the aligned TMEM loads
            if (!ok) break;
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16) + buf * (2 * kAccCols);
            const int row = 32 * q + lane;
            for (int c0 = 0; c0 < it.n; c0 += 32) {
                float v0[32], v1[32];
                tmem_ld32(t0 + c0, v0);
                tmem_ld32(t0 + kAccCols + c0, v1);
                if (c0 + 32 >= it.n) {
                    // last read of this buffer: hand it back to the MMA warp before the stores
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
                }
                if (MODE == 1) {
                    const int f = 128 * it.mb + row;
                    if (f < out_rows) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (c0 + j < it.n)
                                out[(size_t)(it.pos0 + c0 + j) * out_ld + f] = __float2bfloat16_rn(silu(v0[j]) * v1[j]);
                    }
                } else {
                    const int r0 = 256 * it.mb + row, r1 = r0 + 128;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (c0 + j < it.n) {
                            __nv_bfloat16 *o = out + (size_t)(it.pos0 + c0 + j) * out_ld;
                            if (r0 < out_rows) o[r0] = __float2bfloat16_rn(v0[j]);
                            if (r1 < out_rows) o[r1] = __float2bfloat16_rn(v1[j]);
                        }
                    }
                }
            }
        }
        if (!ok && lane == 0) {
            if (!*abort_flag) atomicExch(&meta[kMetaError], 3);
            s_abort = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// x rows gathered into pair order: xs[p] = x[pair_token[p]] for p < P (16-byte vectors).
__global__ void __launch_bounds__(256)
gather_rows_kernel(const __nv_bfloat16 *__restrict__ x, const int32_t *__restrict__ pair_token,
                   const int32_t *__restrict__ meta, int d, __nv_bfloat16 *__restrict__ xs) {
    const int P = meta[kMetaPairs];
    const int vec = d / 8;
    for (int p = blockIdx.x; p < P; p += gridDim.x) {
        const uint4 *src = reinterpret_cast<const uint4 *>(x + (size_t)pair_token[p] * d);
        uint4 *dst = reinterpret_cast<uint4 *>(xs + (size_t)p * d);
        for (int c = threadIdx.x; c < vec; c += blockDim.x) dst[c] = __ldg(src + c);
    }
}

template <int MODE, int TN_MAX, int STAGES>
constexpr int tile_smem_bytes() { return STAGES * (2 * kATileBytes + TN_MAX * kBlockK * 2) + 1024; }

template <int MODE, int TN_MAX, int STAGES>
bool set_smem_attr() {
    return cudaFuncSetAttribute(expert_gemm_tile_kernel<MODE, TN_MAX, STAGES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                tile_smem_bytes<MODE, TN_MAX, STAGES>()) == cudaSuccess;
}

constexpr int kSmallTN = 64, kSmallStages = 5, kBigTN = 128, kBigStages = 4;

}  // namespace

int init_tile_kernels(zeda_moe *h) {
    const zeda_moe_config_t &c = h->cfg;
    TileMaps *tm = static_cast<TileMaps *>(aligned_alloc(64, sizeof(TileMaps)));
    if (!tm) { set_error("out of host memory"); return -1; }
    const cuuint64_t E = c.n_real, d = c.d_model, He = c.d_expert;
    const cuuint64_t rows = (cuuint64_t)c.max_tokens * c.top_k + kTileM;
    bool ok = true;
    {
        const cuuint64_t dims[3] = {d, 2 * He, E};
        const cuuint64_t strides[2] = {d * 2, 2 * He * d * 2};
        const cuuint32_t box[3] = {kBlockK, 128, 1};
        ok = ok && encode_bf16_map(&tm->w_gate_up, h->w_gate_up, 3, dims, strides, box);
    }
    {
        const cuuint64_t dims[3] = {He, d, E};
        const cuuint64_t strides[2] = {He * 2, d * He * 2};
        const cuuint32_t box[3] = {kBlockK, 128, 1};
        ok = ok && encode_bf16_map(&tm->w_down, h->w_down, 3, dims, strides, box);
    }
    {
        const cuuint64_t dims[2] = {d, rows};
        const cuuint64_t strides[1] = {d * 2};
        const cuuint32_t box[2] = {kBlockK, kBBoxRows};
        ok = ok && encode_bf16_map(&tm->x_sorted, h->ws.x_sorted, 2, dims, strides, box);
    }
    {
        const cuuint64_t dims[2] = {He, rows};
        const cuuint64_t strides[1] = {He * 2};
        const cuuint32_t box[2] = {kBlockK, kBBoxRows};
        ok = ok && encode_bf16_map(&tm->hmid, h->ws.hmid, 2, dims, strides, box);
    }
    ok = ok && set_smem_attr<1, kSmallTN, kSmallStages>() && set_smem_attr<2, kSmallTN, kSmallStages>() &&
         set_smem_attr<1, kBigTN, kBigStages>() && set_smem_attr<2, kBigTN, kBigStages>();
    if (!ok) {
        free(tm);
        if (zeda_last_error()[0] == 0) set_error("tile kernel set-up failed: %s", cudaGetErrorString(cudaGetLastError()));
        return -1;
    }
    h->tmaps = tm;
    return 0;
}

int launch_gather_rows(const zeda_moe *h, const __nv_bfloat16 *x, int T, cudaStream_t s) {
    const int grid = min(T * h->cfg.top_k, h->sm_count * 8);
    gather_rows_kernel<<<grid, 256, 0, s>>>(x, h->ws.pair_token, h->ws.meta, h->cfg.d_model, h->ws.x_sorted);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_experts_gemm1_tile(const zeda_moe *h, int T, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    const TileMaps *tm = static_cast<const TileMaps *>(h->tmaps);
    const int m_blocks = (c.d_expert + 127) / 128;
    if (T <= kSmallTN)
        expert_gemm_tile_kernel<1, kSmallTN, kSmallStages><<<h->sm_count, kThreads, tile_smem_bytes<1, kSmallTN, kSmallStages>(), s>>>(
            tm->w_gate_up, tm->x_sorted, ws.counts, ws.offsets, ws.tile_expert, ws.tile_row0, ws.meta, c.d_model,
            c.d_expert, c.d_expert, m_blocks, ws.hmid, c.d_expert);
    else
        expert_gemm_tile_kernel<1, kBigTN, kBigStages><<<h->sm_count, kThreads, tile_smem_bytes<1, kBigTN, kBigStages>(), s>>>(
            tm->w_gate_up, tm->x_sorted, ws.counts, ws.offsets, ws.tile_expert, ws.tile_row0, ws.meta, c.d_model,
            c.d_expert, c.d_expert, m_blocks, ws.hmid, c.d_expert);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_experts_gemm2_tile(const zeda_moe *h, int T, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    const TileMaps *tm = static_cast<const TileMaps *>(h->tmaps);
    const int m_blocks = (c.d_model + 255) / 256;
    if (T <= kSmallTN)
        expert_gemm_tile_kernel<2, kSmallTN, kSmallStages><<<h->sm_count, kThreads, tile_smem_bytes<2, kSmallTN, kSmallStages>(), s>>>(
            tm->w_down, tm->hmid, ws.counts, ws.offsets, ws.tile_expert, ws.tile_row0, ws.meta, c.d_expert, c.d_model,
            128, m_blocks, ws.obuf, c.d_model);
    else
        expert_gemm_tile_kernel<2, kBigTN, kBigStages><<<h->sm_count, kThreads, tile_smem_bytes<2, kBigTN, kBigStages>(), s>>>(
            tm->w_down, tm->hmid, ws.counts, ws.offsets, ws.tile_expert, ws.tile_row0, ws.meta, c.d_expert, c.d_model,
            128, m_blocks, ws.obuf, c.d_model);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
