// Grouped expert GEMMs on CTA pairs: tcgen05.mma.cta_group::2 (M = 256 over two SMs), accumulators
// in TMEM, weights and Hmid staged in shared memory by TMA, the x rows of GEMM1 gathered straight
// from the token-order x by cp.async (no gathered copy of x is ever written).
//
// Appendix D: each normal expert has gate, up and down projections; a surviving (token, expert)
// pair costs 6*H*H_e FLOPs, a zero-expert slot none (it never reaches these kernels).  Both GEMMs
// run "weights as the M operand": the 256 rows of the MMA are weight rows (128 in each CTA of the
// pair), its N <= 256 columns are pair rows of ONE expert (N/2 loaded by each CTA), so a ragged
// expert costs its pair count rounded up to 32 columns, and each CTA loads 128 weight rows plus at
// most 128 activation rows per 128 x 256 block of outputs.
//
//   work item  = (expert e, block of <= 256 of its pair rows, block mb of weight rows)
//   GEMM1      A tile of CTA r = the 64 features of 64-row block (2 mb + r) as four groups of 16 gate
//              rows each followed by the matching 16 up rows (one 5-D TMA box); B = x rows of the
//              pairs, fetched by four gather warps through pair_token with 16-byte cp.async into
//              the 128-byte-swizzled layout; K = H.  An epilogue warp's 32 TMEM lanes thus hold the
//              gate values (lanes 0-15) and the up values (lanes 16-31) of the same 16 features:
//              the halves meet through one warp shuffle per column pair, SwiGLU, store of Hmid.
//   GEMM2      A tile of CTA r = 128 down rows [256 mb + 128 r, +128); B = Hmid rows; K = H_e.
//
// One CTA per SM, persistent over a device-side work list (the host never learns P or the counts).
// Warp 0: TMA producer (weights).  Warp 1: TMEM allocation, and in the leader CTA the MMA issue.
// Warp 2 (GEMM1): gather relay.  Warp 3 (GEMM2): TMA producer of the Hmid rows.  Warps 4-7:
// epilogue.  Warps 8-11 (GEMM1): x-row gather.  One more warp per TMA stream (GEMM1: warp 12; GEMM2:
// warps 8 and 9) takes every second k-step.  Full barriers live in the leader CTA and count the
// TMA bytes (and gather relays) of both CTAs; stage-empty and accumulator-full barriers are
// signalled in both CTAs by multicast commits.  The issuing warps (TMA producers, MMA issue, relay)
// run their loops with all 32 lanes converged: every lane waits on the barrier, one elected lane
// issues.  A loop confined to a single lane of a diverged warp costs about twice the cycles per
// k-step, and that lane's instruction stream is what bounds a narrow tile.  Every mbarrier wait is
// bounded; on expiry the CTA records an error word, skips the rest of its work, and leaves through
// the common exit (cluster barrier, TMEM free).
#include <utility>

#include "tc_common.cuh"

namespace zeda {

namespace {

using namespace tc;

constexpr int kBlockK = 64;                     // bf16 elements per k-step = one 128-byte swizzle row
constexpr int kATileBytes = 128 * kBlockK * 2;  // 16 KB: this CTA's 128 weight rows of one k-step
constexpr int kRowBytes = kBlockK * 2;          // 128
constexpr int kAccCols = 256;                   // TMEM columns of one accumulator buffer
constexpr int kThreads = 320;                   // GEMM2: warps 8, 9 are the second issuers of the two TMA streams
constexpr int kThreadsGather = 416;             // GEMM1: four gather warps, warp 12 the second weight issuer
constexpr int kProducers = 2;                   // warps that share a TMA stream, k-step c going to warp c mod 2
constexpr int kPatchBytes = 4 * 32 * 32 * 2;    // per epilogue warp: [32 pair rows][32 features] bf16, for 16-byte stores

// Hmid row blocks come in boxes of 128, 64, 32 and 16 rows: a block of 16 k rows is loaded with
// at most four TMA instructions (few large boxes: issuing a TMA instruction costs a few hundred cycles).
struct RowMaps {
    CUtensorMap m[4];  // box {64, 128 >> i}
};

struct PairMaps {
    CUtensorMap w_gate_up;  // [N][He/16 groups][gate | up][16 rows][d]  box {64, 16, 2, 4, 1}
    CUtensorMap w_down;     // [N][d][He]   box {64, 128, 1}
    RowMaps hmid;           // [rows][He]
};

struct Item {
    int e, pos0, n, mb;
};

// one k-step of an item in the ring: the weight tile(s), then this CTA's pair rows
template <int HALF_MAX, int DBL_ROWS>
struct StageBytes {
    static constexpr int kSingle = kATileBytes + HALF_MAX * kRowBytes;
    static constexpr int kDouble = DBL_ROWS > 0 ? 2 * kATileBytes + (DBL_ROWS / 2) * kRowBytes : 0;
    static constexpr int value = kSingle > kDouble ? kSingle : kDouble;
};

__device__ __forceinline__ Item load_item(long long item, int m_blocks, int tile_rows, const int32_t *tile_expert,
                                          const int32_t *tile_row0, const int32_t *counts, const int32_t *offsets) {
    Item it;
    const int tile = (int)(item / m_blocks);
    it.mb = (int)(item % m_blocks);
    it.e = tile_expert[tile];
    const int r0 = tile_row0[tile];
    it.n = min(tile_rows, counts[it.e] - r0);
    it.pos0 = offsets[it.e] + r0;
    return it;
}

// ---- work items handed out at run time --------------------------------------------------------
// The clusters do not own fixed shares of the item list: each takes the next unclaimed item from
// a device counter whenever its weight producer starts on the item before (an atomic add by one
// scheduler warp of the leader CTA), so that a cluster that drew cheap items simply draws more of
// them.  The scheduler packs the item's description into one 64-bit word and stores it into slot
// (sequence number mod kItemSlots) of a small queue in BOTH CTAs' shared memory; every role reads
// the sequence of items from its own CTA's queue, polling the slot until its tag matches.
//   bits 63..51 tag = sequence number mod 8191, plus 1 (never 0: an unwritten slot matches nothing)
//   bit  50     end of the list          49..41 expert       40..35 weight-row block
//   34..27      pair rows in the tile - 1                    26..0  first pair position
// A slot is overwritten kItemSlots items later.  The scheduler runs at most one item ahead of the
// weight producer, the producer at most STAGES k-steps (at most that many items) ahead of the MMA
// warp, the MMA warp at most two tiles ahead of the slowest epilogue warp of either CTA (it needs
// every epilogue warp's arrival to reuse an accumulator): with STAGES <= 10 no reader is more than
// 15 items behind the scheduler, and kItemSlots = 32.
constexpr int kItemSlots = 32;
constexpr int kSchedAhead = 1;  // items the scheduler may run ahead of the weight producer

__device__ __forceinline__ unsigned long long pack_item(uint32_t seq, bool end, const Item &it) {
    return ((unsigned long long)(seq % 8191u + 1u) << 51) | ((unsigned long long)(end ? 1 : 0) << 50) |
           ((unsigned long long)(uint32_t)it.e << 41) | ((unsigned long long)(uint32_t)it.mb << 35) |
           ((unsigned long long)(uint32_t)(it.n - 1) << 27) | (unsigned long long)(uint32_t)it.pos0;
}

// The item with sequence number seq from this CTA's queue; called by all 32 lanes of a converged warp
// (lane 0 polls, the word is broadcast).  Returns 1 with the item, 0 at the end of the list, -1 if the
// entry did not arrive within the wait limit or another role of this CTA gave up.
__device__ __forceinline__ int next_item(const volatile unsigned long long *queue, uint32_t seq, Item &it,
                                         volatile int *abort_flag) {
    const unsigned long long want = seq % 8191u + 1u;
    unsigned long long v = 0ull;
    int status = 1;
    if ((threadIdx.x & 31) == 0) {
        v = queue[seq % kItemSlots];
        if ((v >> 51) != want) {
            const long long t0 = clock64();
            int spins = 0;
            while (((v = queue[seq % kItemSlots]) >> 51) != want) {
                if ((++spins & 63) == 0 && (*abort_flag || clock64() - t0 > kWaitLimitCycles)) { status = -1; break; }
            }
        }
    }
    status = __shfl_sync(0xffffffffu, status, 0);
    if (status < 0) return -1;
    v = __shfl_sync(0xffffffffu, v, 0);
    if ((v >> 50) & 1ull) return 0;
    it.e = (int)((v >> 41) & 0x1ffu);
    it.mb = (int)((v >> 35) & 0x3fu);
    it.n = (int)((v >> 27) & 0xffu) + 1;
    it.pos0 = (int)(v & 0x7ffffffu);
    return 1;
}

__device__ __forceinline__ float swiglu(float g, float u) { return __fdividef(g * u, 1.f + __expf(-g)); }

// A tile of at most DBL_ROWS pair rows takes two blocks of weight rows per item ("double item"): a
// k-step of such a tile costs the pipeline the same time whether it carries one block or two (the
// tensor pipe is idle most of it: an MMA of N <= 128 columns takes about 70 cycles however narrow it
// is, and the rest is the barrier round trips of the stage), so a double item moves an expert's weights
// through the SM pair twice as fast.  Its two accumulators share one TMEM buffer (columns 0.. and
// 128..), its stage holds both weight tiles and the pair rows: 16 + 16 + DBL_ROWS / 2 * 128 bytes.
__device__ __forceinline__ bool double_item(int dbl_rows, int n, int mb, int m_blocks) {
    return n <= dbl_rows && !(mb & 1) && mb + 1 < m_blocks;
}

// MODE 1: GEMM1 + SwiGLU -> Hmid[pos, f].   MODE 2: GEMM2 -> O[pos, row].
// HALF_MAX: most B rows one CTA loads per k-step (the tile's column count is at most 2 * HALF_MAX).
// DBL_ROWS: tiles of at most this many pair rows run as double items (0: none; at most 128).
// One CTA per SM with two accumulator buffers in TMEM: the epilogue of a tile runs under the MMAs of
// the CTA's next tile.
template <int MODE, int HALF_MAX, int STAGES, int DBL_ROWS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MODE == 1 ? kThreadsGather : kThreads, 1)
expert_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ RowMaps maps_b,
                        const __nv_bfloat16 *__restrict__ x, int x_ld, const int32_t *__restrict__ counts,
                        const int32_t *__restrict__ offsets, const int32_t *__restrict__ tile_expert,
                        const int32_t *__restrict__ tile_row0, const int32_t *__restrict__ pair_token,
                        int32_t *__restrict__ meta, int kdim, int out_rows, int m_blocks,
                        __nv_bfloat16 *__restrict__ out, int out_ld, int tile_rows) {
    static_assert(STAGES <= 10, "the item queue's depth assumes at most 10 ring stages");
    static_assert(DBL_ROWS <= 128 && DBL_ROWS % 32 == 0 && DBL_ROWS <= 2 * HALF_MAX, "two accumulators of a double item share 256 columns");
    constexpr int kStageBytes = StageBytes<HALF_MAX, DBL_ROWS>::value;
    constexpr int kTmemCols = 2 * kAccCols;
    if (MODE == 2) pdl_launch_dependents();
    extern __shared__ __align__(1024) unsigned char pair_smem[];
    __shared__ __align__(8) unsigned long long bars[3 * STAGES + 4];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;
    __shared__ __align__(8) unsigned long long s_items[kItemSlots];  // this CTA's copy of the item queue
    __shared__ int s_prod_seq;                                       // item the weight producer is on (leader CTA)

    // 1024-byte alignment of the operand ring (the swizzle pattern is a function of the address)
    const uint32_t ring = (smem_u32(pair_smem) + 1023u) & ~1023u;
    unsigned char *after_ring = pair_smem + (ring - smem_u32(pair_smem)) + STAGES * kStageBytes;
    __nv_bfloat16 *patches = reinterpret_cast<__nv_bfloat16 *>(after_ring);
    const uint32_t bar_full = smem_u32(&bars[0]);                 // used in the leader CTA only
    const uint32_t bar_empty = smem_u32(&bars[STAGES]);           // one set per CTA
    const uint32_t bar_tfull = smem_u32(&bars[2 * STAGES]);       // one set per CTA
    const uint32_t bar_tempty = smem_u32(&bars[2 * STAGES + 2]);  // used in the leader CTA only
    const uint32_t bar_gfull = smem_u32(&bars[2 * STAGES + 4]);   // GEMM1: this CTA's gathered rows of a stage have landed
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;

    if (threadIdx.x < kItemSlots) s_items[threadIdx.x] = 0ull;
    if (threadIdx.x == 0) {
        s_abort = 0;
        s_prod_seq = -1;
        // full: the TMA producer's expect_tx arrival (+ GEMM1: the gather relay of each CTA)
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, MODE == 1 ? 3 : 1);
            mbar_init(bar_empty + 8 * i, 1);
            mbar_init(bar_gfull + 8 * i, 128);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(bar_tfull + 8 * i, 1); mbar_init(bar_tempty + 8 * i, 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(&s_tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // both CTAs' barriers are initialised before any remote signal
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int *abort_flag = &s_abort;
    // Everything above is local set-up.  GEMM1 reads the routing results from here on, so it waits for
    // its predecessor, and only then releases GEMM2: a GEMM2 CTA therefore never runs before the routing
    // pass is complete, and of GEMM2's roles only the producers of the Hmid rows have to wait for
    // GEMM1 itself.  The others (weight producers, scheduler) start on the first items as soon as the
    // CTA is resident, under GEMM1's tail.
    if (MODE == 1) {
        pdl_wait();
        pdl_launch_dependents();
    }

    const int k_steps = kdim / kBlockK;
    const volatile unsigned long long *queue = s_items;
    const uint32_t full0 = mapa(bar_full, 0);      // the leader's full barriers, as seen from either CTA
    const uint32_t tempty0 = mapa(bar_tempty, 0);  // the leader's accumulator-free barriers

    const int w_prod = warp == 0 ? 0 : (warp == (MODE == 1 ? 12 : 8) ? 1 : -1);
    const int b_prod = MODE == 2 ? (warp == 3 ? 0 : (warp == 9 ? 1 : -1)) : -1;
    if (w_prod >= 0) {
        // ------------------------------------------------------------------ TMA producers (weights)
        // Issuing one tensor copy keeps a warp busy for several hundred cycles; two warps take the
        // k-steps in turn.
        {
            uint32_t it_count = 0;
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq) {
                Item it;
                const int got = next_item(queue, seq, it, abort_flag);
                if (got <= 0) { ok = got == 0; break; }
                if (w_prod == 0 && lane == 0) *reinterpret_cast<volatile int *>(&s_prod_seq) = (int)seq;  // read by the scheduler warp
                const int half = ((it.n + 31) >> 5) << 4;  // B rows of this CTA; the tile has 2 * half columns
                const bool dbl = double_item(DBL_ROWS, it.n, it.mb, m_blocks);
                const uint32_t bytes = 2u * (uint32_t)((dbl ? 2 : 1) * kATileBytes + (MODE == 2 ? half * kRowBytes : 0));
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    if ((int)(it_count % kProducers) != w_prod) continue;
                    const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag));
                    if (!ok) break;
                    const uint32_t full = full0 + 8 * s;
                    const uint32_t sa = ring + s * kStageBytes;
                    if (elect_one()) {
                        if (leader) mbar_expect_tx(bar_full + 8 * s, bytes);  // the TMA bytes of both CTAs
                        if (MODE == 1)  // one box: the 64 features of block (2 mb + rank), 16 gate rows then their 16 up rows, four times
                            tma_load_5d_pair(sa, &map_a, ks * kBlockK, 0, 0, 4 * (2 * it.mb + (int)rank), it.e, full);
                        else
                            tma_load_3d_pair(sa, &map_a, ks * kBlockK, 256 * it.mb + 128 * (int)rank, it.e, full);
                        if (DBL_ROWS > 0 && dbl) {  // the next block of weight rows behind it
                            if (MODE == 1)
                                tma_load_5d_pair(sa + kATileBytes, &map_a, ks * kBlockK, 0, 0, 4 * (2 * it.mb + 2 + (int)rank), it.e, full);
                            else
                                tma_load_3d_pair(sa + kATileBytes, &map_a, ks * kBlockK, 256 * it.mb + 256 + 128 * (int)rank, it.e, full);
                        }
                    }
                    __syncwarp();
                }
            }
            if (!ok && lane == 0) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 11);
                s_abort = 1;
            }
        }
    } else if (b_prod >= 0) {
        // ------------------------------------------------------------------ TMA producers of the Hmid rows (GEMM2)
        pdl_wait();  // Hmid is GEMM1's output
        {
            uint32_t it_count = 0;
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq) {
                Item it;
                const int got = next_item(queue, seq, it, abort_flag);
                if (got <= 0) { ok = got == 0; break; }
                const int half = ((it.n + 31) >> 5) << 4;
                const int brow0 = (int)rank * half;  // first tile column / pair row this CTA loads
                const uint32_t b_off = (double_item(DBL_ROWS, it.n, it.mb, m_blocks) ? 2 : 1) * kATileBytes;
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    if ((int)(it_count % kProducers) != b_prod) continue;
                    const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag));
                    if (!ok) break;
                    const uint32_t full = full0 + 8 * s;
                    const uint32_t sb = ring + s * kStageBytes + b_off;
                    if (elect_one()) {
                        int b = 0;
#pragma unroll
                        for (int lvl = 0; lvl < 4; ++lvl) {
                            const int rows = 128 >> lvl;
                            if (rows <= HALF_MAX && half - b >= rows) {
                                tma_load_2d_pair(sb + b * kRowBytes, &maps_b.m[lvl], ks * kBlockK, it.pos0 + brow0 + b, full);
                                b += rows;
                            }
                        }
                    }
                    __syncwarp();
                }
            }
            if (!ok && lane == 0) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 16);
                s_abort = 1;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA)
        if (leader) {
            uint32_t tile_count = 0;
            uint32_t s = 0, ph = 0;  // ring stage of the next k-step and the parity of its use
            // descriptors of stage 0; stage s is (s * kStageBytes) >> 4 further in the address field
            const uint64_t a0 = smem_desc_sw128(ring), b0 = smem_desc_sw128(ring + kATileBytes);
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq, ++tile_count) {
                Item it;
                const int got = next_item(queue, seq, it, abort_flag);
                if (got <= 0) { ok = got == 0; break; }
                const int n_cols = ((it.n + 31) >> 5) << 5;
                const uint32_t idesc = instr_desc_pair(n_cols);
                const bool dbl = double_item(DBL_ROWS, it.n, it.mb, m_blocks);
                const uint32_t buf = tile_count & 1u;
                const uint32_t tph = (tile_count >> 1) & 1u;
                ok = __all_sync(0xffffffffu, mbar_wait(bar_tempty + 8 * buf, tph ^ 1u, abort_flag));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d = tmem_base + buf * kAccCols;
                if (DBL_ROWS > 0 && dbl) {
                    for (int ks = 0; ks < k_steps; ++ks) {
                        ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t a = a0 + (uint64_t)(s * (kStageBytes >> 4));
                        const uint64_t b = b0 + (uint64_t)(s * (kStageBytes >> 4) + (kATileBytes >> 4));  // the pair rows follow the second weight tile
                        if (elect_one()) {  // always the same lane: a commit covers the MMAs of the thread that issues it
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k) {  // +32 bytes per 16-element k slice inside the swizzle row
                                umma_bf16_pair(d, a + 2 * k, b + 2 * k, idesc, (ks | k) ? 1u : 0u);
                                // the second block of weight rows, into columns 128..
                                umma_bf16_pair(d + 128, a + (kATileBytes >> 4) + 2 * k, b + 2 * k, idesc, (ks | k) ? 1u : 0u);
                            }
                            umma_commit_pair(bar_empty + 8 * s);  // the stage is free in both CTAs once these MMAs have read it
                        }
                        __syncwarp();
                        if (++s == STAGES) { s = 0; ph ^= 1u; }
                    }
                } else {
                    for (int ks = 0; ks < k_steps; ++ks) {
                        ok = __all_sync(0xffffffffu, mbar_wait(bar_full + 8 * s, ph, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t a = a0 + (uint64_t)(s * (kStageBytes >> 4));
                        const uint64_t b = b0 + (uint64_t)(s * (kStageBytes >> 4));
                        if (elect_one()) {  // always the same lane: a commit covers the MMAs of the thread that issues it
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)  // +32 bytes per 16-element k slice inside the swizzle row
                                umma_bf16_pair(d, a + 2 * k, b + 2 * k, idesc, (ks | k) ? 1u : 0u);
                            umma_commit_pair(bar_empty + 8 * s);  // the stage is free in both CTAs once these MMAs have read it
                        }
                        __syncwarp();
                        if (++s == STAGES) { s = 0; ph ^= 1u; }
                    }
                }
                if (!ok) break;
                if (elect_one()) umma_commit_pair(bar_tfull + 8 * buf);    // accumulators complete in both CTAs
                __syncwarp();
            }
            if (!ok && lane == 0) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 12);
                s_abort = 1;
            }
        }
    } else if (MODE == 1 && warp == 2) {
        // ------------------------------------------------------------------ gather relay (GEMM1)
        // cp.async can only signal an mbarrier of its own CTA: this thread forwards "this CTA's
        // gathered rows of stage s have landed" to the leader's full barrier.
        {
            uint32_t it_count = 0;
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq) {
                Item it;
                const int got = next_item(queue, seq, it, abort_flag);
                if (got <= 0) { ok = got == 0; break; }
                for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                    const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                    ok = __all_sync(0xffffffffu, mbar_wait(bar_gfull + 8 * s, ph, abort_flag));
                    if (!ok) break;
                    if (elect_one()) {
                        // the rows were written by cp.async (generic proxy) and are read by the MMA through
                        // the async proxy: order the two before the stage is handed over
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                        mbar_arrive_cluster(full0 + 8 * s);
                    }
                    __syncwarp();
                }
            }
            if (!ok && lane == 0) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 15);
                s_abort = 1;
            }
        }
    } else if (warp == (MODE == 1 ? 3 : 2)) {
        // ------------------------------------------------------------------ item scheduler (leader CTA)
        if (leader) {
            const long long n_items = (long long)meta[kMetaPairTiles] * m_blocks;
            int32_t *counter = meta + (MODE == 1 ? kMetaNextItem1 : kMetaNextItem2);
            const uint32_t peer_queue = mapa(smem_u32(s_items), 1);
            const volatile int *prod_seq = &s_prod_seq;
            bool ok = true;
            for (uint32_t seq = 0; ok; ++seq) {
                // at most kSchedAhead items ahead of the one the weight producer is loading
                if (lane == 0 && (int)seq > *prod_seq + kSchedAhead) {
                    const long long t0 = clock64();
                    int spins = 0;
                    while ((int)seq > *prod_seq + kSchedAhead) {
                        __nanosleep(64);
                        if ((++spins & 63) == 0 && (*abort_flag || clock64() - t0 > kWaitLimitCycles)) { ok = false; break; }
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                bool end = false;
                if (lane == 0) {
                    Item it = {0, 0, 1, 0};
                    for (;;) {
                        const long long item = atomicAdd(counter, 1);
                        end = item >= n_items;
                        if (end) break;
                        it = load_item(item, m_blocks, tile_rows, tile_expert, tile_row0, counts, offsets);
                        // the odd block of a narrow tile belongs to the double item of the block before it
                        if (!(DBL_ROWS > 0 && it.n <= DBL_ROWS && (it.mb & 1))) break;
                    }
                    if (end) it = Item{0, 0, 1, 0};
                    const unsigned long long rec = pack_item(seq, end, it);
                    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(peer_queue + 8 * (seq % kItemSlots)), "l"(rec) : "memory");
                    *reinterpret_cast<volatile unsigned long long *>(&s_items[seq % kItemSlots]) = rec;
                }
                if (__shfl_sync(0xffffffffu, end, 0)) break;
            }
            if (!ok && lane == 0) {
                if (!*abort_flag) atomicExch(&meta[kMetaError], 17);
                s_abort = 1;
            }
        }
    } else if (MODE == 1 && warp >= 8 && warp < 12) {
        // ------------------------------------------------------------------ x-row gather (GEMM1)
        // Thread gt copies 16-byte chunk (gt & 7) of rows (gt >> 3) + 16 i, i = 0..7, of this CTA's
        // half of the tile's pair rows.  The chunk lands where the 128-byte swizzle puts it
        // (chunk index XOR row mod 8).  Each thread's copies of a stage arrive on the stage's
        // local barrier when they complete; nothing here waits for a copy.
        const int gt = threadIdx.x - 256;
        const int chunk = gt & 7, rsub = gt >> 3;
        const uint32_t dst_off = (uint32_t)(rsub * kRowBytes + ((chunk ^ (rsub & 7)) << 4));
        uint32_t it_count = 0;
        bool ok = true;
        for (uint32_t seq = 0; ok; ++seq) {
            Item it;
            const int got = next_item(queue, seq, it, abort_flag);
            if (got <= 0) { ok = got == 0; break; }
            const int half = ((it.n + 31) >> 5) << 4;
            const int brow0 = (int)rank * half;
            const uint32_t b_off = (double_item(DBL_ROWS, it.n, it.mb, m_blocks) ? 2 : 1) * kATileBytes;
            const __nv_bfloat16 *src[HALF_MAX / 16];
#pragma unroll
            for (int i = 0; i < HALF_MAX / 16; ++i) {
                const int rb = brow0 + rsub + 16 * i;
                // padding rows read token 0: their columns are never stored
                const int tok = (rsub + 16 * i < half && rb < it.n) ? pair_token[it.pos0 + rb] : 0;
                src[i] = x + (size_t)tok * x_ld + chunk * 8;
            }
            for (int ks = 0; ks < k_steps; ++ks, ++it_count) {
                const uint32_t s = it_count % STAGES, ph = (it_count / STAGES) & 1u;
                if (lane == 0) ok = mbar_wait(bar_empty + 8 * s, ph ^ 1u, abort_flag);
                ok = __shfl_sync(0xffffffffu, ok, 0);
                if (!ok) break;
                const uint32_t sb = ring + s * kStageBytes + b_off + dst_off;
#pragma unroll
                for (int i = 0; i < HALF_MAX / 16; ++i)
                    if (rsub + 16 * i < half) cp_async16(sb + i * 16 * kRowBytes, src[i] + ks * kBlockK);
                cp_async_arrive_noinc(bar_gfull + 8 * s);
            }
        }
        cp_async_wait_all();  // the copies issued so far land in this CTA before it may leave
        if (!ok && lane == 0) {
            if (!*abort_flag) atomicExch(&meta[kMetaError], 14);
            s_abort = 1;
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------------------------ epilogue warps
        const int q = warp & 3;      // TMEM lane quarter this warp may read
        const bool upper = lane >= 16;  // GEMM1: this lane holds up values; lane - 16 the gate values of the same feature
        __nv_bfloat16 *patch = patches + q * 1024;   // [32 pair rows][32 features]
        const int prow = lane >> 2, pch = lane & 3;  // 16-byte piece this lane stores: rows prow + 8 i, features 8 pch ..
        uint32_t tile_count = 0;
        bool ok = true;
        for (uint32_t seq = 0; ok; ++seq, ++tile_count) {
            Item it;
            int status = next_item(queue, seq, it, abort_flag);  // 1 item, 0 end of the list, -1 gave up
            const uint32_t buf = tile_count & 1u;
            const uint32_t tph = (tile_count >> 1) & 1u;
            if (status > 0 && !mbar_wait(bar_tfull + 8 * buf, tph, abort_flag)) status = -1;
            status = __reduce_min_sync(0xffffffffu, status);  // also reconverges the warp before the aligned TMEM loads
            if (status <= 0) { ok = status == 0; break; }
            tc_fence_after();
            // one block of weight rows of the item: accumulator columns col0.., block mb; `last`: the
            // buffer goes back to the MMA warp after this block's last read
            auto drain = [&](uint32_t col0, int mb, bool last_sub) {
            const uint32_t t0 = tmem_base + ((uint32_t)(32 * q) << 16) + buf * kAccCols + col0;
            if (MODE == 1) {
                const int f0 = 128 * mb + 64 * (int)rank + 16 * q;  // first of this warp's 16 features
                const bool f_ok = f0 < out_rows;
                for (int c0 = 0; c0 < it.n; c0 += 32) {
                    uint32_t v[32];
                    tmem_ld32_nowait(t0 + c0, v);
                    tmem_ld_wait();
                    if (last_sub && c0 + 32 >= it.n) {
                        // last read of this buffer: hand it back to the MMA warp before the stores
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty0 + 8 * buf);
                    }
                    // Columns in pairs: the gate lane finishes the even column, the up lane the odd one;
                    // one shuffle hands each the value it lacks.
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float even = __uint_as_float(v[2 * i]), odd = __uint_as_float(v[2 * i + 1]);
                        const float got = __shfl_xor_sync(0xffffffffu, upper ? even : odd, 16);
                        const float h = upper ? swiglu(got, odd) : swiglu(even, got);
                        patch[(2 * i + (upper ? 1 : 0)) * 16 + (lane & 15)] = __float2bfloat16_rn(h);  // [32 pair rows][16 features]
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int piece = lane + 32 * i;  // 16-byte piece: pair row piece / 2, features 8 (piece & 1) ..
                        const int r = piece >> 1;
                        const uint4 val = *reinterpret_cast<const uint4 *>(patch + piece * 8);
                        if (f_ok && c0 + r < it.n)
                            *reinterpret_cast<uint4 *>(out + (size_t)(it.pos0 + c0 + r) * out_ld + f0 + (piece & 1) * 8) = val;
                    }
                    __syncwarp();
                }
            } else {
                const int row0 = 256 * mb + 128 * (int)rank + 32 * q;  // first of this warp's 32 output features
                const bool r_ok = row0 < out_rows;
                for (int c0 = 0; c0 < it.n; c0 += 32) {
                    float v[32];
                    tmem_ld32(t0 + c0, v);
                    if (last_sub && c0 + 32 >= it.n) {
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(tempty0 + 8 * buf);
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) patch[j * 32 + lane] = __float2bfloat16_rn(v[j]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int r = prow + 8 * i;
                        const uint4 val = *reinterpret_cast<const uint4 *>(patch + r * 32 + pch * 8);
                        if (r_ok && c0 + r < it.n)
                            *reinterpret_cast<uint4 *>(out + (size_t)(it.pos0 + c0 + r) * out_ld + row0 + pch * 8) = val;
                    }
                    __syncwarp();
                }
            }
            };
            if (DBL_ROWS > 0 && double_item(DBL_ROWS, it.n, it.mb, m_blocks)) {
                drain(0, it.mb, false);
                drain(128, it.mb + 1, true);
            } else {
                drain(0, it.mb, true);
            }
        }
        if (!ok && lane == 0) {
            if (!*abort_flag) atomicExch(&meta[kMetaError], 13);
            s_abort = 1;
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA leaves (or frees TMEM) while the other may still signal or read it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

template <int MODE, int HALF_MAX, int STAGES, int DBL_ROWS>
constexpr int pair_smem_bytes() {
    return STAGES * StageBytes<HALF_MAX, DBL_ROWS>::value + kPatchBytes + 1024;
}

// One configuration of the kernel: its attribute set-up and its launch.
template <int MODE, int HALF_MAX, int STAGES, int DBL_ROWS>
struct PairKernel {
    static constexpr int kSmem = pair_smem_bytes<MODE, HALF_MAX, STAGES, DBL_ROWS>();
    static bool prepare() {
        return cudaFuncSetAttribute(expert_gemm_pair_kernel<MODE, HALF_MAX, STAGES, DBL_ROWS>,
                                    cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem) == cudaSuccess;
    }
    template <typename... Args>
    static cudaError_t launch(const zeda_moe *h, cudaStream_t s, Args &&...args) {
        const int grid = (h->sm_count / 2) * 2;
        return launch_kernel(h->pdl, expert_gemm_pair_kernel<MODE, HALF_MAX, STAGES, DBL_ROWS>, dim3(grid),
                             dim3(MODE == 1 ? kThreadsGather : kThreads), kSmem, s, std::forward<Args>(args)...);
    }
};

// small: at most 64 pair rows per expert (decode batches, T <= 64), a weight stream with many small
// stages; big: tiles of up to 256 pair rows
using Gemm1Small = PairKernel<1, 32, 6, 64>;   // every tile of a small batch is a double item: 6 x (16 + 16 + 4 KB)
using Gemm2Small = PairKernel<2, 32, 10, 0>;
using Gemm1Mid = PairKernel<1, 64, 9, 0>;
using Gemm2Mid = PairKernel<2, 64, 9, 0>;
// Large tiles: six stages of 36 KB (a full tile's 16 + 16 KB, a double item of up to 64 pair rows
// 16 + 16 + 4 KB).  GEMM1 has a second form for batches whose experts mostly hold 65..128 pairs: double
// items up to 128 rows on five stages of 40 KB.
using Gemm1Big = PairKernel<1, 128, 6, 64>;
using Gemm1Wide = PairKernel<1, 128, 5, 128>;
using Gemm2Big = PairKernel<2, 128, 6, 64>;
constexpr int kSmallRowsMax = 64;
constexpr int kMidRowsPerExpert = 100;  // mean slots per candidate (T K / (N + N_Z)) up to which the mid geometry is used
constexpr int kWideRowsPerExpert = 256; // ... and up to which GEMM1 runs tiles of up to 128 rows as double items

// The small geometry holds at most kSmallRowsMax pair rows of one expert.  Without expert parallelism
// an expert has at most one pair per token of the call; with it, any number of the received rows.
bool small_geometry(const zeda_moe *h, const ExpertWork &w) {
    const int per_expert_bound = h->cfg.ep_size >= 1 ? w.rows_bound : w.rows_bound / h->cfg.top_k;
    return per_expert_bound <= kSmallRowsMax;
}

}  // namespace

// Mid-sized batches, where an expert holds fewer than about 100 pairs on average and the layer streams
// every expert's weights once (HBM-bound), get tiles of 128 rows and the ring of eight 24 KB stages:
// more weight bytes in flight per SM than the six 32 KB stages whose activation half stays half empty.
// The host knows neither the counts nor the zero share of a call; it goes by the mean number of slots
// per candidate.
int tile_rows_for(const zeda_moe *h, int T) {
    const zeda_moe_config_t &c = h->cfg;
    if (c.ep_size >= 1) return kPairTileM;
    return (long long)T * c.top_k <= (long long)kMidRowsPerExpert * (c.n_real + c.n_zero) ? kMidTileM : kPairTileM;
}

int init_pair_kernels(zeda_moe *h) {
    const zeda_moe_config_t &c = h->cfg;
    PairMaps *pm = static_cast<PairMaps *>(aligned_alloc(64, sizeof(PairMaps)));
    if (!pm) { set_error("out of host memory"); return -1; }
    const cuuint64_t E = h->n_local, d = c.d_model, He = c.d_expert;
    const cuuint64_t rows = (cuuint64_t)h->pair_rows + kPairTileM;
    bool ok = true;
    {
        // a 5-D view of [N][2 He][d] that lets one box fetch 64 features as four groups of 16 gate rows
        // each followed by the matching 16 up rows: (k, row in group, gate | up, group of 16 rows, expert)
        const cuuint64_t dims[5] = {d, 16, 2, He / 16, E};
        const cuuint64_t strides[4] = {d * 2, He * d * 2, 16 * d * 2, 2 * He * d * 2};
        const cuuint32_t box[5] = {kBlockK, 16, 2, 4, 1};
        ok = ok && encode_bf16_map(&pm->w_gate_up, h->w_gate_up, 5, dims, strides, box);
    }
    {
        const cuuint64_t dims[3] = {He, d, E};
        const cuuint64_t strides[2] = {He * 2, d * He * 2};
        const cuuint32_t box[3] = {kBlockK, 128, 1};
        ok = ok && encode_bf16_map(&pm->w_down, h->w_down, 3, dims, strides, box);
    }
    for (int i = 0; i < 4; ++i) {
        const cuuint64_t dims[2] = {He, rows};
        const cuuint64_t strides[1] = {He * 2};
        const cuuint32_t box[2] = {kBlockK, (cuuint32_t)(128 >> i)};
        ok = ok && encode_bf16_map(&pm->hmid.m[i], h->ws.hmid, 2, dims, strides, box);
    }
    ok = ok && Gemm1Small::prepare() && Gemm2Small::prepare() && Gemm1Mid::prepare() && Gemm2Mid::prepare() &&
         Gemm1Big::prepare() && Gemm1Wide::prepare() && Gemm2Big::prepare();
    if (!ok) {
        free(pm);
        if (zeda_last_error()[0] == 0) set_error("pair kernel set-up failed: %s", cudaGetErrorString(cudaGetLastError()));
        return -1;
    }
    h->pmaps = pm;
    return 0;
}

int launch_experts_gemm1_pair(const zeda_moe *h, const __nv_bfloat16 *x, const ExpertWork &w, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    const PairMaps *pm = static_cast<const PairMaps *>(h->pmaps);
    const int m_blocks = (c.d_expert + 127) / 128;
    auto go = [&](auto k) {
        return decltype(k)::launch(h, s, pm->w_gate_up, pm->hmid, x, c.d_model, w.counts, w.offsets, w.tile_expert,
                                   w.tile_row0, w.pair_row, ws.meta, c.d_model, c.d_expert, m_blocks, ws.hmid, c.d_expert,
                                   w.tile_rows);
    };
    // an expert cannot hold more pair rows than the call has tokens (a token selects it at most once)
    // (an expert-parallel rank does not know its load from the call's shape: it takes the form for large batches)
    const bool wide = c.ep_size < 1 && (long long)w.rows_bound <= (long long)kWideRowsPerExpert * (c.n_real + c.n_zero);
    const cudaError_t e = small_geometry(h, w) ? go(Gemm1Small{}) : w.tile_rows == kMidTileM ? go(Gemm1Mid{}) : wide ? go(Gemm1Wide{}) : go(Gemm1Big{});
    return e == cudaSuccess ? 1 : -1;
}

int launch_experts_gemm2_pair(const zeda_moe *h, const ExpertWork &w, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    const PairMaps *pm = static_cast<const PairMaps *>(h->pmaps);
    const int m_blocks = (c.d_model + 255) / 256;
    auto go = [&](auto k) {
        return decltype(k)::launch(h, s, pm->w_down, pm->hmid, (const __nv_bfloat16 *)nullptr, 0, w.counts, w.offsets,
                                   w.tile_expert, w.tile_row0, w.pair_row, ws.meta, c.d_expert, c.d_model, m_blocks,
                                   ws.obuf, c.d_model, w.tile_rows);
    };
    const cudaError_t e = small_geometry(h, w) ? go(Gemm2Small{}) : w.tile_rows == kMidTileM ? go(Gemm2Mid{}) : go(Gemm2Big{});
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
