// Routing stage: router logits over the N + N_Z candidates, softmax / top-K / routing weights
// (Section 2.1), then the compaction that drops zero-expert slots and counting-sorts the surviving
// (token, normal expert) pairs by expert in a stable order.
#include <cooperative_groups.h>

#include <atomic>

#include "expert_scan.cuh"

namespace zeda {

namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}

// ---------------------------------------------------------------------------------------------
// Router logits, CUDA-core version: l[t, j] = <x_t, W_r[j]> + b[j] in fp32.
// One CTA = kTok tokens (bf16 rows staged in shared memory) x a slice of the candidates; one warp
// per candidate row, lanes striding the feature axis with 16-byte loads.
// ---------------------------------------------------------------------------------------------
constexpr int kTok = 8;
constexpr int kRouterUnroll = 8;  // 16-byte weight loads a lane keeps in flight

__global__ void __launch_bounds__(256)
router_logits_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ router_w,
                     const float *__restrict__ router_bias, int T, int d, int n_cand,
                     int cand_per_cta, float *__restrict__ logits) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __nv_bfloat16 *xs = reinterpret_cast<__nv_bfloat16 *>(smem_raw);  // [kTok][d]
    const int t0 = blockIdx.x * kTok;
    const int nt = min(kTok, T - t0);
    const int vec_per_row = d / 8;
    // eight 16-byte loads in flight per thread (a plain load-store loop waits for each load in turn)
    for (int i0 = threadIdx.x; i0 < kTok * vec_per_row; i0 += 8 * blockDim.x) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u * blockDim.x;
            const int r = i / vec_per_row, c = i % vec_per_row;
            v[u] = make_uint4(0, 0, 0, 0);
            if (i < kTok * vec_per_row && r < nt) v[u] = __ldg(reinterpret_cast<const uint4 *>(x + (size_t)(t0 + r) * d) + c);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = i0 + u * blockDim.x;
            if (i < kTok * vec_per_row) reinterpret_cast<uint4 *>(xs + (size_t)(i / vec_per_row) * d)[i % vec_per_row] = v[u];
        }
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int j_begin = blockIdx.y * cand_per_cta;
    const int j_end = min(n_cand, j_begin + cand_per_cta);
    for (int j = j_begin + warp; j < j_end; j += 8) {
        float acc[kTok];
#pragma unroll
        for (int r = 0; r < kTok; ++r) acc[r] = 0.f;
        const float4 *wrow = reinterpret_cast<const float4 *>(router_w + (size_t)j * d);
        for (int c4 = lane; c4 < d / 4; c4 += 32 * kRouterUnroll) {
            float4 w[kRouterUnroll];
#pragma unroll
            for (int u = 0; u < kRouterUnroll; ++u)  // independent 16-byte loads in flight per lane
                w[u] = (c4 + 32 * u < d / 4) ? __ldg(wrow + c4 + 32 * u) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < kRouterUnroll; ++u) {
                if (c4 + 32 * u < d / 4) {
#pragma unroll
                    for (int r = 0; r < kTok; ++r) {
                        const uint2 xv = reinterpret_cast<const uint2 *>(xs + (size_t)r * d)[c4 + 32 * u];
                        const float x0 = __uint_as_float(xv.x << 16), x1 = __uint_as_float(xv.x & 0xffff0000u);
                        const float x2 = __uint_as_float(xv.y << 16), x3 = __uint_as_float(xv.y & 0xffff0000u);
                        acc[r] = fmaf(w[u].x, x0, acc[r]);
                        acc[r] = fmaf(w[u].y, x1, acc[r]);
                        acc[r] = fmaf(w[u].z, x2, acc[r]);
                        acc[r] = fmaf(w[u].w, x3, acc[r]);
                    }
                }
            }
        }
        const float b = router_bias ? __ldg(router_bias + j) : 0.f;
#pragma unroll
        for (int r = 0; r < kTok; ++r) {
            const float s = warp_sum(acc[r]);
            if (lane == 0 && r < nt) logits[(size_t)(t0 + r) * n_cand + j] = s + b;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Softmax, top-K and routing weights: one warp per token, logits held in registers (candidate
// j lives in lane j % 32, register j / 32).  K rounds of warp arg-max; equal logits go to the
// lower candidate id.
// ---------------------------------------------------------------------------------------------
constexpr int kRegsPerLane = kMaxCand / 32;

// Top-K and routing weights of one token by one warp.  On return lane k < K holds slot k.
// RPL = logits per lane (32 * RPL >= n_cand).
// The row may arrive as n_parts partial sums, part_stride floats apart; they are added in order.
template <int RPL>
__device__ __forceinline__ void topk_gate_token(const float *__restrict__ row, int n_parts, size_t part_stride,
                                                int n_real, int n_cand, int K,
                                                int gate_mode, int lane, int &my_idx, float &my_w) {
    float v[RPL];
#pragma unroll
    for (int r = 0; r < RPL; ++r) {
        const int j = r * 32 + lane;
        v[r] = (j < n_cand) ? row[j] : -INFINITY;
    }
    for (int p = 1; p < n_parts; ++p) {
#pragma unroll
        for (int r = 0; r < RPL; ++r) {
            const int j = r * 32 + lane;
            if (j < n_cand) v[r] += row[p * part_stride + j];
        }
    }
    // row maximum and softmax denominator over all candidates
    float m = v[0];
#pragma unroll
    for (int r = 1; r < RPL; ++r) m = fmaxf(m, v[r]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
    float den = 0.f;
#pragma unroll
    for (int r = 0; r < RPL; ++r) {
        const int j = r * 32 + lane;
        if (j < n_cand) den += expf(v[r] - m);
    }
    den = warp_sum(den);

    // Selection on order-preserving integer keys (0 = not available), so that one warp-wide integer
    // maximum finds the best logit and one integer minimum the lowest candidate id that holds it.
    unsigned key[RPL];
#pragma unroll
    for (int r = 0; r < RPL; ++r) {
        unsigned u = __float_as_uint(v[r]);
        if (u == 0x80000000u) u = 0u;  // -0 and +0 are equal logits: the lower id decides between them
        key[r] = (r * 32 + lane < n_cand) ? ((u & 0x80000000u) ? ~u : (u | 0x80000000u)) : 0u;
    }
    unsigned my_key = 0u;
    my_idx = -1;
    for (int k = 0; k < K; ++k) {
        unsigned lm = key[0];
#pragma unroll
        for (int r = 1; r < RPL; ++r) lm = max(lm, key[r]);
        const unsigned gm = __reduce_max_sync(kFull, lm);
        int cand = 0x7fffffff;
#pragma unroll
        for (int r = RPL - 1; r >= 0; --r)
            if (key[r] == gm) cand = r * 32 + lane;  // ends on this lane's lowest id with that logit
        const int bj = __reduce_min_sync(kFull, cand);
#pragma unroll
        for (int r = 0; r < RPL; ++r)
            if (r * 32 + lane == bj) key[r] = 0u;
        if (lane == k) { my_idx = bj; my_key = gm; }
    }
    // lane k < K holds slot k: its softmax probability, then the sums over the selected slots
    float my_p = 0.f;
    if (lane < K) {
        const float bv = __uint_as_float((my_key & 0x80000000u) ? (my_key & 0x7fffffffu) : ~my_key);
        my_p = expf(bv - m) / den;
    }
    const float sum_sel = warp_sum(my_p);
    const float sum_real = warp_sum(my_idx >= 0 && my_idx < n_real ? my_p : 0.f);
    my_w = my_p;
    if (gate_mode == ZEDA_GATE_TOPK_NORM) my_w = my_p / sum_sel;
    else if (gate_mode == ZEDA_GATE_RENORM_REAL) my_w = (my_idx < n_real && sum_real > 0.f) ? my_p / sum_real : 0.f;
}

// block_hist (optional): pass 1 of the counting sort done here.  Every slot on a normal expert adds 1
// to its entry of the histogram of its block of kSortTokens tokens (integer adds: the counts do not
// depend on their order).  The histograms must be zero on entry; the placement kernel that consumes
// them zeroes them again.
template <int RPL>
__global__ void __launch_bounds__(256)
topk_gate_kernel(const float *__restrict__ logits, int n_parts, int T, int n_real, int n_cand, int K, int gate_mode,
                 int32_t *__restrict__ topk_idx, float *__restrict__ topk_w, int32_t *__restrict__ block_hist) {
    pdl_launch_dependents();
    pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + warp;
    if (t >= T) return;
    int my_idx;
    float my_w;
    topk_gate_token<RPL>(logits + (size_t)t * n_cand, n_parts, (size_t)T * n_cand, n_real, n_cand, K, gate_mode, lane,
                         my_idx, my_w);
    if (lane < K) {
        topk_idx[(size_t)t * K + lane] = my_idx;
        topk_w[(size_t)t * K + lane] = my_w;
        if (block_hist && (unsigned)my_idx < (unsigned)n_real)
            atomicAdd(block_hist + (size_t)(t / kSortTokens) * n_real + my_idx, 1);
    }
}

// ---------------------------------------------------------------------------------------------
// Counting sort, pass 1 as a kernel of its own (the paths that do not take it in the top-K kernel):
// per-CTA histogram of the normal-expert slots of kSortTokens tokens.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
slot_hist_kernel(const int32_t *__restrict__ topk_idx, int T, int K, int n_real,
                 int32_t *__restrict__ block_hist) {
    pdl_launch_dependents();
    pdl_wait();
    extern __shared__ int32_t hist[];  // [n_real]
    for (int e = threadIdx.x; e < n_real; e += blockDim.x) hist[e] = 0;
    __syncthreads();
    const int s0 = blockIdx.x * kSortTokens * K;
    const int s1 = min(T * K, s0 + kSortTokens * K);
    for (int s = s0 + threadIdx.x; s < s1; s += blockDim.x) {
        const int e = topk_idx[s];
        if ((unsigned)e < (unsigned)n_real) atomicAdd(&hist[e], 1);  // zero experts and ids < 0 are dropped
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n_real; e += blockDim.x) block_hist[(size_t)blockIdx.x * n_real + e] = hist[e];
}

// ---------------------------------------------------------------------------------------------
// Counting sort, pass 2 (one CTA): column-wise exclusive scan over the CTA histograms, expert
// counts, exclusive offsets, P, U, and the work lists of the expert kernels.
// ---------------------------------------------------------------------------------------------
constexpr int kScanSlabInts = 8192;  // 32 KB of CTA histograms per slab of the expert scan

// Copies n ints from global to shared memory with sixteen loads in flight per thread: a plain
// load-store loop issues its loads one L2 round trip after another (the store waits for the load).
__device__ __forceinline__ void stage_ints(int32_t *__restrict__ dst, const int32_t *__restrict__ src, int n) {
    constexpr int kInFlight = 16;
    for (int i0 = threadIdx.x; i0 < n; i0 += kInFlight * blockDim.x) {
        int32_t v[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int i = i0 + u * blockDim.x;
            v[u] = i < n ? __ldg(src + i) : 0;
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int i = i0 + u * blockDim.x;
            if (i < n) dst[i] = v[u];
        }
    }
}

__global__ void __launch_bounds__(512)
expert_scan_kernel(int32_t *__restrict__ block_hist, int nblk, int n_real, int total_slots,
                   int32_t *__restrict__ counts, int32_t *__restrict__ offsets,
                   int32_t *__restrict__ n_pairs_out, int32_t *__restrict__ meta, const WorkLists wl, int tile_rows) {
    __shared__ ScanShared sh;
    // Exclusive scan of every expert column over the CTA histograms.  The histograms are staged in
    // shared memory slab by slab with independent coalesced loads (a load-scan-store loop straight
    // on global memory is a chain of dependent L2 round trips), scanned by one thread per expert,
    // and written back coalesced.
    __shared__ int32_t slab[kScanSlabInts];
    const int slab_blocks = max(1, kScanSlabInts / n_real);
    const int e = threadIdx.x;
    int run = 0;
    for (int b0 = 0; b0 < nblk; b0 += slab_blocks) {
        const int nb = min(slab_blocks, nblk - b0);
        int32_t *g = block_hist + (size_t)b0 * n_real;
        for (int i = threadIdx.x; i < nb * n_real; i += blockDim.x) slab[i] = g[i];
        __syncthreads();
        if (e < n_real) {
            for (int b = 0; b < nb; ++b) {
                const int c = slab[b * n_real + e];
                slab[b * n_real + e] = run;  // pairs of expert e in earlier CTAs
                run += c;
            }
        }
        __syncthreads();
        for (int i = threadIdx.x; i < nb * n_real; i += blockDim.x) g[i] = slab[i];
        __syncthreads();
    }
    if (e < n_real) sh.cnt[e] = run;
    __syncthreads();
    finish_expert_scan(sh, n_real, total_slots, counts, offsets, n_pairs_out, meta, wl, true, 0, 1, tile_rows);
}

// ---------------------------------------------------------------------------------------------
// Small batches (T <= 128, decode): top-K, routing weights and the whole counting sort in ONE
// launch of a thread-block cluster.  Each CTA of the cluster takes 16 tokens (one warp per token)
// and records "token t selected expert e" as bit t of a T-bit mask that lives in CTA 0's shared
// memory (distributed shared memory, atomicOr).  A token selects an expert at most once, so an
// expert's count is a popcount and the stable rank of a pair is the popcount of the lower token
// bits: the (expert, token) order needs no atomics on positions and no second pass.  After the
// cluster barrier CTA 0 scans the experts and places the pairs.
// ---------------------------------------------------------------------------------------------
constexpr int kSmallTokens = 128;
constexpr int kSmallCluster = 8;
constexpr int kSmallThreads = 32 * (kSmallTokens / kSmallCluster);  // one warp per token

template <int RPL>
__global__ void __cluster_dims__(kSmallCluster, 1, 1) __launch_bounds__(kSmallThreads)
route_small_kernel(const float *__restrict__ logits, int T, int n_real, int n_cand, int K, int gate_mode,
                   int32_t *__restrict__ topk_idx, float *__restrict__ topk_w, int32_t *__restrict__ counts,
                   int32_t *__restrict__ offsets, int32_t *__restrict__ n_pairs_out, int32_t *__restrict__ meta,
                   const WorkLists wl, int tile_rows, int32_t *__restrict__ perm,
                   int32_t *__restrict__ perm_user, int32_t *__restrict__ inv, int32_t *__restrict__ pair_token) {
    pdl_launch_dependents();
    pdl_wait();
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ ScanShared sh;
    __shared__ uint32_t sel[kMaxCand][kSmallTokens / 32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const unsigned rank = cluster.block_rank();
    if (rank == 0)
        for (int i = threadIdx.x; i < n_real * (kSmallTokens / 32); i += blockDim.x) (&sel[0][0])[i] = 0u;
    cluster.sync();
    uint32_t *sel0 = cluster.map_shared_rank(&sel[0][0], 0);
    const int t = rank * (kSmallThreads / 32) + warp;
    if (t < T) {
        int my_idx;
        float my_w;
        topk_gate_token<RPL>(logits + (size_t)t * n_cand, 1, 0, n_real, n_cand, K, gate_mode, lane, my_idx, my_w);
        if (lane < K) {
            topk_idx[(size_t)t * K + lane] = my_idx;
            topk_w[(size_t)t * K + lane] = my_w;
            if (my_idx < n_real) atomicOr(sel0 + my_idx * (kSmallTokens / 32) + (t >> 5), 1u << (t & 31));
        }
    }
    cluster.sync();  // release/acquire at cluster scope: masks and topk_idx of every CTA are visible
    if (rank != 0) return;
    if ((int)threadIdx.x < n_real) {
        int c = 0;
#pragma unroll
        for (int i = 0; i < kSmallTokens / 32; ++i) c += __popc(sel[threadIdx.x][i]);
        sh.cnt[threadIdx.x] = c;
    }
    __syncthreads();
    finish_expert_scan(sh, n_real, T * K, counts, offsets, n_pairs_out, meta, wl, true, 0, 1, tile_rows);
    for (int s = threadIdx.x; s < T * K; s += blockDim.x) {
        const int e = topk_idx[s], tk = s / K;
        int p = -1;
        if (e < n_real) {
            int r = __popc(sel[e][tk >> 5] & ((1u << (tk & 31)) - 1u));
            for (int i = 0; i < (tk >> 5); ++i) r += __popc(sel[e][i]);
            p = sh.off[e] + r;
            perm[p] = s;
            if (perm_user) perm_user[p] = s;
            pair_token[p] = tk;
        }
        inv[s] = p;
    }
}

// ---------------------------------------------------------------------------------------------
// Counting sort, pass 3: stable placement.  Each CTA re-walks its kSortTokens*K slots in slot
// order; each warp owns a contiguous run of slots, ranks equal experts inside a 32-slot step with
// match.any / popc (a warp-level prefix count) and carries per-expert running positions in shared
// memory.  No atomics decide a position, so the order is (expert, token) ascending every run.
// ---------------------------------------------------------------------------------------------
constexpr int kPlaceWarps = 8;
constexpr int kFoldMaxBlocks = 256;  // up to this many CTA histograms the placement CTAs scan them themselves

__global__ void __launch_bounds__(kPlaceWarps * 32)
slot_place_kernel(const int32_t *__restrict__ topk_idx, int T, int K, int n_real,
                  const int32_t *__restrict__ block_base, const int32_t *__restrict__ offsets,
                  int32_t *__restrict__ perm, int32_t *__restrict__ perm_user,
                  int32_t *__restrict__ inv, int32_t *__restrict__ pair_token) {
    extern __shared__ int32_t pos[];  // [kPlaceWarps][n_real]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < kPlaceWarps * n_real; i += blockDim.x) pos[i] = 0;
    __syncthreads();
    const int s0 = blockIdx.x * kSortTokens * K;
    const int s1 = min(T * K, s0 + kSortTokens * K);
    const int per_warp = ((kSortTokens * K + kPlaceWarps - 1) / kPlaceWarps + 31) / 32 * 32;
    const int w0 = s0 + warp * per_warp;
    const int w1 = min(s1, w0 + per_warp);
    int32_t *mine = pos + warp * n_real;
    const unsigned lt = (1u << lane) - 1u;
    // count this warp's slots per expert
    for (int s = w0 + lane; s - lane < w1; s += 32) {
        int e = (s < w1) ? topk_idx[s] : -1;
        if ((unsigned)e >= (unsigned)n_real) e = -1;  // zero experts; ids < 0 are dropped the same way
        const unsigned grp = __match_any_sync(kFull, e);
        if (e >= 0 && (grp & lt) == 0) mine[e] += __popc(grp);
        __syncwarp();
    }
    __syncthreads();
    // turn counts into start positions: global offset + earlier CTAs + earlier warps
    for (int e = threadIdx.x; e < n_real; e += blockDim.x) {
        int run = offsets[e] + block_base[(size_t)blockIdx.x * n_real + e];
        for (int w = 0; w < kPlaceWarps; ++w) {
            const int c = pos[w * n_real + e];
            pos[w * n_real + e] = run;
            run += c;
        }
    }
    __syncthreads();
    for (int s = w0 + lane; s - lane < w1; s += 32) {
        int e = (s < w1) ? topk_idx[s] : -1;
        const bool in_range = s < w1;
        if ((unsigned)e >= (unsigned)n_real) e = -1;  // zero experts; ids < 0 are dropped the same way
        const unsigned grp = __match_any_sync(kFull, e);
        int p = -1;
        if (e >= 0) p = mine[e] + __popc(grp & lt);
        __syncwarp();
        if (e >= 0 && (grp & lt) == 0) mine[e] += __popc(grp);
        __syncwarp();
        if (in_range) {
            inv[s] = p;
            if (p >= 0) {
                perm[p] = s;
                if (perm_user) perm_user[p] = s;
                pair_token[p] = s / K;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Counting sort, passes 2 + 3 in one launch (used while the CTA histograms are few): every CTA
// sums the histogram columns itself (pairs of each expert in earlier CTAs, and in all CTAs), scans
// the expert totals, and places its slots as above.  CTA 0 also publishes counts, offsets and the
// counters; the work lists are filled by all CTAs, a share each.  Saves a launch and the single-CTA
// scan between two short kernels.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPlaceWarps * 32)
slot_scan_place_kernel(const int32_t *__restrict__ topk_idx, int T, int K, int n_real, int nblk,
                       int32_t *__restrict__ block_hist, int32_t *__restrict__ counts,
                       int32_t *__restrict__ offsets, int32_t *__restrict__ n_pairs_out, int32_t *__restrict__ meta,
                       const WorkLists wl, int tile_rows, int32_t *__restrict__ perm, int32_t *__restrict__ perm_user,
                       int32_t *__restrict__ inv, int32_t *__restrict__ pair_token) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ ScanShared sh;
    extern __shared__ int32_t pos[];       // [kPlaceWarps][n_real], then base[n_real], then a histogram slab
    int32_t *base = pos + kPlaceWarps * n_real;
    int32_t *slab = base + n_real;         // [kScanSlabInts]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // this warp's slots, fetched now (their latency passes under the histogram sums below): slot
    // w0 + 32 u + lane in e_reg[u], -1 for zero-expert slots and beyond the end
    constexpr int kSlotRegs = kSortTokens * kMaxTopK / kPlaceWarps / 32;
    const int s0 = blockIdx.x * kSortTokens * K;
    const int s1 = min(T * K, s0 + kSortTokens * K);
    const int per_warp = ((kSortTokens * K + kPlaceWarps - 1) / kPlaceWarps + 31) / 32 * 32;
    const int w0 = s0 + warp * per_warp;
    const int w1 = min(s1, w0 + per_warp);
    int e_reg[kSlotRegs];
#pragma unroll
    for (int u = 0; u < kSlotRegs; ++u) {
        const int s = w0 + 32 * u + lane;
        int e = (32 * u < per_warp && s < w1) ? __ldg(topk_idx + s) : -1;
        e_reg[u] = (unsigned)e >= (unsigned)n_real ? -1 : e;
    }
    for (int i = threadIdx.x; i < kPlaceWarps * n_real; i += blockDim.x) pos[i] = 0;
    for (int e = threadIdx.x; e < n_real; e += blockDim.x) { base[e] = 0; sh.cnt[e] = 0; }
    // column sums of the CTA histograms: staged slab by slab with independent coalesced loads (a
    // per-thread loop over global memory would be one L2 round trip after another)
    const int slab_blocks = max(1, kScanSlabInts / n_real);
    for (int b0 = 0; b0 < nblk; b0 += slab_blocks) {
        const int nb = min(slab_blocks, nblk - b0);
        const int32_t *g = block_hist + (size_t)b0 * n_real;
        __syncthreads();
        stage_ints(slab, g, nb * n_real);
        __syncthreads();
        for (int e = threadIdx.x; e < n_real; e += blockDim.x) {
            int before = 0, total = 0;
            for (int b = 0; b < nb; ++b) {
                const int c = slab[b * n_real + e];
                total += c;
                if (b0 + b < (int)blockIdx.x) before += c;
            }
            base[e] += before;
            sh.cnt[e] += total;
        }
    }
    __syncthreads();
    // The histograms go back to zero for the next call's top-K kernel: the CTA that is last to have
    // read them (a ticket, nobody waits) clears them and the ticket counter.
    __shared__ int s_ticket;
    if (threadIdx.x == 0) {
        __threadfence();
        s_ticket = atomicAdd(meta + kMetaHistTicket, 1);
    }
    __syncthreads();
    if (s_ticket == (int)gridDim.x - 1) {
        for (int i = threadIdx.x; i < nblk * n_real; i += blockDim.x) block_hist[i] = 0;
        if (threadIdx.x == 0) meta[kMetaHistTicket] = 0;
    }
    finish_expert_scan(sh, n_real, T * K, counts, offsets, n_pairs_out, meta, wl, blockIdx.x == 0, blockIdx.x, gridDim.x, tile_rows);
    __syncthreads();
    int32_t *mine = pos + warp * n_real;
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int u = 0; u < kSlotRegs; ++u) {
        if (w0 + 32 * u >= w1 || 32 * u >= per_warp) break;  // (uniform over the warp)
        const int e = e_reg[u];
        const unsigned grp = __match_any_sync(kFull, e);
        if (e >= 0 && (grp & lt) == 0) mine[e] += __popc(grp);
        __syncwarp();
    }
    __syncthreads();
    for (int e = threadIdx.x; e < n_real; e += blockDim.x) {
        int run = sh.off[e] + base[e];
        for (int w = 0; w < kPlaceWarps; ++w) {
            const int c = pos[w * n_real + e];
            pos[w * n_real + e] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int u = 0; u < kSlotRegs; ++u) {
        if (w0 + 32 * u >= w1 || 32 * u >= per_warp) break;  // (uniform over the warp)
        const int s = w0 + 32 * u + lane;
        const int e = e_reg[u];
        const bool in_range = s < w1;
        const unsigned grp = __match_any_sync(kFull, e);
        int p = -1;
        if (e >= 0) p = mine[e] + __popc(grp & lt);
        __syncwarp();
        if (e >= 0 && (grp & lt) == 0) mine[e] += __popc(grp);
        __syncwarp();
        if (in_range) {
            inv[s] = p;
            if (p >= 0) {
                perm[p] = s;
                if (perm_user) perm_user[p] = s;
                pair_token[p] = s / K;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Routing statistics (Eq. 4-6 forward values), two deterministic passes: per-CTA partial sums of
// the selection indicator and of the softmax probabilities, then a fixed-order final reduction.
// ---------------------------------------------------------------------------------------------
constexpr int kStatTokens = 64;

__global__ void __launch_bounds__(256)
stats_partial_kernel(const float *__restrict__ logits, const int32_t *__restrict__ topk_idx, int T, int K,
                     int n_cand, float *__restrict__ part) {
    extern __shared__ float sm[];  // [2][n_cand]
    float *sf = sm, *sp = sm + n_cand;
    for (int i = threadIdx.x; i < 2 * n_cand; i += blockDim.x) sm[i] = 0.f;
    __syncthreads();
    __shared__ float s_max[kStatTokens], s_den[kStatTokens];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * kStatTokens;
    const int t1 = min(T, t0 + kStatTokens);
    // per-token softmax maximum and denominator, one warp per token
    for (int t = t0 + warp; t < t1; t += (blockDim.x >> 5)) {
        const float *row = logits + (size_t)t * n_cand;
        float m = -INFINITY;
        for (int c = lane; c < n_cand; c += 32) m = fmaxf(m, row[c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, o));
        float den = 0.f;
        for (int c = lane; c < n_cand; c += 32) den += expf(row[c] - m);
        den = warp_sum(den);
        if (lane == 0) { s_max[t - t0] = m; s_den[t - t0] = den; }
    }
    __syncthreads();
    // one thread per candidate, tokens summed in increasing order
    for (int j = threadIdx.x; j < n_cand; j += blockDim.x) {
        float accp = 0.f, accf = 0.f;
        for (int t = t0; t < t1; ++t) {
            accp += expf(logits[(size_t)t * n_cand + j] - s_max[t - t0]) / s_den[t - t0];
            for (int k = 0; k < K; ++k) accf += (topk_idx[(size_t)t * K + k] == j) ? 1.f : 0.f;
        }
        sf[j] = accf;
        sp[j] = accp;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * n_cand; i += blockDim.x) part[(size_t)blockIdx.x * 2 * n_cand + i] = sm[i];
}

__global__ void __launch_bounds__(512)
stats_final_kernel(const float *__restrict__ part, int nblk, int T, int K, int n_real, int n_cand,
                   float *__restrict__ f, float *__restrict__ p_mean, float *__restrict__ out) {
    __shared__ float sf[kMaxCand], sp[kMaxCand];
    const int j = threadIdx.x;
    if (j < n_cand) {
        float af = 0.f, ap = 0.f;
        for (int b = 0; b < nblk; ++b) {
            af += part[(size_t)b * 2 * n_cand + j];
            ap += part[(size_t)b * 2 * n_cand + n_cand + j];
        }
        sf[j] = af / T;
        sp[j] = ap / T;
        if (f) f[j] = sf[j];
        if (p_mean) p_mean[j] = sp[j];
    }
    __syncthreads();
    if (threadIdx.x == 0 && out) {
        float la = 0.f, fE = 0.f, pE = 0.f, fZ = 0.f, pZ = 0.f;
        for (int i = 0; i < n_cand; ++i) {
            la += sf[i] * sp[i];
            if (i < n_real) { fE += sf[i]; pE += sp[i]; } else { fZ += sf[i]; pZ += sp[i]; }
        }
        out[0] = fZ / K;
        out[1] = la;
        out[2] = fE * pE;
        out[3] = fZ * pZ;
    }
}

// Per-token zero-expert ratio (Section 2.2, looked at per token in Section 4.1): the share of the
// token's K slots that selected a zero expert.
__global__ void __launch_bounds__(256)
token_zero_share_kernel(const int32_t *__restrict__ topk_idx, int T, int K, int n_real, float *__restrict__ out) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    int zero = 0;
    for (int k = 0; k < K; ++k) zero += topk_idx[(size_t)t * K + k] >= n_real ? 1 : 0;
    out[t] = (float)zero / (float)K;
}

}  // namespace

int launch_token_zero_share(const zeda_moe *h, int T, float *out, cudaStream_t s) {
    token_zero_share_kernel<<<(T + 255) / 256, 256, 0, s>>>(h->ws.topk_idx, T, h->cfg.top_k, h->cfg.n_real, out);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int init_route_kernels(const zeda_moe *h) {
    const size_t smem = (size_t)kTok * h->cfg.d_model * sizeof(__nv_bfloat16);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(router_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return -1;
    // placement CTAs: static scan state plus (per-warp positions, bases, a histogram slab) pass 48 KB
    // together when there are many experts
    const int place_smem = (int)sizeof(int32_t) * ((kPlaceWarps + 1) * kMaxCand + kScanSlabInts);
    if (cudaFuncSetAttribute(slot_scan_place_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, place_smem) != cudaSuccess)
        return -1;
    return 0;
}

int launch_router_logits(const zeda_moe *h, const __nv_bfloat16 *x, int T, float *logits, cudaStream_t s, int *n_parts) {
    if (n_parts) *n_parts = 1;
    // large batches: the GEMM goes to the tensor cores (exact three-way bf16 split of the weights)
    if (T >= 256 && h->router_maps) {
        const int split = n_parts ? router_split_factor(h, T) : 1;
        if (n_parts) *n_parts = split;
        return launch_router_logits_tile(h, x, T, logits, split, s);
    }
    const int d = h->cfg.d_model, n_cand = h->cfg.n_real + h->cfg.n_zero;
    const int tiles = (T + kTok - 1) / kTok;
    // split the candidates over grid.y until the grid covers the SMs about twice
    int splits = 1;
    const int max_splits = (n_cand + 7) / 8;
    while (tiles * splits < 2 * h->sm_count && splits < max_splits) splits *= 2;
    if (splits > max_splits) splits = max_splits;
    const int per = (n_cand + splits - 1) / splits;
    const size_t smem = (size_t)kTok * d * sizeof(__nv_bfloat16);
    const cudaError_t e = launch_kernel(h->pdl, router_logits_kernel, dim3(tiles, (n_cand + per - 1) / per), dim3(256), smem, s,
                                        x, h->router_w, h->router_bias, T, d, n_cand, per, logits);
    return e == cudaSuccess ? 1 : -1;
}

int launch_route_from_logits(const zeda_moe *h, const float *logits, int T, const RouteOut &out, cudaStream_t s, int n_parts) {
    const zeda_moe_config_t &c = h->cfg;
    const int n_cand = c.n_real + c.n_zero, K = c.top_k;
    const Workspace &ws = h->ws;
    const int nblk = (T + kSortTokens - 1) / kSortTokens;
    int launches = 4;
    const WorkLists wl = {ws.ptile_expert, ws.ptile_row0};
    const int tile_rows = tile_rows_for(h, T);
#define ZEDA_RPL_DISPATCH(CALL)                        \
    do {                                               \
        if (n_cand <= 64) { CALL(2); }                 \
        else if (n_cand <= 128) { CALL(4); }           \
        else if (n_cand <= 192) { CALL(6); }           \
        else if (n_cand <= 256) { CALL(8); }           \
        else { CALL(16); }                             \
    } while (0)
    if (T <= kSmallTokens && c.n_real <= kSmallThreads) {
#define ZEDA_CALL_SMALL(R)                                                                                         \
    launch_kernel(h->pdl, route_small_kernel<R>, dim3(kSmallCluster), dim3(kSmallThreads), 0, s,                    \
        logits, T, c.n_real, n_cand, K, c.gate_mode, ws.topk_idx, ws.topk_w, ws.counts, ws.offsets, out.n_pairs,   \
        ws.meta, wl, tile_rows, ws.perm, out.perm, ws.inv, ws.pair_token)
        ZEDA_RPL_DISPATCH(ZEDA_CALL_SMALL);
#undef ZEDA_CALL_SMALL
        launches = 1;
    } else {
        // up to kFoldMaxBlocks sort blocks the top-K kernel counts the slots itself and one more launch
        // scans and places; beyond, histogram, scan and placement are kernels of their own
        const bool fold = nblk <= kFoldMaxBlocks;
        int32_t *hist_in_topk = fold ? ws.block_hist : nullptr;
#define ZEDA_CALL_TOPK(R) \
    launch_kernel(h->pdl, topk_gate_kernel<R>, dim3((T + 7) / 8), dim3(256), 0, s, logits, n_parts, T, c.n_real, n_cand, K, \
                  c.gate_mode, ws.topk_idx, ws.topk_w, hist_in_topk)
        ZEDA_RPL_DISPATCH(ZEDA_CALL_TOPK);
#undef ZEDA_CALL_TOPK
        if (fold) {
            launch_kernel(h->pdl, slot_scan_place_kernel, dim3(nblk), dim3(kPlaceWarps * 32),
                          sizeof(int32_t) * ((kPlaceWarps + 1) * c.n_real + kScanSlabInts), s, (const int32_t *)ws.topk_idx, T, K, c.n_real,
                          nblk, ws.block_hist, ws.counts, ws.offsets, out.n_pairs, ws.meta, wl, tile_rows, ws.perm,
                          out.perm, ws.inv, ws.pair_token);
            launches = 2;
        } else {
            launch_kernel(h->pdl, slot_hist_kernel, dim3(nblk), dim3(256), sizeof(int32_t) * c.n_real, s,
                          (const int32_t *)ws.topk_idx, T, K, c.n_real, ws.block_hist);
            expert_scan_kernel<<<1, 512, 0, s>>>(ws.block_hist, nblk, c.n_real, T * K, ws.counts, ws.offsets,
                                                 out.n_pairs, ws.meta, wl, tile_rows);
            slot_place_kernel<<<nblk, kPlaceWarps * 32, sizeof(int32_t) * kPlaceWarps * c.n_real, s>>>(
                ws.topk_idx, T, K, c.n_real, ws.block_hist, ws.offsets, ws.perm, out.perm, ws.inv, ws.pair_token);
        }
    }
    if (cudaGetLastError() != cudaSuccess) return -1;
    // copies for a caller that asked for the routing itself
    const cudaMemcpyKind d2d = cudaMemcpyDeviceToDevice;
    if (out.topk_idx) cudaMemcpyAsync(out.topk_idx, ws.topk_idx, sizeof(int32_t) * (size_t)T * K, d2d, s);
    if (out.topk_w) cudaMemcpyAsync(out.topk_w, ws.topk_w, sizeof(float) * (size_t)T * K, d2d, s);
    if (out.counts) cudaMemcpyAsync(out.counts, ws.counts, sizeof(int32_t) * c.n_real, d2d, s);
    if (out.offsets) cudaMemcpyAsync(out.offsets, ws.offsets, sizeof(int32_t) * (c.n_real + 1), d2d, s);
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

int launch_stats(const zeda_moe *h, const float *logits, const int32_t *topk_idx, int T, float *f,
                 float *p_mean, float *out, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const int n_cand = c.n_real + c.n_zero;
    const int nblk = (T + kStatTokens - 1) / kStatTokens;
    stats_partial_kernel<<<nblk, 256, sizeof(float) * 2 * n_cand, s>>>(logits, topk_idx, T, c.top_k, n_cand,
                                                                      h->ws.stat_part);
    stats_final_kernel<<<1, 512, 0, s>>>(h->ws.stat_part, nblk, T, c.top_k, c.n_real, n_cand, f, p_mean, out);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace zeda

// ---------------------------------------------------------------------------------------------
// zeda_compact_static: the counting sort above for callers that cannot allocate device memory.
// Its scratch (per-CTA histograms, slot -> position table, pair -> token table, work lists,
// counters) lives in the fixed array below instead of a caller-provided workspace.  Every GPU
// that loads this library holds the array until the process exits.
// ---------------------------------------------------------------------------------------------
namespace zeda {
namespace {

constexpr int kStaticMaxTokens = ZEDA_STATIC_MAX_TOKENS;
constexpr int kStaticMaxSlots = ZEDA_STATIC_MAX_SLOTS;
constexpr int kStaticBlocks = (kStaticMaxTokens + kSortTokens - 1) / kSortTokens;
constexpr int kStaticLists = kStaticMaxSlots / kPairTileM + kMaxCand + 1;

struct StaticScratch {
    int32_t block_hist[kStaticBlocks * kMaxCand];
    int32_t inv[kStaticMaxSlots];
    int32_t pair_token[kStaticMaxSlots];
    int32_t ptile_expert[kStaticLists];
    int32_t ptile_row0[kStaticLists];
    int32_t meta[kMetaCount];
};

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

constexpr int kMaxDevices = 64;
// device address of the array, per device; atomic so that host threads may race on the first call
std::atomic<StaticScratch *> g_static_ptr[kMaxDevices] = {};

}  // namespace
}  // namespace zeda

extern "C" zeda_status_t zeda_compact_static(const int32_t *topk_idx, int32_t T, int32_t top_k, int32_t n_real,
                                             int32_t *expert_counts, int32_t *expert_offsets, int32_t *perm,
                                             int32_t *n_pairs, void *stream) {
    using namespace zeda;
    if (T == 0) return ZEDA_OK;
    if (T < 0 || T > kStaticMaxTokens || top_k < 1 || top_k > kMaxTopK || (long long)T * top_k > kStaticMaxSlots) {
        set_error("zeda_compact_static handles at most %d tokens and %d slots (T * top_k); got T=%d, top_k=%d",
                  kStaticMaxTokens, kStaticMaxSlots, T, top_k);
        return ZEDA_ERR_UNSUPPORTED;
    }
    if (n_real < 1 || n_real > kMaxCand) { set_error("n_real must be in [1, %d]", kMaxCand); return ZEDA_ERR_UNSUPPORTED; }
    if (!topk_idx || !expert_counts || !expert_offsets || !perm || !n_pairs) {
        set_error("zeda_compact_static: every pointer is required");
        return ZEDA_ERR_INVALID_ARG;
    }
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { set_error("cudaGetDevice: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
    if (dev < 0 || dev >= kMaxDevices) { set_error("device ordinal %d not supported", dev); return ZEDA_ERR_UNSUPPORTED; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    StaticScratch *sc = g_static_ptr[dev].load(std::memory_order_acquire);
    if (!sc) {
        // One-time set-up for this device: in host code the array's name is only a stand-in, the
        // kernels need its device address.  The lookup is not a stream operation, so it must not
        // happen while the stream is being captured.
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        e = cudaStreamIsCapturing(s, &cap);
        if (e != cudaSuccess) { set_error("cudaStreamIsCapturing: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
        if (cap != cudaStreamCaptureStatusNone) {
            set_error("zeda_compact_static: the first call on a device must come before stream capture begins");
            return ZEDA_ERR_INVALID_ARG;
        }
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) { set_error("cudaGetSymbolAddress: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
        sc = static_cast<StaticScratch *>(p);
        g_static_ptr[dev].store(sc, std::memory_order_release);  // every thread would store the same address
    }
    // the array keeps the previous call's contents; the counters start from zero every call
    e = cudaMemsetAsync(sc->meta, 0, sizeof(sc->meta), s);
    if (e != cudaSuccess) { set_error("cudaMemsetAsync: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
    const int nblk = (T + kSortTokens - 1) / kSortTokens;
    slot_hist_kernel<<<nblk, 256, sizeof(int32_t) * n_real, s>>>(topk_idx, T, top_k, n_real, sc->block_hist);
    const WorkLists wl = {sc->ptile_expert, sc->ptile_row0};
    expert_scan_kernel<<<1, 512, 0, s>>>(sc->block_hist, nblk, n_real, T * top_k, expert_counts, expert_offsets,
                                         n_pairs, sc->meta, wl, kPairTileM);
    slot_place_kernel<<<nblk, kPlaceWarps * 32, sizeof(int32_t) * kPlaceWarps * n_real, s>>>(
        topk_idx, T, top_k, n_real, sc->block_hist, expert_offsets, perm, nullptr, sc->inv, sc->pair_token);
    e = cudaGetLastError();
    if (e != cudaSuccess) { set_error("zeda_compact_static launch: %s", cudaGetErrorString(e)); return ZEDA_ERR_CUDA; }
    return ZEDA_OK;
}

