// Device work of one rank of an expert-parallel group.  The experts are partitioned over G ranks in
// contiguous blocks, the tokens stay with their rank.  Zero-expert slots are dropped by the routing
// pass before anything is packed, so they cost neither FLOPs nor link bytes (Section 2.1: a zero
// expert outputs 0; Appendix A names expert-parallel dispatch as future work).
//
//   pack    x rows of the surviving pairs in (expert, token) order -> send buffer; rows per
//           destination rank from the expert offsets (experts of one rank are a contiguous range)
//   plan    from the G x N_local matrix of received pair counts: per-expert counts and offsets of
//           the received rows, the tile list of the expert kernels, and the two maps between the
//           received order (source rank, expert, token) and the sorted order (expert, source rank,
//           token)
//   unsort  expert outputs from the sorted order back into the received order
// The exchange between the calls is the caller's (an all-to-all with per-rank row counts).
#include "expert_scan.cuh"

namespace zeda {

namespace {

// 16-byte copies of whole rows: dst[r] = src[idx[r]] for r < n_rows, where n_rows is read from
// device memory when n_rows_dev is given (the host does not know P).
__global__ void __launch_bounds__(256)
gather_rows_kernel(__nv_bfloat16 *__restrict__ dst, const __nv_bfloat16 *__restrict__ src,
                   const int32_t *__restrict__ idx, int n_rows, const int32_t *__restrict__ n_rows_dev, int d) {
    pdl_launch_dependents();
    pdl_wait();
    if (n_rows_dev) n_rows = min(n_rows, *n_rows_dev);
    const int chunks = d / 8;
    const int rows_per_cta = blockDim.x / 32;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int r = blockIdx.x * rows_per_cta + warp; r < n_rows; r += gridDim.x * rows_per_cta) {
        const uint4 *s = reinterpret_cast<const uint4 *>(src + (size_t)__ldg(idx + r) * d);
        uint4 *o = reinterpret_cast<uint4 *>(dst + (size_t)r * d);
        for (int c0 = lane; c0 < chunks; c0 += 128) {  // four loads in flight per lane
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (c0 + 32 * u < chunks) v[u] = __ldg(s + c0 + 32 * u);
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (c0 + 32 * u < chunks) o[c0 + 32 * u] = v[u];
        }
    }
}

// Rows per destination rank: experts [r * n_local, (r + 1) * n_local) belong to rank r.
__global__ void ep_send_counts_kernel(const int32_t *__restrict__ offsets, const int32_t *__restrict__ counts,
                                      int n_ranks, int n_local, int32_t *__restrict__ send_counts,
                                      int32_t *__restrict__ expert_counts) {
    pdl_launch_dependents();
    pdl_wait();
    for (int r = threadIdx.x; r < n_ranks; r += blockDim.x)
        send_counts[r] = offsets[(r + 1) * n_local] - offsets[r * n_local];
    if (expert_counts)
        for (int e = threadIdx.x; e < n_ranks * n_local; e += blockDim.x) expert_counts[e] = counts[e];
}

// One CTA per source rank s.  Every CTA sums the count matrix (it is small), runs the expert scan
// (CTA 0 publishes counts, offsets and counters; the tile list is filled by all CTAs, a share each)
// and then maps its own source's rows: received row = rows of earlier sources + rows of this source
// for earlier experts + i; sorted position = expert offset + rows of earlier sources for the same
// expert + i.
__global__ void __launch_bounds__(512)
ep_plan_kernel(const int32_t *__restrict__ recv_counts, int n_ranks, int n_local, int n_rows,
               int32_t *__restrict__ counts, int32_t *__restrict__ offsets, int32_t *__restrict__ meta,
               const WorkLists wl, int32_t *__restrict__ pair_row, int32_t *__restrict__ row_pos) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ ScanShared sh;
    __shared__ int32_t before[kMaxCand];      // rows of sources < s for expert j
    __shared__ int32_t mine[kMaxCand + 1];    // exclusive scan of this source's counts
    __shared__ int32_t s_src_base, s_total;
    const int s = blockIdx.x;
    for (int j = threadIdx.x; j < n_local; j += blockDim.x) {
        int total = 0, bef = 0;
        for (int q = 0; q < n_ranks; ++q) {
            const int c = max(0, __ldg(recv_counts + q * n_local + j));
            total += c;
            if (q < s) bef += c;
        }
        sh.cnt[j] = total;
        before[j] = bef;
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        // rows of this source before expert j, and the rows of all earlier sources
        int base = 0;
        for (int j0 = 0; j0 < n_local; j0 += 32) {
            const int j = j0 + threadIdx.x;
            const int c = j < n_local ? max(0, __ldg(recv_counts + s * n_local + j)) : 0;
            int sc = c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(kFull, sc, o);
                if ((int)threadIdx.x >= o) sc += a;
            }
            if (j < n_local) mine[j] = base + sc - c;
            base += __shfl_sync(kFull, sc, 31);
        }
        int earlier = 0;
        for (int j = threadIdx.x; j < n_local; j += 32) earlier += before[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) earlier += __shfl_xor_sync(kFull, earlier, o);
        int total = 0;
        for (int j = threadIdx.x; j < n_local; j += 32) total += sh.cnt[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) total += __shfl_xor_sync(kFull, total, o);
        if (threadIdx.x == 0) {
            mine[n_local] = base;
            s_src_base = earlier;
            s_total = total;
        }
    }
    __syncthreads();
    // The caller's row count must be the matrix's sum (the buffers were sized by it): if it is not,
    // the call is marked failed and planned as empty.
    const bool consistent = s_total == n_rows;
    if (!consistent) {
        if (s == 0 && threadIdx.x == 0) atomicExch(&meta[kMetaError], 21);
        for (int j = threadIdx.x; j < n_local; j += blockDim.x) sh.cnt[j] = 0;
        // the unsort pass still runs over n_rows rows: every one of them reads row 0 of the result
        // buffer (in bounds; the call's output is undefined)
        for (int r = s * blockDim.x + threadIdx.x; r < n_rows; r += gridDim.x * blockDim.x) row_pos[r] = 0;
        __syncthreads();
    }
    finish_expert_scan(sh, n_local, consistent ? n_rows : 0, counts, offsets, nullptr, meta, wl, s == 0, s, gridDim.x);
    __syncthreads();
    const int my_rows = consistent ? mine[n_local] : 0, src_base = s_src_base;
    for (int i = threadIdx.x; i < my_rows; i += blockDim.x) {
        int lo = 0, hi = n_local;  // invariant: mine[lo] <= i < mine[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (mine[mid] <= i) lo = mid; else hi = mid;
        }
        const int row = src_base + i;
        const int pos = sh.off[lo] + before[lo] + (i - mine[lo]);
        if (row < n_rows && pos < n_rows) {
            pair_row[pos] = row;
            row_pos[row] = pos;
        }
    }
}

}  // namespace

int launch_ep_pack(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *send_rows, int32_t *send_counts,
                   int32_t *expert_counts, cudaStream_t s) {
    const zeda_moe_config_t &c = h->cfg;
    const Workspace &ws = h->ws;
    const int slots = T * c.top_k;
    const int grid = min((slots + 7) / 8, 8 * h->sm_count);
    cudaError_t e = launch_kernel(h->pdl, gather_rows_kernel, dim3(grid), dim3(256), 0, s, send_rows, x,
                                  (const int32_t *)ws.pair_token, slots, (const int32_t *)(ws.meta + kMetaPairs), c.d_model);
    if (e != cudaSuccess) return -1;
    e = launch_kernel(h->pdl, ep_send_counts_kernel, dim3(1), dim3(256), 0, s, (const int32_t *)ws.offsets,
                      (const int32_t *)ws.counts, (int)c.ep_size, h->n_local, send_counts, expert_counts);
    return e == cudaSuccess ? 2 : -1;
}

int launch_ep_plan(const zeda_moe *h, const int32_t *recv_counts, int n_rows, cudaStream_t s) {
    const Workspace &ws = h->ws;
    const WorkLists wl = {ws.ep_tile_expert, ws.ep_tile_row0};
    const cudaError_t e = launch_kernel(h->pdl, ep_plan_kernel, dim3(h->cfg.ep_size), dim3(512), 0, s, recv_counts,
                                        (int)h->cfg.ep_size, h->n_local, n_rows, ws.ep_counts, ws.ep_offsets, ws.meta, wl,
                                        ws.ep_pair_row, ws.ep_row_pos);
    return e == cudaSuccess ? 1 : -1;
}

int launch_ep_unsort(const zeda_moe *h, int n_rows, __nv_bfloat16 *out_rows, cudaStream_t s) {
    const int grid = min((n_rows + 7) / 8, 8 * h->sm_count);
    const cudaError_t e = launch_kernel(h->pdl, gather_rows_kernel, dim3(grid), dim3(256), 0, s, out_rows,
                                        (const __nv_bfloat16 *)h->ws.obuf, (const int32_t *)h->ws.ep_row_pos, n_rows,
                                        (const int32_t *)nullptr, h->cfg.d_model);
    return e == cudaSuccess ? 1 : -1;
}

}  // namespace zeda
