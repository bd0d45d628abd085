// The expert scan shared by the routing pass and the expert-parallel plan: from per-expert pair
// counts to exclusive offsets, the counters of the call and the tile list of the expert kernels.
#pragma once

#include "zeda_internal.h"

namespace zeda {

constexpr unsigned kFull = 0xffffffffu;

struct ScanShared {
    int32_t cnt[kMaxCand];
    int32_t off[kMaxCand + 1];
    int32_t ptile[kMaxCand + 1];  // exclusive scan of the experts' tile counts
};

// From per-expert pair counts in sh.cnt: exclusive offsets, P, U, and the tile list of the expert
// kernels (experts in id order, each with its tiles of tile_rows rows in row order; the last tile of
// an expert may be ragged).  Called by every thread of the CTA (blockDim.x >= 32); contains CTA
// barriers.
__device__ __forceinline__ void finish_expert_scan(ScanShared &sh, int n_real, int total_slots,
                                                   int32_t *__restrict__ counts, int32_t *__restrict__ offsets,
                                                   int32_t *__restrict__ n_pairs_out, int32_t *__restrict__ meta,
                                                   const WorkLists &wl, bool write_global = true,
                                                   int list_part = 0, int list_parts = 1, int tile_rows = kPairTileM) {
    if (threadIdx.x < 32) {
        // warp 0 scans the per-expert sequences in steps of 32 with shuffle prefix sums
        int base_off = 0, base_ptile = 0, active = 0, max_rows = 0;
        for (int e0 = 0; e0 < n_real; e0 += 32) {
            const int i = e0 + threadIdx.x;
            const int c = (i < n_real) ? sh.cnt[i] : 0;
            const int pt = (c + tile_rows - 1) / tile_rows;
            int so = c, sp = pt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(kFull, so, o);
                const int q = __shfl_up_sync(kFull, sp, o);
                if ((int)threadIdx.x >= o) { so += a; sp += q; }
            }
            if (i < n_real) {
                sh.off[i] = base_off + so - c;
                sh.ptile[i] = base_ptile + sp - pt;
            }
            base_off += __shfl_sync(kFull, so, 31);
            base_ptile += __shfl_sync(kFull, sp, 31);
            active += __popc(__ballot_sync(kFull, c > 0));
            int mx = c;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(kFull, mx, o));
            max_rows = max(max_rows, mx);
        }
        if (threadIdx.x == 0) {
            sh.off[n_real] = base_off;
            sh.ptile[n_real] = base_ptile;
        }
        if (threadIdx.x == 0 && write_global) {
            meta[kMetaPairs] = base_off;
            meta[kMetaActive] = active;
            meta[kMetaZeroSlots] = total_slots - base_off;
            meta[kMetaPairTiles] = base_ptile;
            meta[kMetaMaxRows] = max_rows;
            meta[kMetaNextItem1] = 0;
            meta[kMetaNextItem2] = 0;
            if (n_pairs_out) *n_pairs_out = base_off;
        }
    }
    __syncthreads();
    if (write_global) {  // (uniform over the CTA)
        for (int e = threadIdx.x; e < n_real; e += blockDim.x) {
            if (counts) counts[e] = sh.cnt[e];
            offsets[e] = sh.off[e];
        }
        if (threadIdx.x == 0) offsets[n_real] = sh.off[n_real];
    }
    // Tile list: every CTA that runs this scan holds the same prefix sums, so the CTAs share the
    // filling (part list_part of list_parts); a CTA outside that sharing passes list_parts = 0.
    if (list_parts <= 0) return;
    // entry i belongs to the expert whose first-entry index is the last one <= i
    const int total = sh.ptile[n_real];
    for (int i = list_part * blockDim.x + threadIdx.x; i < total; i += list_parts * blockDim.x) {
        int lo = 0, hi = n_real;  // invariant: ptile[lo] <= i < ptile[hi]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (sh.ptile[mid] <= i) lo = mid; else hi = mid;
        }
        wl.ptile_expert[i] = lo;
        wl.ptile_row0[i] = (i - sh.ptile[lo]) * tile_rows;
    }
}

}  // namespace zeda
