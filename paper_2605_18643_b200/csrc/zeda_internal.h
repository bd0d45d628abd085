// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "zeda.h"

namespace zeda {

constexpr int kMaxCand = 512;       // N + N_Z limit (16 logits per lane in the top-K warp)
constexpr int kMaxTopK = 16;
constexpr int kSortTokens = 128;    // tokens per CTA in the counting sort (histogram / placement)
constexpr int kPairTileM = 256;     // most pair rows per tile of the expert kernels (one CTA pair, N <= 256)
constexpr int kMidTileM = 128;      // tile rows of the geometry for mid-sized batches
constexpr int kMaxEpRanks = 64;     // expert-parallel group size limit

// Device-resident counters of one call.
enum MetaSlot {
    kMetaPairs = 0,      // P
    kMetaActive = 1,     // U
    kMetaZeroSlots = 2,  // slots that landed on zero experts
    kMetaError = 5,      // sticky error word written by bounded device waits
    kMetaMaxRows = 6,    // largest per-expert pair count
    kMetaPairTiles = 7,  // entries of the expert kernels' tile list
    kMetaNextItem1 = 8,  // next unclaimed work item of the GEMM1 kernel (reset by the routing pass)
    kMetaNextItem2 = 9,  // the same for GEMM2
    kMetaHistTicket = 10,  // placement CTAs that have read the block histograms (the last one clears them)
    kMetaCount = 16
};

struct Workspace {
    int32_t *topk_idx;     // [maxT*K]
    float *topk_w;         // [maxT*K]
    int32_t *inv;          // [maxT*K] slot -> sorted position, -1 for zero slots
    int32_t *perm;         // [maxT*K] sorted position -> slot
    int32_t *pair_token;   // [maxT*K] sorted position -> token
    int32_t *block_hist;   // [nblk*N]
    int32_t *counts;       // [N]
    int32_t *offsets;      // [N+1]
    int32_t *meta;         // [kMetaCount]
    int32_t *ptile_expert; // [maxTiles] tiles of at most kPairTileM pair rows of one expert
    int32_t *ptile_row0;   // [maxTiles] first row of the tile within its expert
    float *logits;         // [maxT*(N+N_Z)]
    float *stat_part;      // [nblk_stats * 2 * (N+N_Z)]
    __nv_bfloat16 *hmid;   // [maxT*K, He]
    __nv_bfloat16 *obuf;   // [maxT*K, d]
    __nv_bfloat16 *router_split; // [3][pad128(N+N_Z)][d] bf16 hi/mid/lo pieces of the router rows
    __nv_bfloat16 *x_stage;// [maxT, d]
    __nv_bfloat16 *y_stage;// [maxT, d]
    // expert-parallel handles only: the plan of the rows received from the group
    int32_t *ep_counts;      // [N_local] received pairs per local expert
    int32_t *ep_offsets;     // [N_local + 1]
    int32_t *ep_pair_row;    // [maxR] sorted position -> received row
    int32_t *ep_row_pos;     // [maxR] received row -> sorted position
    int32_t *ep_tile_expert; // [maxR / kPairTileM + N_local + 1]
    int32_t *ep_tile_row0;
};

// What one launch of the expert kernels works on: per-expert counts and offsets of the pair rows,
// the tile list, and for GEMM1 the row of the activation matrix that each pair row reads.
struct ExpertWork {
    const int32_t *counts, *offsets, *tile_expert, *tile_row0, *pair_row;
    int rows_bound;  // upper bound of the pair rows of a call (host-side; picks the kernel geometry)
    int tile_rows;   // pair rows per tile of the tile list (kPairTileM or kMidTileM)
};

// Device-side tile list written by the expert scan: experts in id order, each with its tiles of at
// most kPairTileM pair rows in row order.
struct WorkLists {
    int32_t *ptile_expert, *ptile_row0;
};

struct RouteOut {  // where one routing pass writes (user buffers or workspace)
    int32_t *topk_idx;
    float *topk_w;
    int32_t *counts;
    int32_t *offsets;
    int32_t *perm;
    int32_t *n_pairs;  // optional extra copy of P
};

}  // namespace zeda

struct zeda_moe {
    zeda_moe_config_t cfg;
    bool pdl;  // launch the forward kernels with programmatic stream serialization
    const float *router_w;
    const float *router_bias;
    const __nv_bfloat16 *w_gate_up;
    const __nv_bfloat16 *w_down;
    zeda::Workspace ws;
    int sm_count;
    int max_tiles;
    int n_local;    // experts whose weights this handle holds (n_real unless expert-parallel)
    int pair_rows;  // capacity of the pair buffers (max_tokens * top_k, or max_recv_pairs)
    int last_launches;
    void *pmaps;  // host-side tensor maps of the expert kernels (owned)
    void *router_maps;  // host-side tensor map of the split router weights (owned)
    bool profiling;
    bool profiled_last;
    int last_routed_tokens;  // T of the most recent routing pass on this handle
    cudaEvent_t ev[ZEDA_STAGE_COUNT + 1];
    // host-buffer entry point: copy streams and events of its two-chunk pipeline (made on first use)
    cudaStream_t copy_in, copy_out;
    cudaEvent_t ev_host[6];
};

namespace zeda {

// ---- launchers (each returns the number of kernels it enqueued, or <0 on a launch error) ----
int init_route_kernels(const zeda_moe *h);
// With n_parts == nullptr the logits are complete.  Otherwise the router may cut the reduction axis
// into *n_parts slices (mid-sized batches on the tensor-core path): slice p then lies at
// logits + p * T * n_cand, and launch_route_from_logits adds the slices in order.
int launch_router_logits(const zeda_moe *h, const __nv_bfloat16 *x, int T, float *logits, cudaStream_t s,
                         int *n_parts = nullptr);
int launch_route_from_logits(const zeda_moe *h, const float *logits, int T, const RouteOut &out, cudaStream_t s,
                             int n_parts = 1);
int launch_stats(const zeda_moe *h, const float *logits, const int32_t *topk_idx, int T, float *f,
                 float *p_mean, float *out, cudaStream_t s);
int router_split_pad(int n_cand);
int init_router_tile(zeda_moe *h);
constexpr int kRouterMaxSplit = 4;
// rows of n_cand floats that the workspace holds for router output (complete logits or their slices)
inline long long router_part_rows(long long max_tokens) {
    const long long cap = 9600;  // past this many tokens the unsplit grid covers the SMs already
    const long long want = kRouterMaxSplit * max_tokens < cap ? kRouterMaxSplit * max_tokens : cap;
    return max_tokens > want ? max_tokens : want;
}
int router_split_factor(const zeda_moe *h, int T);
int launch_router_logits_tile(const zeda_moe *h, const __nv_bfloat16 *x, int T, float *logits, int split, cudaStream_t s);
int init_pair_kernels(zeda_moe *h);
// Pair rows per tile for a call of T tokens on this handle: the routing pass builds the tile list with
// it and the expert kernels of the same call are picked to match.
int tile_rows_for(const zeda_moe *h, int T);
int launch_token_zero_share(const zeda_moe *h, int T, float *out, cudaStream_t s);
int launch_experts_gemm1_pair(const zeda_moe *h, const __nv_bfloat16 *x, const ExpertWork &w, cudaStream_t s);
int launch_experts_gemm2_pair(const zeda_moe *h, const ExpertWork &w, cudaStream_t s);
// expert-parallel pieces (expert_parallel.cu)
int launch_ep_pack(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *send_rows, int32_t *send_counts,
                   int32_t *expert_counts, cudaStream_t s);
int launch_ep_plan(const zeda_moe *h, const int32_t *recv_counts, int n_rows, cudaStream_t s);
int launch_ep_unsort(const zeda_moe *h, int n_rows, __nv_bfloat16 *out_rows, cudaStream_t s);
int launch_combine_rows(const zeda_moe *h, const __nv_bfloat16 *rows, const __nv_bfloat16 *x, int T, __nv_bfloat16 *y,
                        cudaStream_t s);
int launch_wait_selftest(const zeda_moe *h, long long limit_cycles, cudaStream_t s);
int launch_combine(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *y, cudaStream_t s);
// combine fused with the residual + RMSNorm glue of a layer stack (rows of up to 2048 elements)
bool combine_glue_supported(const zeda_moe *h);
int launch_combine_glue(const zeda_moe *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *resid, __nv_bfloat16 *h_next, float eps,
                        cudaStream_t s);

void set_error(const char *fmt, ...);
// remembers the error of a failed kernel launch for the status message of the API call (the runtime's
// own "last error" may have been read and cleared by a later launch check)
void note_launch_error(cudaError_t e);

// ---- programmatic dependent launch ------------------------------------------------------------
// The kernels of one forward pass are launched back to back on one stream.  Launched with the
// attribute below, a kernel may start (launch latency, barrier and TMEM set-up) while its
// predecessor is still draining; it touches no global memory until pdl_wait() returns, which is
// when the predecessor has completed and its writes are visible.  Each kernel calls
// pdl_launch_dependents() first thing so that its successor is released as early as possible.
// Without the attribute both calls do nothing.
#if defined(__CUDACC__)
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                 Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
    if (e != cudaSuccess) note_launch_error(e);
    return e;
}
#endif

}  // namespace zeda
