/*
 * zeda.h - C ABI of the B200 (sm_100a) forward pass of an MoE layer with zero-output experts.
 *
 * The layer (paper Section 2.1 "Zero-Expert Injection", Eq. 1): a router scores N normal experts
 * and N_Z zero experts (Z_j(h) = 0), keeps the top-K of the union, and the output is
 *     y~(h) = sum over the selected slots that are normal experts of g~_i(h) * E_i(h),
 * with the routing weights of the surviving slots left as they were (Section 4.3.4: no
 * renormalisation; Eq. 7 is the renormalised variant).  Each expert has gate, up and down
 * projections (Appendix D), read here as down(silu(gate x) * up x).
 *
 * Conventions
 *   - Candidate ids: 0..N-1 normal experts, N..N+N_Z-1 zero experts (E' = E u Z).
 *   - "dev" pointers are CUDA device pointers on the handle's device, "host" pointers are host
 *     memory.  The caller owns every buffer it passes (weights, workspace, inputs, outputs) and
 *     keeps weights and workspace alive and unmodified until zeda_moe_destroy.  The library never
 *     allocates, frees or resizes device memory.
 *   - bf16 tensors are passed as const void* / void* (16-bit patterns), row-major, 16-byte aligned.
 *   - Calls enqueue work on the given cudaStream_t (passed as void*, NULL = default stream) and
 *     return without synchronising, except where stated.  Outputs are valid once the stream has
 *     been synchronised.  A handle is not thread-safe; distinct handles are independent.
 *   - zeda_moe_forward, zeda_route and zeda_residual_rmsnorm only enqueue kernels and device-to-device
 *     copies: a call can be captured in a CUDA graph and replayed on new contents of the same buffers
 *     (the buffer addresses and T are part of the captured launches).
 *   - Every entry point returns a zeda_status_t (ZEDA_OK = 0); nothing throws, aborts or traps.
 *     Arguments are checked before anything is launched; zeda_last_error() gives a text for the
 *     last failure on the calling thread.
 */
#ifndef ZEDA_H_
#define ZEDA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct zeda_moe zeda_moe_t; /* opaque; host memory owned by the library */

typedef enum {
    ZEDA_OK = 0,
    ZEDA_ERR_INVALID_ARG = -1, /* null/misaligned pointer, bad size, T > max_tokens, ... */
    ZEDA_ERR_UNSUPPORTED = -2, /* a shape the kernels do not cover (see zeda_moe_config_t) */
    ZEDA_ERR_WORKSPACE = -3,   /* workspace smaller than zeda_moe_workspace_bytes() */
    ZEDA_ERR_CUDA = -4,        /* a CUDA runtime call failed; text in zeda_last_error() */
    ZEDA_ERR_TIMEOUT = -5      /* a bounded device-side wait expired or a device-side check failed (reported
                                  by a later call) */
} zeda_status_t;

/* How the routing weight g~ of a selected slot is formed from p = softmax(logits over N+N_Z).
 * The paper says "normalized routing weight" (Section 2.1) without giving the formula. */
typedef enum {
    ZEDA_GATE_TOPK_NORM = 0,   /* p_i / sum of p over the K selected slots (zero slots included
                                  in the sum); default */
    ZEDA_GATE_SOFTMAX_RAW = 1, /* p_i itself */
    ZEDA_GATE_RENORM_REAL = 2  /* Eq. 7: p_i / sum of p over the selected NORMAL experts; zero
                                  slots get weight 0 */
} zeda_gate_mode_t;

/* What an injected expert outputs. */
typedef enum {
    ZEDA_EXPERT_ZERO = 0, /* Z_j(h) = 0 (Section 2.1) */
    ZEDA_EXPERT_COPY = 1  /* copy expert of Appendix B: adds (sum of zero-slot weights) * h */
} zeda_expert_kind_t;

/* Supported shapes: d_model and d_expert multiples of 64 in [64, 8192], 1 <= top_k <= 16,
 * n_real >= 1, n_zero >= 0, n_real + n_zero <= 512, top_k <= n_real + n_zero,
 * max_tokens >= 1 and max_tokens * top_k < 2^27. */
typedef struct {
    int32_t d_model;     /* H: hidden size */
    int32_t d_expert;    /* H_e: expert intermediate size */
    int32_t n_real;      /* N: normal experts */
    int32_t n_zero;      /* N_Z: zero experts (0 = the static top-K layer) */
    int32_t top_k;       /* K */
    int32_t max_tokens;  /* largest T any call will pass */
    int32_t gate_mode;   /* zeda_gate_mode_t */
    int32_t expert_kind; /* zeda_expert_kind_t */
    int32_t device;      /* CUDA device ordinal */
    int32_t flags;       /* ZEDA_FLAG_* */
    /* Expert parallelism (zeda_ep_* calls below).  ep_size = 0: a plain handle that holds all N
     * experts.  ep_size = G >= 1: this handle is rank ep_rank of a group of G; it routes over all
     * N + N_Z candidates but holds only the weights of experts [ep_rank * N/G, (ep_rank+1) * N/G)
     * (N must be a multiple of G, G <= 64) and can take in up to max_recv_pairs pair rows per call. */
    int32_t ep_size;
    int32_t ep_rank;
    int32_t max_recv_pairs;
} zeda_moe_config_t;

enum {
    ZEDA_FLAG_NONE = 0,
    ZEDA_FLAG_NO_DEPENDENT_LAUNCH = 4   /* launch every kernel fully stream-ordered (no programmatic
                                           dependent launch between the kernels of a call); any
                                           other bit is rejected */
};

/* Device workspace the handle needs for the given configuration (bytes, multiple of 256);
 * 0 if the configuration is invalid. */
size_t zeda_moe_workspace_bytes(const zeda_moe_config_t *cfg);

/* Builds a handle.  Section 2.1: the router has N + N_Z rows.
 *   router_w     dev [N+N_Z, d_model] fp32, rows 0..N-1 normal, N.. zero experts
 *   router_bias  dev [N+N_Z] fp32 added to the logits, or NULL (the paper's layer has none)
 *   w_gate_up    dev [N, 2*d_expert, d_model] bf16; per expert rows 0..H_e-1 = gate, H_e.. = up
 *   w_down       dev [N, d_model, d_expert] bf16
 *   workspace    dev, >= zeda_moe_workspace_bytes(cfg), 256-byte aligned; the library carves it
 * Makes the configured device current, may launch a one-time set-up kernel on the default stream
 * and synchronises before returning. */
zeda_status_t zeda_moe_create(const zeda_moe_config_t *cfg, const float *router_w,
                              const float *router_bias, const void *w_gate_up, const void *w_down,
                              void *workspace, size_t workspace_bytes, zeda_moe_t **out);

/* Routing only (Section 2.1: top-K over E'; zero slots dropped; surviving pairs grouped by expert).
 *   x               dev [T, d_model] bf16
 *   topk_idx        dev [T, K] int32: candidates in descending logit order, ties to the lower id
 *   topk_w          dev [T, K] fp32 routing weights per gate_mode
 *   expert_counts   dev [N] int32 pairs per normal expert
 *   expert_offsets  dev [N+1] int32 exclusive prefix sum; [N] = P
 *   perm            dev [T*K] int32; the first P entries list the surviving slots t*K+k ordered by
 *                   (expert ascending, token ascending); the rest is left untouched
 *   n_pairs         dev [1] int32 = P
 * Any output pointer may be NULL.  T == 0 returns ZEDA_OK and touches nothing. */
zeda_status_t zeda_route(zeda_moe_t *h, const void *x, int32_t T, int32_t *topk_idx, float *topk_w,
                         int32_t *expert_counts, int32_t *expert_offsets, int32_t *perm,
                         int32_t *n_pairs, void *stream);

/* Test entry: as zeda_route, but the top-K is taken over caller-supplied fp32 logits
 * dev [T, N+N_Z] instead of x * router_w^T + bias. */
zeda_status_t zeda_route_from_logits(zeda_moe_t *h, const float *logits, int32_t T,
                                     int32_t *topk_idx, float *topk_w, int32_t *expert_counts,
                                     int32_t *expert_offsets, int32_t *perm, int32_t *n_pairs,
                                     void *stream);

/* Test entry: the fp32 router logits x * router_w^T + bias, dev [T, N+N_Z].  zeda_route and
 * zeda_moe_forward compute the same sums, for mid-sized batches (256 <= T, up to a few thousand
 * tokens) in two or four slices of the reduction axis that are added afterwards: their logits can
 * differ from these in the last bits (fp32 addition order), never in the exact products. */
zeda_status_t zeda_router_logits(zeda_moe_t *h, const void *x, int32_t T, float *logits, void *stream);

/* Layer forward, Eq. 1 (Eq. 7 / Appendix B through the configured modes).
 *   x  dev [T, d_model] bf16      y  dev [T, d_model] bf16, fully overwritten
 * A token whose K slots all fall on zero experts gets exact +0 in every element of its row.
 * x and y must not overlap.  T == 0 returns ZEDA_OK and touches nothing. */
zeda_status_t zeda_moe_forward(zeda_moe_t *h, const void *x, int32_t T, void *y, void *stream);

/* The same forward for callers whose activations live in HOST memory: copies x to the device,
 * runs the layer, copies y back, and returns once y_host is complete (it synchronises `stream`).
 *   x_host  host [T, d_model] bf16     y_host  host [T, d_model] bf16
 * Pinned host memory makes the copies asynchronous; pageable memory works but is slower.
 * Batches of 4096 tokens or more are processed as two chunks (the layer is per token): the device
 * work of both stays on `stream`, the copies run on two streams that the handle creates on first use
 * (host objects; no device memory), so the second chunk is copied in while the first is computed and
 * the first is copied back while the second is computed.  The result is, bit for bit, that of
 * zeda_moe_forward on the two chunks (the first (T/2 rounded up to a multiple of 256) tokens, then the
 * rest); against one call on the whole batch the routing weights can differ in their last bits,
 * because the router slices its reduction axis by batch size.  Afterwards the routing kept in the
 * handle (statistics, counters) is that of the second chunk, except the launch count, which covers
 * both. */
zeda_status_t zeda_moe_forward_host(zeda_moe_t *h, const void *x_host, int32_t T, void *y_host,
                                    void *stream);

/* Glue between stacked layers (the paper's models stack 48 such MoE layers, Section 4.2; the
 * paper defines nothing between them, this is the layer-stack workload's device): in one pass
 *   r <- bf16(r + y)                         residual stream, updated in place (y NULL: r is kept)
 *   h  = r / sqrt(mean(r^2) + eps)           gain-free RMS normalisation, fp32 math, bf16 out
 *   r  dev [T, d_model] bf16 (in/out)   y  dev [T, d_model] bf16 or NULL   h  dev [T, d_model] bf16
 * Runs on the current device; needs no handle.  d_model: multiple of 64 in [64, 8192] (else
 * ZEDA_ERR_UNSUPPORTED); pointers 16-byte aligned; h must not overlap r or y.  T = 0 touches nothing. */
zeda_status_t zeda_residual_rmsnorm(void *r, const void *y, void *h, int32_t T, int32_t d_model, float eps,
                                    void *stream);

/* One layer of a stack with the glue fused into its last pass (same layer as zeda_moe_forward, Eq. 1;
 * same glue as zeda_residual_rmsnorm): the layer output y~ is not stored, instead
 *   r      <- bf16(r + bf16(y~(x)))          residual stream, updated in place
 *   h_next  = r / sqrt(mean(r^2) + eps)      the next layer's input
 * The results are, bit for bit, those of zeda_moe_forward(h, x, T, y) followed by
 * zeda_residual_rmsnorm(r, y, h_next, T, d_model, eps): one launch and one round trip of y through
 * device memory fewer per layer.
 *   x  dev [T, d_model] bf16 (this layer's input)   r  dev [T, d_model] bf16 (in/out)
 *   h_next  dev [T, d_model] bf16 (out)
 * x, r and h_next must not overlap one another (ZEDA_ERR_INVALID_ARG).  d_model <= 2048 (a token's
 * row is held by one thread block), otherwise ZEDA_ERR_UNSUPPORTED: use the two calls.  Other
 * arguments, errors and the routing kept in the handle as for zeda_moe_forward. */
zeda_status_t zeda_moe_forward_residual(zeda_moe_t *h, const void *x, int32_t T, void *r, void *h_next, float eps,
                                        void *stream);

/* Routing statistics of the most recent zeda_route / zeda_moe_forward call on this handle
 * (Section 2.2, Eq. 4-6), computed on the device from that call's routing:
 *   f      dev [N+N_Z] fp32  share of tokens whose top-K set holds candidate i (f_i), or NULL
 *   p_mean dev [N+N_Z] fp32  mean softmax probability of candidate i over the batch (P_i), or NULL
 *   out    dev [4] fp32      {r_ZE, sum_i f_i P_i, f_E P_E, f_Z P_Z}; the caller scales these into
 *                            L_A and L_GA with its alpha and w
 * Needs the logits, so it re-runs the router on x. */
zeda_status_t zeda_moe_stats(zeda_moe_t *h, const void *x, int32_t T, float *f, float *p_mean,
                             float *out, void *stream);

/* Per-token zero-expert ratio of the most recent routing on this handle (zeda_route, zeda_moe_forward,
 * zeda_moe_stats or zeda_ep_dispatch): r_ze[t] = (slots of token t that selected a zero expert) / K
 * (Section 2.2 defines r_ZE; Section 4.1 studies how it varies from token to token).
 *   T     must be the token count of that routing call      r_ze  dev [T] fp32
 * Reads the routing kept in the workspace; computes nothing else. */
zeda_status_t zeda_moe_token_zero_share(zeda_moe_t *h, int32_t T, float *r_ze, void *stream);

/* Counters of the last forward call, read back after synchronising the stream (blocking):
 * out[0] = P (surviving pairs), out[1] = U (normal experts with at least one pair),
 * out[2] = zero-expert slots, out[3] = kernels launched by that call. */
zeda_status_t zeda_moe_last_counters(zeda_moe_t *h, int64_t out[4], void *stream);

/* Per-stage device timing for measurement.  With profiling enabled, every later forward call
 * records CUDA events on its stream between the stages; zeda_moe_stage_ms synchronises on the
 * events of the last forward call (blocking) and returns the elapsed milliseconds of
 * {router logits, top-K + counting sort, expert GEMM1 + SwiGLU, expert GEMM2, combine}.
 * Enabling creates host-side event objects only (no device memory). */
enum { ZEDA_STAGE_ROUTER = 0, ZEDA_STAGE_SORT = 1, ZEDA_STAGE_GEMM1 = 2, ZEDA_STAGE_GEMM2 = 3,
       ZEDA_STAGE_COMBINE = 4, ZEDA_STAGE_COUNT = 5 };
zeda_status_t zeda_moe_set_profiling(zeda_moe_t *h, int32_t enable);
zeda_status_t zeda_moe_stage_ms(zeda_moe_t *h, float ms[ZEDA_STAGE_COUNT]);

/* Compaction and counting sort without any device allocation.  (The paper has no counterpart of
 * this entry point; it exists for the callers described here.)
 *
 * Everything else in this library works out of a workspace that the caller allocates.  Some
 * callers cannot allocate device memory at all: code running inside a region where the CUDA
 * allocator must not be called (for example between other libraries' captured or timed sections),
 * plug-ins that are handed device buffers by a host framework but have no allocator of their own,
 * or processes whose memory budget is fixed before they start.  For them this call performs the
 * same stable counting sort as zeda_route (drop the slots that chose a zero expert, count the
 * surviving pairs per normal expert, exclusive offsets, permutation ordered by expert then token)
 * on top-K indices the caller already has, and keeps its scratch in a fixed array inside the
 * library instead of a workspace.
 *   topk_idx        dev [T, top_k] int32 candidate ids (input); ids >= n_real are zero experts and
 *                   are dropped, and so is any id < 0 (a padding slot)
 *   expert_counts   dev [n_real] int32          expert_offsets  dev [n_real + 1] int32
 *   perm            dev [T * top_k] int32, first P entries written      n_pairs  dev [1] int32
 * All pointers are required and belong to the CURRENT device.  Limits: T <= ZEDA_STATIC_MAX_TOKENS
 * and T * top_k <= ZEDA_STATIC_MAX_SLOTS, n_real <= 512, top_k <= 16; larger sizes are rejected
 * with ZEDA_ERR_UNSUPPORTED and nothing is launched.  T == 0 returns ZEDA_OK and touches nothing.
 * The scratch array (about a third of a megabyte) is part of the library image: every GPU that loads the library
 * holds it until the process exits.  The call makes no cudaMalloc / cudaFree and uses no
 * allocating library routine; it enqueues a small memset and three kernels on `stream`.
 * The first call on each device looks up the array's device address (one cudaGetSymbolAddress,
 * with that device current); make that first call before any stream capture begins: a first call
 * on a stream that is being captured is refused with ZEDA_ERR_INVALID_ARG and launches nothing.
 * Host threads may make their first calls concurrently (the cached address is an atomic).
 * All calls on a device share the one array, which keeps the previous call's contents: the call
 * clears the words that must start at zero itself, but two calls whose work overlaps on the GPU
 * (different streams, or threads) race on it.  Serialise them on one stream. */
#define ZEDA_STATIC_MAX_TOKENS 4096
#define ZEDA_STATIC_MAX_SLOTS 32768
zeda_status_t zeda_compact_static(const int32_t *topk_idx, int32_t T, int32_t top_k, int32_t n_real,
                                  int32_t *expert_counts, int32_t *expert_offsets, int32_t *perm,
                                  int32_t *n_pairs, void *stream);

/* Expert-parallel forward: the experts are partitioned over G ranks (one handle each), the tokens
 * stay data-parallel.  Zero-expert slots are dropped BEFORE anything is exchanged, so they cost no
 * link bytes either (the paper's Appendix A, limitations, points at expert-parallel dispatch in the
 * DeepEP style as future work; the arithmetic is still Eq. 1).  The library does the device work
 * of one rank; the caller moves the rows between ranks (an all-to-all with per-rank row counts,
 * NCCL or any other transport) between the three calls:
 *
 *   zeda_ep_dispatch  routes this rank's T tokens (as zeda_route; the routing stays in the handle
 *                     for the combine) and packs the x rows of the surviving pairs, in the order
 *                     (expert ascending, token ascending), into send_rows.  Experts are owned in
 *                     contiguous blocks, so the rows for rank r are the contiguous range that
 *                     follows the rows for ranks < r.
 *       x             dev [T, d_model] bf16
 *       send_rows     dev [T*K, d_model] bf16, first P rows written
 *       send_counts   dev [G] int32: rows for each destination rank (sum = P)
 *       expert_counts dev [N] int32: pairs per expert; rank r needs entries [r*N/G, (r+1)*N/G)
 *   (exchange: every rank sends block r of send_rows and of expert_counts to rank r)
 *   zeda_ep_experts   runs this rank's experts on the rows received from the group.
 *       recv_rows     dev [n_rows, d_model] bf16: the blocks received from source ranks 0..G-1 in
 *                     that order, each in its sender's (expert, token) order
 *       recv_counts   dev [G, N/G] int32: recv_counts[s][j] = rows from source s for local expert j
 *       n_rows        sum of recv_counts (host value, <= max_recv_pairs); a mismatch with the
 *                     device-side sum is recorded like an expired wait (ZEDA_ERR_TIMEOUT later)
 *       out_rows      dev [n_rows, d_model] bf16: E_i(row), in the order of recv_rows
 *   (exchange back: block s of out_rows returns to rank s)
 *   zeda_ep_combine   Eq. 1 on the returned rows, which are in the order of send_rows.
 *       x             the same activations as in zeda_ep_dispatch (read by copy experts only)
 *       back_rows     dev [P, d_model] bf16        y  dev [T, d_model] bf16
 * All three only enqueue kernels on `stream`.  A handle with ep_size >= 1 serves these calls, the
 * routing calls and zeda_moe_stats, not zeda_moe_forward (its pair buffers are sized by
 * max_recv_pairs); with G = 1 the three calls in a row, without an exchange, are the plain layer. */
zeda_status_t zeda_ep_dispatch(zeda_moe_t *h, const void *x, int32_t T, void *send_rows,
                               int32_t *send_counts, int32_t *expert_counts, void *stream);
zeda_status_t zeda_ep_experts(zeda_moe_t *h, const void *recv_rows, const int32_t *recv_counts,
                              int32_t n_rows, void *out_rows, void *stream);
zeda_status_t zeda_ep_combine(zeda_moe_t *h, const void *x, const void *back_rows, int32_t T, void *y,
                              void *stream);

/* Failure reporting.  Every device-side wait in the tensor-core kernels is bounded; a wait that
 * expires makes its CTA record an error word in the workspace, skip its remaining work and leave
 * normally (the context stays usable, the call's outputs are undefined).  The word is sticky:
 * zeda_moe_last_counters and zeda_moe_destroy report ZEDA_ERR_TIMEOUT until it is cleared.
 *   zeda_moe_selftest_wait  exercises that path without a fault: a one-thread kernel waits, for at
 *                           most limit_us microseconds (1..100000), on a barrier that nothing signals,
 *                           and records the expiry like the kernels do.  Asynchronous on the stream.
 *   zeda_moe_clear_error    resets the error word (stream-ordered). */
zeda_status_t zeda_moe_selftest_wait(zeda_moe_t *h, int32_t limit_us, void *stream);
zeda_status_t zeda_moe_clear_error(zeda_moe_t *h, void *stream);

/* Reports a pending device-side error word (ZEDA_ERR_TIMEOUT) if any, then releases the handle.
 * Does not touch caller-owned device memory. */
zeda_status_t zeda_moe_destroy(zeda_moe_t *h);

/* Text of the last failure on the calling thread ("" if none). Never NULL. */
const char *zeda_last_error(void);

/* Library version string. */
const char *zeda_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ZEDA_H_ */
