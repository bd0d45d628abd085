// Host side of the C ABI: argument checks, workspace carving, stream-ordered launches.
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "zeda_internal.h"

namespace zeda {

static thread_local char g_err[512] = "";

void set_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof g_err, fmt, ap);
    va_end(ap);
}

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

bool config_ok(const zeda_moe_config_t *c, const char **why) {
    const char *w = nullptr;
    if (!c) w = "config is NULL";
    else if (c->d_model < 64 || c->d_model % 64 || c->d_model > 8192) w = "d_model must be a multiple of 64 in [64, 8192]";
    else if (c->d_expert < 64 || c->d_expert % 64 || c->d_expert > 8192) w = "d_expert must be a multiple of 64 in [64, 8192]";
    else if (c->n_real < 1) w = "n_real must be >= 1";
    else if (c->n_zero < 0) w = "n_zero must be >= 0";
    else if (c->n_real + c->n_zero > kMaxCand) w = "n_real + n_zero must be <= 512";
    else if (c->top_k < 1 || c->top_k > kMaxTopK) w = "top_k must be in [1, 16]";
    else if (c->top_k > c->n_real + c->n_zero) w = "top_k exceeds the number of candidates";
    else if (c->max_tokens < 1) w = "max_tokens must be >= 1";
    else if ((long long)c->max_tokens * c->top_k >= (1LL << 27)) w = "max_tokens * top_k must be < 2^27";
    else if (c->gate_mode < 0 || c->gate_mode > 2) w = "unknown gate_mode";
    else if (c->expert_kind < 0 || c->expert_kind > 1) w = "unknown expert_kind";
    else if (c->flags & ~ZEDA_FLAG_NO_DEPENDENT_LAUNCH) w = "unknown flag";
    else if (c->ep_size < 0 || c->ep_size > kMaxEpRanks) w = "ep_size must be in [0, 64]";
    else if (c->ep_size >= 1 && (c->n_real % c->ep_size) != 0) w = "n_real must be a multiple of ep_size";
    else if (c->ep_size >= 1 && (c->ep_rank < 0 || c->ep_rank >= c->ep_size)) w = "ep_rank outside [0, ep_size)";
    else if (c->ep_size >= 1 && (c->max_recv_pairs < 1 || c->max_recv_pairs >= (1 << 27))) w = "max_recv_pairs must be in [1, 2^27)";
    if (why) *why = w;
    return w == nullptr;
}

size_t hist_bytes(const zeda_moe_config_t &c) {
    return (size_t)((c.max_tokens + kSortTokens - 1) / kSortTokens) * c.n_real * sizeof(int32_t);
}

// Walks the workspace layout; with base == nullptr it only measures.
size_t carve(const zeda_moe_config_t &c, unsigned char *base, Workspace *ws, int *max_tiles) {
    size_t off = 0;
    auto take = [&](size_t bytes) -> void * {
        void *p = base ? base + off : nullptr;
        off = align_up(off + bytes, 256);
        return p;
    };
    const size_t slots = (size_t)c.max_tokens * c.top_k;
    const size_t n_cand = (size_t)c.n_real + c.n_zero;
    const size_t nblk = (c.max_tokens + kSortTokens - 1) / kSortTokens;
    const size_t tiles = slots / kMidTileM + c.n_real + 1;
    // an expert-parallel handle holds n_local experts and sizes its pair buffers for the rows it may receive
    const bool ep = c.ep_size >= 1;
    const size_t n_local = ep ? (size_t)c.n_real / c.ep_size : (size_t)c.n_real;
    const size_t pair_rows = ep ? (size_t)c.max_recv_pairs : slots;
    const size_t ep_tiles = pair_rows / kPairTileM + n_local + 1;
    const size_t nblk_stats = (c.max_tokens + 63) / 64;
    Workspace w;
    w.topk_idx = (int32_t *)take(slots * 4);
    w.topk_w = (float *)take(slots * 4);
    w.inv = (int32_t *)take(slots * 4);
    w.perm = (int32_t *)take(slots * 4);
    w.pair_token = (int32_t *)take(slots * 4);
    w.block_hist = (int32_t *)take(hist_bytes(c));
    w.counts = (int32_t *)take((size_t)c.n_real * 4);
    w.offsets = (int32_t *)take((size_t)(c.n_real + 1) * 4);
    w.meta = (int32_t *)take(kMetaCount * 4);
    w.ptile_expert = (int32_t *)take(tiles * 4);
    w.ptile_row0 = (int32_t *)take(tiles * 4);
    w.logits = (float *)take((size_t)router_part_rows(c.max_tokens) * n_cand * 4);
    w.stat_part = (float *)take(nblk_stats * 2 * n_cand * 4);
    // pair buffers carry one tile of slack rows so that a full tile may be read past the last pair
    w.hmid = (__nv_bfloat16 *)take((pair_rows + kPairTileM) * c.d_expert * 2);
    w.obuf = (__nv_bfloat16 *)take((pair_rows + kPairTileM) * c.d_model * 2);
    w.router_split = (__nv_bfloat16 *)take((size_t)3 * router_split_pad((int)n_cand) * c.d_model * 2);
    w.x_stage = (__nv_bfloat16 *)take((size_t)c.max_tokens * c.d_model * 2);
    w.y_stage = (__nv_bfloat16 *)take((size_t)c.max_tokens * c.d_model * 2);
    w.ep_counts = w.ep_offsets = w.ep_pair_row = w.ep_row_pos = w.ep_tile_expert = w.ep_tile_row0 = nullptr;
    if (ep) {
        w.ep_counts = (int32_t *)take(n_local * 4);
        w.ep_offsets = (int32_t *)take((n_local + 1) * 4);
        w.ep_pair_row = (int32_t *)take(pair_rows * 4);
        w.ep_row_pos = (int32_t *)take(pair_rows * 4);
        w.ep_tile_expert = (int32_t *)take(ep_tiles * 4);
        w.ep_tile_row0 = (int32_t *)take(ep_tiles * 4);
    }
    if (ws) *ws = w;
    if (max_tiles) *max_tiles = (int)tiles;
    return off;
}

// text for the sticky device-side error word
const char kDeviceFailure[] = "a bounded device wait expired or a device-side check failed (code %d; 21 = the row count "
                              "passed to zeda_ep_experts is not the sum of its count matrix)";

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

thread_local cudaError_t t_launch_error = cudaSuccess;

zeda_status_t cuda_fail(const char *what, cudaError_t e) {
    if (e == cudaSuccess) e = t_launch_error;  // a launch that failed earlier in this call
    t_launch_error = cudaSuccess;
    set_error("%s: %s", what, cudaGetErrorString(e));
    return ZEDA_ERR_CUDA;
}

zeda_status_t check_call(zeda_moe_t *h, const void *in, int32_t T, const char *in_name) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (T < 0 || T > h->cfg.max_tokens) { set_error("T=%d outside [0, max_tokens=%d]", T, h->cfg.max_tokens); return ZEDA_ERR_INVALID_ARG; }
    if (T > 0 && !in) { set_error("%s is NULL", in_name); return ZEDA_ERR_INVALID_ARG; }
    if (T > 0 && !aligned16(in)) { set_error("%s is not 16-byte aligned", in_name); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    return ZEDA_OK;
}

// Routing into the workspace (+ optional user copies); returns launches or <0.
// full_logits: the caller reads ws.logits afterwards, so the router may not leave them in slices.
int route_into(zeda_moe_t *h, const __nv_bfloat16 *x, const float *logits_in, int T, const RouteOut &out, cudaStream_t s,
               bool full_logits = false) {
    int n = 0, n_parts = 1;
    h->last_routed_tokens = T;
    const float *logits = logits_in;
    if (!logits) {
        int r = launch_router_logits(h, x, T, h->ws.logits, s, full_logits ? nullptr : &n_parts);
        if (r < 0) return r;
        n += r;
        logits = h->ws.logits;
    }
    int r = launch_route_from_logits(h, logits, T, out, s, n_parts);
    if (r < 0) return r;
    return n + r;
}

// With resid given, the call ends in the fused combine + glue pass: resid <- bf16(resid + y) and
// the normalised residual goes where y would have gone.
zeda_status_t forward_device(zeda_moe_t *h, const __nv_bfloat16 *x, int T, __nv_bfloat16 *y, cudaStream_t s,
                             __nv_bfloat16 *resid = nullptr, float eps = 0.f) {
    const bool prof = h->profiling;
    auto mark = [&](int i) { if (prof) cudaEventRecord(h->ev[i], s); };
    mark(0);
    h->last_routed_tokens = T;
    int n_parts = 1;
    int n = launch_router_logits(h, x, T, h->ws.logits, s, &n_parts);
    if (n < 0) return cuda_fail("router launch", cudaGetLastError());
    mark(1);
    RouteOut none = {};
    int r = launch_route_from_logits(h, h->ws.logits, T, none, s, n_parts);
    if (r < 0) return cuda_fail("routing launch", cudaGetLastError());
    n += r;
    mark(2);
    const Workspace &ws = h->ws;
    const ExpertWork work = {ws.counts, ws.offsets, ws.ptile_expert, ws.ptile_row0, ws.pair_token, T * h->cfg.top_k, tile_rows_for(h, T)};
    r = launch_experts_gemm1_pair(h, x, work, s);
    if (r < 0) return cuda_fail("expert GEMM1 launch", cudaGetLastError());
    n += r;
    mark(3);
    r = launch_experts_gemm2_pair(h, work, s);
    if (r < 0) return cuda_fail("expert GEMM2 launch", cudaGetLastError());
    n += r;
    mark(4);
    r = resid ? launch_combine_glue(h, x, T, resid, y, eps, s) : launch_combine(h, x, T, y, s);
    if (r < 0) return cuda_fail("combine launch", cudaGetLastError());
    mark(5);
    h->profiled_last = prof;
    h->last_launches = n + r;
    return ZEDA_OK;
}

}  // namespace

void note_launch_error(cudaError_t e) {
    if (t_launch_error == cudaSuccess) t_launch_error = e;
}

}  // namespace zeda

using namespace zeda;

extern "C" {

size_t zeda_moe_workspace_bytes(const zeda_moe_config_t *cfg) {
    const char *why = nullptr;
    if (!config_ok(cfg, &why)) { set_error("%s", why); return 0; }
    return carve(*cfg, nullptr, nullptr, nullptr);
}

zeda_status_t zeda_moe_create(const zeda_moe_config_t *cfg, const float *router_w, const float *router_bias,
                              const void *w_gate_up, const void *w_down, void *workspace, size_t workspace_bytes,
                              zeda_moe_t **out) {
    if (out) *out = nullptr;
    const char *why = nullptr;
    if (!config_ok(cfg, &why)) {
        set_error("%s", why);
        const bool shape = cfg && why && (strstr(why, "multiple of 64") || strstr(why, "<= 512") || strstr(why, "[1, 16]"));
        return shape ? ZEDA_ERR_UNSUPPORTED : ZEDA_ERR_INVALID_ARG;
    }
    if (!out) { set_error("out is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (!router_w || !w_gate_up || !w_down || !workspace) { set_error("a required pointer is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (!aligned16(router_w) || !aligned16(w_gate_up) || !aligned16(w_down) || (router_bias && (reinterpret_cast<uintptr_t>(router_bias) & 3u))) {
        set_error("weights must be 16-byte aligned");
        return ZEDA_ERR_INVALID_ARG;
    }
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) { set_error("workspace must be 256-byte aligned"); return ZEDA_ERR_INVALID_ARG; }
    const size_t need = carve(*cfg, nullptr, nullptr, nullptr);
    if (workspace_bytes < need) { set_error("workspace has %zu bytes, %zu needed", workspace_bytes, need); return ZEDA_ERR_WORKSPACE; }
    int ndev = 0;
    cudaError_t e = cudaGetDeviceCount(&ndev);
    if (e != cudaSuccess) return cuda_fail("cudaGetDeviceCount", e);
    if (cfg->device < 0 || cfg->device >= ndev) { set_error("device %d not present (%d devices)", cfg->device, ndev); return ZEDA_ERR_INVALID_ARG; }
    e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, cfg->device);
    if (e != cudaSuccess) return cuda_fail("cudaGetDeviceProperties", e);
    if (prop.major != 10) { set_error("this library is built for sm_100a only; device is sm_%d%d", prop.major, prop.minor); return ZEDA_ERR_UNSUPPORTED; }

    zeda_moe *h = new (std::nothrow) zeda_moe();
    if (!h) { set_error("out of host memory"); return ZEDA_ERR_INVALID_ARG; }
    h->cfg = *cfg;
    h->router_w = router_w;
    h->router_bias = router_bias;
    h->w_gate_up = static_cast<const __nv_bfloat16 *>(w_gate_up);
    h->w_down = static_cast<const __nv_bfloat16 *>(w_down);
    h->sm_count = prop.multiProcessorCount;
    h->pdl = !(cfg->flags & ZEDA_FLAG_NO_DEPENDENT_LAUNCH);
    h->last_launches = 0;
    h->last_routed_tokens = 0;
    h->n_local = cfg->ep_size >= 1 ? cfg->n_real / cfg->ep_size : cfg->n_real;
    h->pair_rows = cfg->ep_size >= 1 ? cfg->max_recv_pairs : cfg->max_tokens * cfg->top_k;
    h->pmaps = nullptr;
    h->router_maps = nullptr;
    h->profiling = false;
    h->profiled_last = false;
    for (auto &ev : h->ev) ev = nullptr;
    h->copy_in = h->copy_out = nullptr;
    for (auto &ev : h->ev_host) ev = nullptr;
    carve(*cfg, static_cast<unsigned char *>(workspace), &h->ws, &h->max_tiles);
    if (init_route_kernels(h) < 0) { delete h; return cuda_fail("kernel set-up", cudaGetLastError()); }
    if (init_pair_kernels(h) < 0) { delete h; return ZEDA_ERR_CUDA; }
    if (init_router_tile(h) < 0) {
        if (h->pmaps) free(h->pmaps);
        delete h;
        return cuda_fail("router set-up", cudaGetLastError());
    }
    e = cudaMemset(h->ws.meta, 0, kMetaCount * 4);
    if (e != cudaSuccess) { delete h; return cuda_fail("cudaMemset(meta)", e); }
    // the block histograms of the counting sort are zero between calls (the top-K kernel adds into them,
    // the placement kernel clears them)
    e = cudaMemset(h->ws.block_hist, 0, hist_bytes(*cfg));
    if (e != cudaSuccess) { delete h; return cuda_fail("cudaMemset(block_hist)", e); }
    e = cudaDeviceSynchronize();
    if (e != cudaSuccess) { delete h; return cuda_fail("cudaDeviceSynchronize", e); }
    *out = h;
    return ZEDA_OK;
}

zeda_status_t zeda_route(zeda_moe_t *h, const void *x, int32_t T, int32_t *topk_idx, float *topk_w,
                         int32_t *expert_counts, int32_t *expert_offsets, int32_t *perm, int32_t *n_pairs,
                         void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    RouteOut out = {topk_idx, topk_w, expert_counts, expert_offsets, perm, n_pairs};
    int n = route_into(h, static_cast<const __nv_bfloat16 *>(x), nullptr, T, out, static_cast<cudaStream_t>(stream));
    if (n < 0) return cuda_fail("routing launch", cudaGetLastError());
    h->last_launches = n;
    return ZEDA_OK;
}

zeda_status_t zeda_route_from_logits(zeda_moe_t *h, const float *logits, int32_t T, int32_t *topk_idx, float *topk_w,
                                     int32_t *expert_counts, int32_t *expert_offsets, int32_t *perm,
                                     int32_t *n_pairs, void *stream) {
    zeda_status_t st = check_call(h, logits, T, "logits");
    if (st != ZEDA_OK || T == 0) return st;
    RouteOut out = {topk_idx, topk_w, expert_counts, expert_offsets, perm, n_pairs};
    int n = route_into(h, nullptr, logits, T, out, static_cast<cudaStream_t>(stream));
    if (n < 0) return cuda_fail("routing launch", cudaGetLastError());
    h->last_launches = n;
    return ZEDA_OK;
}

zeda_status_t zeda_router_logits(zeda_moe_t *h, const void *x, int32_t T, float *logits, void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    if (!logits) { set_error("logits is NULL"); return ZEDA_ERR_INVALID_ARG; }
    int n = launch_router_logits(h, static_cast<const __nv_bfloat16 *>(x), T, logits, static_cast<cudaStream_t>(stream));
    if (n < 0) return cuda_fail("router launch", cudaGetLastError());
    h->last_launches = n;
    return ZEDA_OK;
}

zeda_status_t zeda_moe_forward(zeda_moe_t *h, const void *x, int32_t T, void *y, void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    if (h->cfg.ep_size >= 1) { set_error("an expert-parallel handle (ep_size >= 1) runs the layer through the zeda_ep_* calls"); return ZEDA_ERR_INVALID_ARG; }
    if (!y || !aligned16(y)) { set_error("y is NULL or not 16-byte aligned"); return ZEDA_ERR_INVALID_ARG; }
    const size_t bytes = (size_t)T * h->cfg.d_model * 2;
    const char *xb = static_cast<const char *>(x), *yb = static_cast<const char *>(y);
    if (xb < yb + bytes && yb < xb + bytes) { set_error("x and y overlap"); return ZEDA_ERR_INVALID_ARG; }
    return forward_device(h, static_cast<const __nv_bfloat16 *>(x), T, static_cast<__nv_bfloat16 *>(y),
                          static_cast<cudaStream_t>(stream));
}

zeda_status_t zeda_moe_forward_residual(zeda_moe_t *h, const void *x, int32_t T, void *r, void *h_next, float eps,
                                        void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    if (h->cfg.ep_size >= 1) { set_error("an expert-parallel handle (ep_size >= 1) runs the layer through the zeda_ep_* calls"); return ZEDA_ERR_INVALID_ARG; }
    if (!combine_glue_supported(h)) { set_error("the fused residual form needs d_model <= 2048"); return ZEDA_ERR_UNSUPPORTED; }
    if (!r || !h_next || !aligned16(r) || !aligned16(h_next)) { set_error("r or h_next is NULL or not 16-byte aligned"); return ZEDA_ERR_INVALID_ARG; }
    if (!(eps >= 0.f)) { set_error("eps must be >= 0"); return ZEDA_ERR_INVALID_ARG; }
    const size_t bytes = (size_t)T * h->cfg.d_model * 2;
    const char *b[3] = {static_cast<const char *>(x), static_cast<const char *>(r), static_cast<const char *>(h_next)};
    for (int i = 0; i < 3; ++i)
        for (int j = i + 1; j < 3; ++j)
            if (b[i] < b[j] + bytes && b[j] < b[i] + bytes) { set_error("x, r and h_next overlap"); return ZEDA_ERR_INVALID_ARG; }
    return forward_device(h, static_cast<const __nv_bfloat16 *>(x), T, static_cast<__nv_bfloat16 *>(h_next),
                          static_cast<cudaStream_t>(stream), static_cast<__nv_bfloat16 *>(r), eps);
}

// Batches of at least this many tokens go through the host-buffer entry point in two chunks, so that
// the copy of the second chunk runs under the layer of the first and the copy back of the first under
// the layer of the second.
static const int kHostSplitMinTokens = 4096;

zeda_status_t zeda_moe_forward_host(zeda_moe_t *h, const void *x_host, int32_t T, void *y_host, void *stream) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (T < 0 || T > h->cfg.max_tokens) { set_error("T=%d outside [0, max_tokens=%d]", T, h->cfg.max_tokens); return ZEDA_ERR_INVALID_ARG; }
    if (T == 0) return ZEDA_OK;
    if (h->cfg.ep_size >= 1) { set_error("an expert-parallel handle (ep_size >= 1) runs the layer through the zeda_ep_* calls"); return ZEDA_ERR_INVALID_ARG; }
    if (!x_host || !y_host) { set_error("host buffer is NULL"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t row = (size_t)h->cfg.d_model * 2;
    if (T < kHostSplitMinTokens) {
        e = cudaMemcpyAsync(h->ws.x_stage, x_host, T * row, cudaMemcpyHostToDevice, s);
        if (e != cudaSuccess) return cuda_fail("copy of x to the device", e);
        zeda_status_t st = forward_device(h, h->ws.x_stage, T, h->ws.y_stage, s);
        if (st != ZEDA_OK) return st;
        e = cudaMemcpyAsync(y_host, h->ws.y_stage, T * row, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_fail("copy of y to the host", e);
        e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
        return ZEDA_OK;
    }
    // Two chunks.  The layer is per token (Eq. 1), so the chunks are two independent calls; their device
    // work stays on `stream`, one after the other (they share the workspace), the copies run on two
    // streams of the handle.
    if (!h->copy_in) {
        e = cudaStreamCreateWithFlags(&h->copy_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&h->copy_out, cudaStreamNonBlocking);
        for (auto &ev : h->ev_host)
            if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail("stream / event creation", e);
    }
    const int T0 = (T / 2 + 255) / 256 * 256, T1 = T - T0;
    const char *xh = static_cast<const char *>(x_host);
    char *yh = static_cast<char *>(y_host);
    __nv_bfloat16 *xs = h->ws.x_stage, *ys = h->ws.y_stage;
    cudaEvent_t *ev = h->ev_host;  // 0 start, 1-2 chunk copied in, 3-4 chunk computed, 5 all copied out
    bool ok = cudaEventRecord(ev[0], s) == cudaSuccess && cudaStreamWaitEvent(h->copy_in, ev[0], 0) == cudaSuccess &&
              cudaStreamWaitEvent(h->copy_out, ev[0], 0) == cudaSuccess;
    ok = ok && cudaMemcpyAsync(xs, xh, T0 * row, cudaMemcpyHostToDevice, h->copy_in) == cudaSuccess &&
         cudaEventRecord(ev[1], h->copy_in) == cudaSuccess &&
         cudaMemcpyAsync(xs + (size_t)T0 * h->cfg.d_model, xh + T0 * row, T1 * row, cudaMemcpyHostToDevice, h->copy_in) == cudaSuccess &&
         cudaEventRecord(ev[2], h->copy_in) == cudaSuccess;
    if (!ok) return cuda_fail("copy of x to the device", cudaGetLastError());
    if (cudaStreamWaitEvent(s, ev[1], 0) != cudaSuccess) return cuda_fail("cudaStreamWaitEvent", cudaGetLastError());
    zeda_status_t st = forward_device(h, xs, T0, ys, s);
    if (st != ZEDA_OK) return st;
    if (cudaEventRecord(ev[3], s) != cudaSuccess || cudaStreamWaitEvent(s, ev[2], 0) != cudaSuccess)
        return cuda_fail("cudaEventRecord", cudaGetLastError());
    const int launches0 = h->last_launches;
    st = forward_device(h, xs + (size_t)T0 * h->cfg.d_model, T1, ys + (size_t)T0 * h->cfg.d_model, s);
    if (st != ZEDA_OK) return st;
    h->last_launches += launches0;
    ok = cudaEventRecord(ev[4], s) == cudaSuccess && cudaStreamWaitEvent(h->copy_out, ev[3], 0) == cudaSuccess &&
         cudaMemcpyAsync(yh, ys, T0 * row, cudaMemcpyDeviceToHost, h->copy_out) == cudaSuccess &&
         cudaStreamWaitEvent(h->copy_out, ev[4], 0) == cudaSuccess &&
         cudaMemcpyAsync(yh + T0 * row, ys + (size_t)T0 * h->cfg.d_model, T1 * row, cudaMemcpyDeviceToHost, h->copy_out) == cudaSuccess &&
         cudaEventRecord(ev[5], h->copy_out) == cudaSuccess;
    if (!ok) return cuda_fail("copy of y to the host", cudaGetLastError());
    e = cudaEventSynchronize(ev[5]);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
    return ZEDA_OK;
}

zeda_status_t zeda_ep_dispatch(zeda_moe_t *h, const void *x, int32_t T, void *send_rows, int32_t *send_counts,
                               int32_t *expert_counts, void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK) return st;
    if (h->cfg.ep_size < 1) { set_error("the handle was not created for expert parallelism (ep_size = 0)"); return ZEDA_ERR_INVALID_ARG; }
    if (!send_counts) { set_error("send_counts is NULL"); return ZEDA_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (T == 0) {  // nothing to route: this rank sends no rows
        cudaError_t e = cudaMemsetAsync(send_counts, 0, sizeof(int32_t) * h->cfg.ep_size, s);
        if (e == cudaSuccess && expert_counts) e = cudaMemsetAsync(expert_counts, 0, sizeof(int32_t) * h->cfg.n_real, s);
        if (e == cudaSuccess) e = cudaMemsetAsync(h->ws.meta + kMetaPairs, 0, sizeof(int32_t), s);
        return e == cudaSuccess ? ZEDA_OK : cuda_fail("cudaMemsetAsync", e);
    }
    if (!send_rows || !aligned16(send_rows)) { set_error("send_rows is NULL or not 16-byte aligned"); return ZEDA_ERR_INVALID_ARG; }
    RouteOut none = {};
    int n = route_into(h, static_cast<const __nv_bfloat16 *>(x), nullptr, T, none, s);
    if (n < 0) return cuda_fail("routing launch", cudaGetLastError());
    int r = launch_ep_pack(h, static_cast<const __nv_bfloat16 *>(x), T, static_cast<__nv_bfloat16 *>(send_rows), send_counts,
                           expert_counts, s);
    if (r < 0) return cuda_fail("pack launch", cudaGetLastError());
    h->last_launches = n + r;
    return ZEDA_OK;
}

zeda_status_t zeda_ep_experts(zeda_moe_t *h, const void *recv_rows, const int32_t *recv_counts, int32_t n_rows,
                              void *out_rows, void *stream) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (h->cfg.ep_size < 1) { set_error("the handle was not created for expert parallelism (ep_size = 0)"); return ZEDA_ERR_INVALID_ARG; }
    if (n_rows < 0 || n_rows > h->cfg.max_recv_pairs) {
        set_error("n_rows=%d outside [0, max_recv_pairs=%d]", n_rows, h->cfg.max_recv_pairs);
        return ZEDA_ERR_INVALID_ARG;
    }
    if (n_rows == 0) return ZEDA_OK;
    if (!recv_rows || !recv_counts || !out_rows || !aligned16(recv_rows) || !aligned16(out_rows)) {
        set_error("recv_rows, recv_counts and out_rows are required; rows 16-byte aligned");
        return ZEDA_ERR_INVALID_ARG;
    }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int n = launch_ep_plan(h, recv_counts, n_rows, s);
    if (n < 0) return cuda_fail("plan launch", cudaGetLastError());
    const Workspace &ws = h->ws;
    const ExpertWork work = {ws.ep_counts, ws.ep_offsets, ws.ep_tile_expert, ws.ep_tile_row0, ws.ep_pair_row, n_rows, kPairTileM};
    int r = launch_experts_gemm1_pair(h, static_cast<const __nv_bfloat16 *>(recv_rows), work, s);
    if (r < 0) return cuda_fail("expert GEMM1 launch", cudaGetLastError());
    n += r;
    r = launch_experts_gemm2_pair(h, work, s);
    if (r < 0) return cuda_fail("expert GEMM2 launch", cudaGetLastError());
    n += r;
    r = launch_ep_unsort(h, n_rows, static_cast<__nv_bfloat16 *>(out_rows), s);
    if (r < 0) return cuda_fail("unsort launch", cudaGetLastError());
    h->last_launches = n + r;
    return ZEDA_OK;
}

zeda_status_t zeda_ep_combine(zeda_moe_t *h, const void *x, const void *back_rows, int32_t T, void *y, void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    if (h->cfg.ep_size < 1) { set_error("the handle was not created for expert parallelism (ep_size = 0)"); return ZEDA_ERR_INVALID_ARG; }
    if (!y || !aligned16(y) || !back_rows || !aligned16(back_rows)) { set_error("back_rows and y are required, 16-byte aligned"); return ZEDA_ERR_INVALID_ARG; }
    int r = launch_combine_rows(h, static_cast<const __nv_bfloat16 *>(back_rows), static_cast<const __nv_bfloat16 *>(x), T,
                                static_cast<__nv_bfloat16 *>(y), static_cast<cudaStream_t>(stream));
    if (r < 0) return cuda_fail("combine launch", cudaGetLastError());
    h->last_launches = r;
    return ZEDA_OK;
}

zeda_status_t zeda_moe_stats(zeda_moe_t *h, const void *x, int32_t T, float *f, float *p_mean, float *out, void *stream) {
    zeda_status_t st = check_call(h, x, T, "x");
    if (st != ZEDA_OK || T == 0) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    RouteOut none = {};
    int n = route_into(h, static_cast<const __nv_bfloat16 *>(x), nullptr, T, none, s, true);
    if (n < 0) return cuda_fail("routing launch", cudaGetLastError());
    int r = launch_stats(h, h->ws.logits, h->ws.topk_idx, T, f, p_mean, out, s);
    if (r < 0) return cuda_fail("stats launch", cudaGetLastError());
    h->last_launches = n + r;
    return ZEDA_OK;
}

zeda_status_t zeda_moe_token_zero_share(zeda_moe_t *h, int32_t T, float *r_ze, void *stream) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (T == 0) return ZEDA_OK;
    if (T < 0 || T != h->last_routed_tokens) {
        set_error("T=%d is not the token count of the last routing pass on this handle (%d)", T, h->last_routed_tokens);
        return ZEDA_ERR_INVALID_ARG;
    }
    if (!r_ze) { set_error("r_ze is NULL"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    if (launch_token_zero_share(h, T, r_ze, static_cast<cudaStream_t>(stream)) < 0)
        return cuda_fail("token_zero_share launch", cudaGetLastError());
    return ZEDA_OK;
}

zeda_status_t zeda_moe_last_counters(zeda_moe_t *h, int64_t out[4], void *stream) {
    if (!h || !out) { set_error("NULL argument"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    int32_t meta[kMetaCount];
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    e = cudaMemcpyAsync(meta, h->ws.meta, sizeof meta, cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return cuda_fail("cudaMemcpyAsync(meta)", e);
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
    out[0] = meta[kMetaPairs];
    out[1] = meta[kMetaActive];
    out[2] = meta[kMetaZeroSlots];
    out[3] = h->last_launches;
    if (meta[kMetaError] != 0) { set_error(kDeviceFailure, meta[kMetaError]); return ZEDA_ERR_TIMEOUT; }
    return ZEDA_OK;
}

zeda_status_t zeda_moe_selftest_wait(zeda_moe_t *h, int32_t limit_us, void *stream) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    if (limit_us < 1 || limit_us > 100000) { set_error("limit_us must be in [1, 100000]"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    int khz = 0;
    e = cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaDeviceGetAttribute", e);
    const long long cycles = (long long)limit_us * (khz > 0 ? khz : 1000000) / 1000;
    if (launch_wait_selftest(h, cycles, static_cast<cudaStream_t>(stream)) < 0)
        return cuda_fail("self-test launch", cudaGetLastError());
    return ZEDA_OK;
}

zeda_status_t zeda_moe_clear_error(zeda_moe_t *h, void *stream) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    e = cudaMemsetAsync(h->ws.meta + kMetaError, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("cudaMemsetAsync", e);
    // a call that failed between its top-K and placement kernels leaves counts in the block histograms
    e = cudaMemsetAsync(h->ws.block_hist, 0, hist_bytes(h->cfg), static_cast<cudaStream_t>(stream));
    if (e == cudaSuccess) e = cudaMemsetAsync(h->ws.meta + kMetaHistTicket, 0, sizeof(int32_t), static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) return cuda_fail("cudaMemsetAsync", e);
    return ZEDA_OK;
}

zeda_status_t zeda_moe_set_profiling(zeda_moe_t *h, int32_t enable) {
    if (!h) { set_error("handle is NULL"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaSetDevice(h->cfg.device);
    if (e != cudaSuccess) return cuda_fail("cudaSetDevice", e);
    if (enable && !h->ev[0]) {
        for (auto &ev : h->ev) {
            e = cudaEventCreate(&ev);
            if (e != cudaSuccess) return cuda_fail("cudaEventCreate", e);
        }
    }
    h->profiling = enable != 0;
    if (!enable) h->profiled_last = false;
    return ZEDA_OK;
}

zeda_status_t zeda_moe_stage_ms(zeda_moe_t *h, float ms[ZEDA_STAGE_COUNT]) {
    if (!h || !ms) { set_error("NULL argument"); return ZEDA_ERR_INVALID_ARG; }
    if (!h->profiled_last) { set_error("the last forward call was not profiled"); return ZEDA_ERR_INVALID_ARG; }
    cudaError_t e = cudaEventSynchronize(h->ev[ZEDA_STAGE_COUNT]);
    if (e != cudaSuccess) return cuda_fail("cudaEventSynchronize", e);
    for (int i = 0; i < ZEDA_STAGE_COUNT; ++i) {
        e = cudaEventElapsedTime(&ms[i], h->ev[i], h->ev[i + 1]);
        if (e != cudaSuccess) return cuda_fail("cudaEventElapsedTime", e);
    }
    return ZEDA_OK;
}

zeda_status_t zeda_moe_destroy(zeda_moe_t *h) {
    if (!h) return ZEDA_OK;
    zeda_status_t st = ZEDA_OK;
    if (cudaSetDevice(h->cfg.device) == cudaSuccess) {
        int32_t err = 0;
        cudaError_t e = cudaDeviceSynchronize();
        if (e == cudaSuccess) e = cudaMemcpy(&err, h->ws.meta + kMetaError, 4, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) st = cuda_fail("zeda_moe_destroy", e);
        else if (err != 0) { set_error(kDeviceFailure, err); st = ZEDA_ERR_TIMEOUT; }
    }
    for (auto &ev : h->ev) if (ev) cudaEventDestroy(ev);
    for (auto &ev : h->ev_host) if (ev) cudaEventDestroy(ev);
    if (h->copy_in) cudaStreamDestroy(h->copy_in);
    if (h->copy_out) cudaStreamDestroy(h->copy_out);
    if (h->pmaps) free(h->pmaps);
    if (h->router_maps) free(h->router_maps);
    delete h;
    return st;
}

const char *zeda_last_error(void) { return g_err; }

const char *zeda_version(void) { return "zeda-moe 0.1 (sm_100a)"; }

}  // extern "C"
