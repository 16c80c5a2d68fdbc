// C ABI of libspice: argument checking, workspace ownership and kernel dispatch.
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "spice_internal.cuh"

using namespace spice;

struct spice_ctx {
    int device;
    spice_layer_cfg cfg;
    int32_t max_tokens;
    void *ws;          // one device allocation, carved below
    size_t ws_bytes;
    Tables tb;
    // call-private copies of routing results when the caller does not want them
    int32_t *ws_idx, *ws_slot, *ws_counts;
    float *ws_gate;
    uint8_t *ws_cls;
    float *y32;        // [Tm, d] fp32 accumulator of the fused call
    GroupScratch gsc;               // scratch of the multi-CTA classify / group kernels
    float *draft_logits;            // [Tm, N] logits of spice_draft_confidence when the caller does not want pi_hat
    // speculative prefetch rollout
    __nv_bfloat16 *roll_h, *roll_y; // [Tm, d] draft state and scratch output
    float *roll_conf;               // [Tm]
    int32_t *roll_active, *roll_active2;   // [Tm] each: "still speculates" flags, read / written alternately per depth
    // fused decode kernel
    float *logits;                  // [Td, N]
    __nv_bfloat16 *act_hit16, *act_shared16, *z16;
    int32_t *sync;
    int32_t sync_words;
    int32_t decode_tokens;          // largest T of the mma.sync decode kernel (0: path unavailable)
    int32_t dtc_tokens;             // largest T of the tcgen05 decode kernel (0: path unavailable)
    float *route_logits;            // [Tm, N] router logits of large batches (tensor-core router)
    cudaStream_t side;              // large batches: the shared expert runs here beside the routing chain (null: in line)
    cudaEvent_t ev_fork, ev_join, ev_grouped;
    float *part_split;              // [splits][Td, d] partial shared-expert outputs of the tcgen05 decode kernel
    uint8_t *x8_h, *act8_hit, *act8_sh;   // 8-bit weight precision: activations as three E5M2 planes
    int n_sms, max_smem_optin;
    TcBuffers tcb;                  // tensor-core path buffers (large batches)
    bool tc_ok;
    int64_t opt_path;               // 0 auto, 1 general kernels only, 2 no fused decode kernel, 3 mma.sync decode kernel
    int64_t opt_spin_limit;
    int64_t launches;
};

namespace {

// NVTX range around the host side of an entry point (named after it): a profiler's timeline shows which call enqueued
// which kernels; without a profiler attached the calls return at once.
struct Range {
    explicit Range(const char *name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
    Range(const Range &) = delete;
    Range &operator=(const Range &) = delete;
};

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Carver {
    char *base;
    size_t off = 0;
    template <typename T>
    T *take(size_t n) {
        off = (off + 255) & ~size_t(255);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

Dims dims_of_cfg(const spice_layer_cfg &g, int T) {
    return Dims{T, g.d, g.n_experts, g.top_k, g.inter, g.inter_shared, g.lore_rank, g.n_slots};
}

void carve(spice_ctx *c, char *base, size_t *total) {
    const spice_layer_cfg &g = c->cfg;
    const size_t Tm = (size_t)c->max_tokens, K = g.top_k, n = Tm * K;
    Carver cv{base};
    c->tb.groups = cv.take<GroupDesc>(1 + (size_t)g.n_slots + g.n_experts);
    c->tb.hdr = cv.take<int32_t>(HDR_WORDS);
    c->tb.status = cv.take<int32_t>(4);
    c->tb.perm_hit = cv.take<int32_t>(n);
    c->tb.perm_low = cv.take<int32_t>(n);
    c->tb.pos_of_entry = cv.take<int32_t>(n);
    c->tb.coef_shared = cv.take<float>(Tm);
    c->tb.act_hit = cv.take<float>(n * g.inter);
    c->tb.act_shared = cv.take<float>(Tm * g.inter_shared);
    c->tb.z_low = cv.take<float>(n * g.lore_rank);
    c->tb.part = cv.take<float>(n * g.d);
    c->tb.part_shared = cv.take<float>(Tm * g.d);
    c->ws_idx = cv.take<int32_t>(n);
    c->ws_slot = cv.take<int32_t>(n);
    c->ws_counts = cv.take<int32_t>(4);
    c->ws_gate = cv.take<float>(n);
    c->ws_cls = cv.take<uint8_t>(n);
    c->y32 = cv.take<float>(Tm * g.d);
    c->gsc.cnt = cv.take<int32_t>(4096);
    c->gsc.off = cv.take<int32_t>(2048);
    c->gsc.blk_miss = cv.take<int32_t>(n / 1024 + 2);
    c->draft_logits = cv.take<float>(Tm * g.n_experts);
    c->route_logits = cv.take<float>(Tm * g.n_experts);
    c->roll_h = cv.take<__nv_bfloat16>(Tm * g.d);
    c->roll_y = cv.take<__nv_bfloat16>(Tm * g.d);
    c->roll_conf = cv.take<float>(Tm);
    c->roll_active = cv.take<int32_t>(Tm);
    c->roll_active2 = cv.take<int32_t>(Tm);
    // decode kernels: activations of a group are kept for every token of the batch ([group][T][width])
    const size_t Td = Tm < 64 ? Tm : 64, nd = Td * K;
    const size_t g_hit = (size_t)g.n_slots < nd ? g.n_slots : nd, g_low = (size_t)g.n_experts < nd ? g.n_experts : nd;
    c->logits = cv.take<float>(Td * g.n_experts);
    c->act_hit16 = cv.take<__nv_bfloat16>((g_hit * Td > nd ? g_hit * Td : nd) * g.inter);
    c->act_shared16 = cv.take<__nv_bfloat16>(Td * g.inter_shared);
    c->z16 = cv.take<__nv_bfloat16>((g_low * Td > nd ? g_low * Td : nd) * g.lore_rank);
    c->part_split = cv.take<float>((size_t)decode_tc_nsplit(dims_of_cfg(g, 1)) * Td * g.d);
    {   // 8-bit weight precision (decode batches of at most 32 tokens)
        const size_t T8 = Tm < 32 ? Tm : 32, n8 = T8 * K, g8 = (size_t)g.n_slots < n8 ? g.n_slots : n8;
        c->x8_h = cv.take<uint8_t>(3 * T8 * g.d);
        c->act8_hit = cv.take<uint8_t>(g8 * 3 * T8 * g.inter);
        c->act8_sh = cv.take<uint8_t>(3 * T8 * g.inter_shared);
    }
    c->sync_words = SY_GROUP0 + 1 + g.n_slots + g.n_experts;
    c->sync = cv.take<int32_t>(c->sync_words);
    {   // buffers of the tensor-core path
        c->tcb.x_perm = cv.take<__nv_bfloat16>(n * g.d);
        c->tcb.act16 = cv.take<__nv_bfloat16>(n * g.inter);
        c->tcb.act_shared16 = cv.take<__nv_bfloat16>(Tm * g.inter_shared);
        c->tcb.mtiles = cv.take<MTile>(n / 128 + (g.n_slots > g.n_experts ? g.n_slots : g.n_experts) + 2);   // hit groups, later LOW groups
        c->tcb.mtiles_shared = cv.take<MTile>(Tm / 128 + 1);
        c->tcb.mtiles_low = cv.take<MTile>(n / 128 + g.n_experts + 2);
        c->tcb.n_mtiles = cv.take<int32_t>(4);
        c->tcb.n_mtiles_shared = cv.take<int32_t>(4);
        c->tcb.n_mtiles_low = cv.take<int32_t>(4);
        c->tcb.status = c->tb.status;
    }
    *total = (cv.off + 255) & ~size_t(255);
}

spice_status check_cfg(const spice_layer_cfg *g, int32_t max_tokens) {
    if (!g) return SPICE_ERR_INVALID_ARG;
    if (max_tokens < 1 || max_tokens > 65535) return SPICE_ERR_INVALID_ARG;
    if (g->d < 8 || g->d % 8 || g->inter < 8 || g->inter % 8 || g->inter_shared < 8 || g->inter_shared % 8 ||
        g->lore_rank < 8 || g->lore_rank % 8)
        return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (g->n_experts < 1 || g->n_experts > 1024 || g->n_slots < 1 || g->n_slots > 1024)
        return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (g->top_k < 1 || g->top_k > 32 || g->top_k > g->n_experts) return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (g->conf_stride != 0 && g->conf_stride != g->n_experts) return SPICE_ERR_INVALID_ARG;
    if ((size_t)g->d * 4 + (size_t)g->n_experts * 4 > 200 * 1024) return SPICE_ERR_UNSUPPORTED_SHAPE;
    return SPICE_OK;
}

Dims dims_of(const spice_ctx *c, int T) {
    const spice_layer_cfg &g = c->cfg;
    return Dims{T, g.d, g.n_experts, g.top_k, g.inter, g.inter_shared, g.lore_rank, g.n_slots};
}

spice_status check_call(const spice_ctx *c, int32_t T) {
    if (!c) return SPICE_ERR_INVALID_ARG;
    if (T < 0 || T > c->max_tokens) return SPICE_ERR_INVALID_ARG;
    return SPICE_OK;
}

bool weights_ok(const spice_layer_weights *w, bool routed, bool shared_lore) {
    if (!w) return false;
    if (routed && !(w->slot_w_gate_up && w->slot_w_down && aligned16(w->slot_w_gate_up) && aligned16(w->slot_w_down)))
        return false;
    if (shared_lore && !(w->shared_w_gate_up && w->shared_w_down && w->lore_A && w->lore_B &&
                         aligned16(w->shared_w_gate_up) && aligned16(w->shared_w_down) && aligned16(w->lore_A) &&
                         aligned16(w->lore_B)))
        return false;
    return true;
}

// the fields of the decode kernels' parameter block that come from the ctx
DecodeParams decode_params_of(const spice_ctx *ctx, const Dims &dm) {
    DecodeParams p{};
    p.dm = dm;
    p.norm_topk = ctx->cfg.norm_topk;
    p.conf_stride = ctx->cfg.conf_stride;
    p.tau = ctx->cfg.tau;
    p.n_r1 = dm.N;   // one router task per expert
    p.spin_limit = (int32_t)ctx->opt_spin_limit;
    p.sync_words = ctx->sync_words;
    p.tb = ctx->tb;
    p.logits = ctx->logits;
    p.act_hit16 = ctx->act_hit16;
    p.act_shared16 = ctx->act_shared16;
    p.z16 = ctx->z16;
    p.sync = ctx->sync;
    p.x_idx = ctx->ws_idx;
    p.x_gate = ctx->ws_gate;
    p.x_cls = ctx->ws_cls;
    return p;
}

// adds n launches or turns a launch failure into SPICE_ERR_CUDA
#define SPICE_LAUNCH(expr)                       \
    do {                                         \
        int n_ = (expr);                         \
        if (n_ < 0) return SPICE_ERR_CUDA;       \
        ctx->launches += n_;                     \
    } while (0)

spice_status layer_general_path(spice_ctx *ctx, const spice_layer_weights *w, const __nv_bfloat16 *hb, const float *conf, int32_t T,
                                const float *y_cpu_residual, spice_bf16 *x_resid, spice_bf16 *y, int32_t *idx, float *gate,
                                uint8_t *cls, int32_t *counts, int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                                float *resid_gate, cudaStream_t st);

}  // namespace

extern "C" {

int32_t spice_version(void) { return 200; }

const char *spice_status_string(spice_status s) {
    switch (s) {
        case SPICE_OK: return "ok";
        case SPICE_ERR_INVALID_ARG: return "invalid argument";
        case SPICE_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case SPICE_ERR_WORKSPACE: return "workspace allocation failed";
        case SPICE_ERR_CUDA: return "CUDA runtime error";
        case SPICE_ERR_BAD_TABLE: return "bad slot table or expert index (device)";
        case SPICE_ERR_TIMEOUT: return "bounded device wait expired";
    }
    return "unknown status";
}

spice_status spice_create(spice_ctx **out, int32_t device, const spice_layer_cfg *cfg, int32_t max_tokens) {
    if (!out) return SPICE_ERR_INVALID_ARG;
    *out = nullptr;
    spice_status s = check_cfg(cfg, max_tokens);
    if (s != SPICE_OK) return s;
    if (cudaSetDevice(device) != cudaSuccess) return SPICE_ERR_CUDA;
    spice_ctx *c = new (std::nothrow) spice_ctx();
    if (!c) return SPICE_ERR_WORKSPACE;
    c->device = device;
    c->cfg = *cfg;
    c->max_tokens = max_tokens;
    c->launches = 0;
    c->opt_path = 0;
    c->opt_spin_limit = 1 << 20;
    int coop = 0;
    if (cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, device) != cudaSuccess) {
        delete c;
        return SPICE_ERR_CUDA;
    }
    c->decode_tokens = (coop && decode_prepare(c->max_smem_optin) == 0) ? (max_tokens < 16 ? max_tokens : 16) : 0;
    c->tcb = TcBuffers{};
    c->tc_ok = tc_available() && tc_prepare() == 0;
    c->side = nullptr;
    c->ev_fork = c->ev_join = c->ev_grouped = nullptr;
    if (c->tc_ok) {
        if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&c->ev_grouped, cudaEventDisableTiming) != cudaSuccess) {
            cudaGetLastError();
            if (c->side) cudaStreamDestroy(c->side);
            if (c->ev_fork) cudaEventDestroy(c->ev_fork);
            if (c->ev_join) cudaEventDestroy(c->ev_join);
            if (c->ev_grouped) cudaEventDestroy(c->ev_grouped);
            c->side = nullptr;
            c->ev_fork = c->ev_join = c->ev_grouped = nullptr;
        }
    }
    c->dtc_tokens = (coop && c->tc_ok && decode_tc_prepare(c->max_smem_optin) == 0) ? (max_tokens < 64 ? max_tokens : 64) : 0;
    carve(c, nullptr, &c->ws_bytes);
    if (cudaMalloc(&c->ws, c->ws_bytes) != cudaSuccess) {
        cudaGetLastError();
        delete c;
        return SPICE_ERR_WORKSPACE;
    }
    size_t total;
    carve(c, static_cast<char *>(c->ws), &total);
    if (cudaMemset(c->ws, 0, c->ws_bytes) != cudaSuccess) {
        cudaFree(c->ws);
        delete c;
        return SPICE_ERR_CUDA;
    }
    *out = c;
    return SPICE_OK;
}

spice_status spice_destroy(spice_ctx *ctx) {
    if (!ctx) return SPICE_OK;
    cudaSetDevice(ctx->device);
    cudaError_t e = cudaFree(ctx->ws);
    if (ctx->side) {
        cudaStreamDestroy(ctx->side);
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
        cudaEventDestroy(ctx->ev_grouped);
    }
    delete ctx;
    return e == cudaSuccess ? SPICE_OK : SPICE_ERR_CUDA;
}

spice_status spice_workspace_bytes(const spice_ctx *ctx, size_t *bytes) {
    if (!ctx || !bytes) return SPICE_ERR_INVALID_ARG;
    *bytes = ctx->ws_bytes;
    return SPICE_OK;
}

spice_status spice_launch_count(const spice_ctx *ctx, int64_t *launches) {
    if (!ctx || !launches) return SPICE_ERR_INVALID_ARG;
    *launches = ctx->launches;
    return SPICE_OK;
}

spice_status spice_get_device_status(spice_ctx *ctx, int32_t *code) {
    if (!ctx || !code) return SPICE_ERR_INVALID_ARG;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return SPICE_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return SPICE_ERR_CUDA;
    int32_t v = 0;
    if (cudaMemcpy(&v, ctx->tb.status, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return SPICE_ERR_CUDA;
    if (cudaMemset(ctx->tb.status, 0, sizeof(int32_t)) != cudaSuccess) return SPICE_ERR_CUDA;
    // a kernel that gave up may have left dependency counters behind
    if (v != 0 && cudaMemset(ctx->sync, 0, sizeof(int32_t) * ctx->sync_words) != cudaSuccess) return SPICE_ERR_CUDA;
    *code = v;
    return SPICE_OK;
}

spice_status spice_set_option(spice_ctx *ctx, int32_t option, int64_t value) {
    if (!ctx) return SPICE_ERR_INVALID_ARG;
    switch (option) {
        case SPICE_OPT_PATH:
            if (value < 0 || value > 3) return SPICE_ERR_INVALID_ARG;
            ctx->opt_path = value;
            return SPICE_OK;
        case SPICE_OPT_SPIN_LIMIT:
            if (value < 1 || value > (1ll << 30)) return SPICE_ERR_INVALID_ARG;
            ctx->opt_spin_limit = value;
            return SPICE_OK;
        case SPICE_OPT_TC_WAIT_LIMIT:
            if (value < 1 || value > (1ll << 30)) return SPICE_ERR_INVALID_ARG;
            ctx->tcb.wait_limit = (uint32_t)value;
            return SPICE_OK;
    }
    return SPICE_ERR_INVALID_ARG;
}

spice_status spice_route_topk(spice_ctx *ctx, const spice_bf16 *h, const spice_bf16 *w_router, int32_t T,
                              int32_t *idx, float *gate, float *logits, void *stream) {
    Range range_("spice_route_topk");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    if (T == 0) return SPICE_OK;
    if (!h || !w_router || !idx || !gate || !aligned16(h) || !aligned16(w_router)) return SPICE_ERR_INVALID_ARG;
    SPICE_LAUNCH(launch_route_topk(dims_of(ctx, T), ctx->cfg.norm_topk, reinterpret_cast<const __nv_bfloat16 *>(h),
                                   reinterpret_cast<const __nv_bfloat16 *>(w_router), idx, gate, logits,
                                   static_cast<cudaStream_t>(stream)));
    return SPICE_OK;
}

int32_t spice_min_lookahead_depth(int32_t n_prefetch, double expert_bytes, double pcie_bytes_per_s, double t_comp_s) {
    if (n_prefetch < 0 || !(expert_bytes >= 0.0) || !(pcie_bytes_per_s > 0.0) || !(t_comp_s > 0.0)) return -1;
    const double x = (double)n_prefetch * expert_bytes / (pcie_bytes_per_s * t_comp_s);
    if (!(x < 2147483647.0)) return -1;
    const int32_t f = (int32_t)x;
    return (double)f < x ? f + 1 : f;
}

spice_status spice_draft_confidence(spice_ctx *ctx, const spice_bf16 *h_hat, const spice_bf16 *w_draft_router, int32_t T,
                                    int32_t *idx_hat, float *pi_hat, float *conf, void *stream) {
    Range range_("spice_draft_confidence");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    if (T == 0) return SPICE_OK;
    if (!h_hat || !w_draft_router || !idx_hat || !conf || !aligned16(h_hat) || !aligned16(w_draft_router))
        return SPICE_ERR_INVALID_ARG;
    SPICE_LAUNCH(launch_draft_confidence(dims_of(ctx, T), reinterpret_cast<const __nv_bfloat16 *>(h_hat),
                                         reinterpret_cast<const __nv_bfloat16 *>(w_draft_router), idx_hat, ctx->ws_gate,
                                         ctx->draft_logits, pi_hat, conf, static_cast<cudaStream_t>(stream)));
    return SPICE_OK;
}

spice_status spice_prefetch_rollout(spice_ctx *ctx, const spice_layer_weights *w, const spice_bf16 *x_current, int32_t T,
                                    int32_t l_min, int32_t l_max, float tau, int32_t *idx_hat, float *conf, int32_t *depth,
                                    spice_bf16 *h_final, uint8_t *prefetch_mask, void *stream) {
    Range range_("spice_prefetch_rollout");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    if (l_max < 1 || l_max > 64 || l_min < 1 || l_min > l_max) return SPICE_ERR_INVALID_ARG;
    if (T == 0) return SPICE_OK;
    if (!w || !x_current || !idx_hat || !conf || !depth || !aligned16(x_current)) return SPICE_ERR_INVALID_ARG;
    for (int l = 0; l < l_max; ++l) {
        if (!w[l].w_router || !aligned16(w[l].w_router)) return SPICE_ERR_INVALID_ARG;
        if (l + 1 < l_max && !weights_ok(&w[l], false, true)) return SPICE_ERR_INVALID_ARG;   // the last depth only routes
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Dims dm = dims_of(ctx, T);
    const size_t bytes = (size_t)T * dm.d * sizeof(__nv_bfloat16);
    if (cudaMemcpyAsync(ctx->roll_h, x_current, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SPICE_ERR_CUDA;
    const bool fused = ctx->opt_path == 0 && T <= ctx->dtc_tokens && decode_tc_supported(dm, 0, (size_t)ctx->max_smem_optin);
    bool done = false;
    if (fused) {
        // one launch of the decode kernel per projecting depth (router, halting rule, shared expert + LoRE, state update);
        // the last depth only routes
        const size_t n = (size_t)T * dm.K;
        int32_t *act[2] = {ctx->roll_active, ctx->roll_active2};
        done = true;
        for (int l = 1; l < l_max && done; ++l) {
            DecodeParams p = decode_params_of(ctx, dm);
            p.norm_topk = 0;
            p.conf_stride = 0;
            p.h = ctx->roll_h;
            p.w = w[l - 1];
            p.w.slot_w_gate_up = p.w.shared_w_gate_up;   // (no resident experts in the rollout: never read)
            p.w.slot_w_down = p.w.shared_w_down;
            p.idx = ctx->ws_idx;
            p.gate = ctx->ws_gate;
            p.cls = ctx->ws_cls;
            p.counts = ctx->ws_counts;
            p.y16 = ctx->roll_y;
            p.x_resid = ctx->roll_h;
            p.roll_depth = l;
            p.roll_l_min = l_min;
            p.roll_tau = tau;
            p.roll_active_in = act[(l + 1) & 1];
            p.roll_active_out = act[l & 1];
            p.roll_idx_out = idx_hat + (size_t)(l - 1) * n;
            p.roll_conf_out = conf + (size_t)(l - 1) * T;
            p.roll_depth_out = depth;
            int k = launch_decode_tc(p, ctx->part_split, ctx->n_sms, ctx->max_smem_optin, st);
            if (k < 0) {
                done = false;      // cooperative launch refused: start over on the general kernels
                break;
            }
            ctx->launches += k;
        }
        if (done) {
            const spice_layer_weights &wl = w[l_max - 1];
            SPICE_LAUNCH(launch_draft_confidence(dm, ctx->roll_h, reinterpret_cast<const __nv_bfloat16 *>(wl.w_router),
                                                 ctx->ws_idx, ctx->ws_gate, ctx->draft_logits, nullptr, ctx->roll_conf, st));
            SPICE_LAUNCH(launch_rollout_mask(dm, l_max, l_min, l_max, tau, ctx->roll_conf, act[(l_max + 1) & 1], ctx->ws_idx,
                                             idx_hat + (size_t)(l_max - 1) * n, conf + (size_t)(l_max - 1) * T, ctx->ws_cls,
                                             depth, st));
        } else if (cudaMemcpyAsync(ctx->roll_h, x_current, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            return SPICE_ERR_CUDA;
        }
    }
    if (!done)
        SPICE_LAUNCH(launch_rollout(dm, w, l_min, l_max, tau, ctx->roll_h, ctx->roll_y, ctx->ws_idx, ctx->ws_gate, ctx->ws_cls,
                                    ctx->roll_conf, ctx->draft_logits, ctx->roll_active, ctx->tb, idx_hat, conf, depth, st));
    if (h_final && cudaMemcpyAsync(h_final, ctx->roll_h, bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return SPICE_ERR_CUDA;
    if (prefetch_mask) SPICE_LAUNCH(launch_prefetch_set(dm, l_max, idx_hat, prefetch_mask, st));
    return SPICE_OK;
}

size_t spice_lore_calibrate_workspace_bytes(int32_t d, int32_t n_tokens, int32_t rank) {
    if (d < 1 || n_tokens < 1 || rank < 1) return 0;
    return lore_calibrate_workspace_bytes(d, n_tokens, rank);
}

spice_status spice_lore_calibrate(int32_t d, int32_t n_tokens, int32_t rank, float ridge, int32_t iterations,
                                  const spice_bf16 *h_cal, const float *resid, spice_bf16 *A_out, spice_bf16 *B_out,
                                  float *loss_out, int32_t *device_status, void *workspace, size_t workspace_bytes,
                                  void *stream) {
    Range range_("spice_lore_calibrate");
    if (d < 8 || d % 8 || rank < 1 || 2 * rank > d || n_tokens < 1 || iterations < 0 || iterations > 1000 || !(ridge >= 0.f))
        return SPICE_ERR_INVALID_ARG;
    if (!h_cal || !resid || !A_out || !B_out || !device_status || !workspace) return SPICE_ERR_INVALID_ARG;
    if (workspace_bytes < lore_calibrate_workspace_bytes(d, n_tokens, rank)) return SPICE_ERR_WORKSPACE;
    int n = launch_lore_calibrate(d, n_tokens, rank, ridge, iterations, reinterpret_cast<const __nv_bfloat16 *>(h_cal), resid,
                                  reinterpret_cast<__nv_bfloat16 *>(A_out), reinterpret_cast<__nv_bfloat16 *>(B_out), loss_out,
                                  device_status, workspace, static_cast<cudaStream_t>(stream));
    return n < 0 ? SPICE_ERR_CUDA : SPICE_OK;
}

spice_status spice_classify_misses(spice_ctx *ctx, const int32_t *idx, const float *gate,
                                   const int32_t *slot_of_expert, const float *conf, int32_t T, uint8_t *cls,
                                   int32_t *slot, int32_t *counts, int32_t *resid_tok, int32_t *resid_k,
                                   int32_t *resid_expert, float *resid_gate, void *stream) {
    Range range_("spice_classify_misses");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (T == 0) {
        if (!counts) return SPICE_OK;
        return cudaMemsetAsync(counts, 0, 3 * sizeof(int32_t), st) == cudaSuccess ? SPICE_OK : SPICE_ERR_CUDA;
    }
    if (!idx || !gate || !slot_of_expert || !conf || !cls || !slot || !counts) return SPICE_ERR_INVALID_ARG;
    if (!(resid_tok && resid_k && resid_expert && resid_gate)) resid_tok = resid_k = resid_expert = nullptr, resid_gate = nullptr;
    SPICE_LAUNCH(launch_classify(dims_of(ctx, T), ctx->cfg.conf_stride, ctx->cfg.tau, idx, gate, slot_of_expert, conf,
                                 cls, slot, counts, resid_tok, resid_k, resid_expert, resid_gate, ctx->tb.status, st, &ctx->gsc));
    return SPICE_OK;
}

spice_status spice_grouped_expert_ffn(spice_ctx *ctx, const spice_layer_weights *w, const spice_bf16 *h,
                                      const int32_t *idx, const float *gate, const uint8_t *cls,
                                      const int32_t *slot, int32_t T, float *y, void *stream) {
    Range range_("spice_grouped_expert_ffn");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    if (T == 0) return SPICE_OK;
    if (!weights_ok(w, true, false) || !h || !idx || !gate || !cls || !slot || !y || !aligned16(h) || !aligned16(y))
        return SPICE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Dims dm = dims_of(ctx, T);
    const __nv_bfloat16 *hb = reinterpret_cast<const __nv_bfloat16 *>(h);
    SPICE_LAUNCH(launch_group(dm, idx, gate, cls, slot, ctx->tb, st, &ctx->gsc));
    if (T > 64 && ctx->opt_path != 1 && ctx->opt_path != 3 && ctx->tc_ok && tc_shape_ok(dm)) {
        SPICE_LAUNCH(launch_tc_routed(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, st));   // grouped GEMM on the tensor cores
    } else {
        SPICE_LAUNCH(launch_gateup(dm, KIND_HIT, *w, hb, ctx->tb, st));
        SPICE_LAUNCH(launch_down(dm, KIND_HIT, *w, ctx->tb, st));
    }
    CombineArgs ca{KIND_HIT, 1, gate, cls, y, nullptr, nullptr, nullptr};
    SPICE_LAUNCH(launch_combine(dm, ca, ctx->tb, st));
    return SPICE_OK;
}

spice_status spice_lore_surrogate(spice_ctx *ctx, const spice_layer_weights *w, const spice_bf16 *h,
                                  const int32_t *idx, const float *gate, const uint8_t *cls, int32_t T, float *y,
                                  void *stream) {
    Range range_("spice_lore_surrogate");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    if (T == 0) return SPICE_OK;
    if (!weights_ok(w, false, true) || !h || !idx || !gate || !cls || !y || !aligned16(h) || !aligned16(y))
        return SPICE_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const Dims dm = dims_of(ctx, T);
    const __nv_bfloat16 *hb = reinterpret_cast<const __nv_bfloat16 *>(h);
    // no slot array: HIT entries are left out of the grouping
    SPICE_LAUNCH(launch_group(dm, idx, gate, cls, nullptr, ctx->tb, st, &ctx->gsc));
    if (T > 64 && ctx->opt_path != 1 && ctx->opt_path != 3 && ctx->tc_ok && tc_shape_ok(dm) && tc_lore_ok(dm)) {
        SPICE_LAUNCH(launch_tc_shared(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, st));
        SPICE_LAUNCH(launch_tc_lore_a(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, st));
        SPICE_LAUNCH(launch_lore_b(dm, *w, ctx->tb, 1, st));
    } else {
        SPICE_LAUNCH(launch_gateup(dm, KIND_SHARED, *w, hb, ctx->tb, st));
        SPICE_LAUNCH(launch_lore_a(dm, *w, hb, ctx->tb, st));
        SPICE_LAUNCH(launch_down(dm, KIND_SHARED | KIND_LOW, *w, ctx->tb, st));
    }
    CombineArgs ca{KIND_SHARED | KIND_LOW, 1, gate, cls, y, nullptr, nullptr, nullptr};
    SPICE_LAUNCH(launch_combine(dm, ca, ctx->tb, st));
    return SPICE_OK;
}

spice_status spice_moe_layer_fwd(spice_ctx *ctx, const spice_layer_weights *w, const spice_bf16 *h,
                                 const float *conf, int32_t T, const float *y_cpu_residual, spice_bf16 *x_resid,
                                 spice_bf16 *y, int32_t *idx, float *gate, uint8_t *cls, int32_t *counts,
                                 int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert, float *resid_gate,
                                 void *stream) {
    Range range_("spice_moe_layer_fwd");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!counts) counts = ctx->ws_counts;
    if (T == 0) return cudaMemsetAsync(counts, 0, 3 * sizeof(int32_t), st) == cudaSuccess ? SPICE_OK : SPICE_ERR_CUDA;
    if (!weights_ok(w, true, true) || !w->w_router || !w->slot_of_expert || !aligned16(w->w_router) || !h || !conf ||
        !y || !aligned16(h) || !aligned16(y))
        return SPICE_ERR_INVALID_ARG;
    if ((y_cpu_residual && !aligned16(y_cpu_residual)) || (x_resid && !aligned16(x_resid))) return SPICE_ERR_INVALID_ARG;
    if (!idx) idx = ctx->ws_idx;
    if (!gate) gate = ctx->ws_gate;
    if (!cls) cls = ctx->ws_cls;
    if (!(resid_tok && resid_k && resid_expert && resid_gate)) resid_tok = resid_k = resid_expert = nullptr, resid_gate = nullptr;
    const Dims dm = dims_of(ctx, T);
    const __nv_bfloat16 *hb = reinterpret_cast<const __nv_bfloat16 *>(h);
    const bool use_dtc = ctx->opt_path == 0 && T <= ctx->dtc_tokens &&
                         decode_tc_supported(dm, ctx->cfg.conf_stride, (size_t)ctx->max_smem_optin);
    const bool use_dec = !use_dtc && (ctx->opt_path == 0 || ctx->opt_path == 3) && T <= ctx->decode_tokens &&
                         decode_supported(dm, (size_t)ctx->max_smem_optin);
    if (use_dtc || use_dec) {
        // small batch: one persistent kernel for the whole layer
        DecodeParams p = decode_params_of(ctx, dm);
        p.h = hb;
        p.conf = conf;
        p.w = *w;
        p.idx = idx;
        p.gate = gate;
        p.cls = cls;
        p.counts = counts;
        p.resid_tok = resid_tok;
        p.resid_k = resid_k;
        p.resid_expert = resid_expert;
        p.resid_gate = resid_gate;
        p.y16 = reinterpret_cast<__nv_bfloat16 *>(y);
        p.y_cpu = y_cpu_residual;
        p.x_resid = reinterpret_cast<__nv_bfloat16 *>(x_resid);
        int n = use_dtc ? launch_decode_tc(p, ctx->part_split, ctx->n_sms, ctx->max_smem_optin, st)
                        : launch_decode(p, ctx->n_sms, st);
        if (n > 0) {
            ctx->launches += n;
            return SPICE_OK;
        }
        // cooperative launch refused (e.g. device shared with another context): use the general path
    }
    return layer_general_path(ctx, w, hb, conf, T, y_cpu_residual, x_resid, y, idx, gate, cls, counts, resid_tok, resid_k,
                              resid_expert, resid_gate, st);
}

spice_status spice_quantize_e4m3_rows(const spice_bf16 *w, int64_t rows, int32_t cols, uint8_t *q, float *scale, void *stream) {
    Range range_("spice_quantize_e4m3_rows");
    if (rows < 0 || cols < 8 || cols % 8) return SPICE_ERR_INVALID_ARG;
    if (rows == 0) return SPICE_OK;
    if (!w || !q || !scale || !aligned16(w) || !aligned16(q)) return SPICE_ERR_INVALID_ARG;
    return launch_quantize_e4m3_rows(reinterpret_cast<const __nv_bfloat16 *>(w), (size_t)rows, cols, q, scale,
                                     static_cast<cudaStream_t>(stream)) < 0 ? SPICE_ERR_CUDA : SPICE_OK;
}

spice_status spice_moe_layer_fwd_fp8(spice_ctx *ctx, const spice_layer_weights_fp8 *w, const spice_bf16 *h, const float *conf,
                                     int32_t T, const float *y_cpu_residual, spice_bf16 *x_resid, spice_bf16 *y, int32_t *idx,
                                     float *gate, uint8_t *cls, int32_t *counts, int32_t *resid_tok, int32_t *resid_k,
                                     int32_t *resid_expert, float *resid_gate, void *stream) {
    Range range_("spice_moe_layer_fwd_fp8");
    spice_status s = check_call(ctx, T);
    if (s != SPICE_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!counts) counts = ctx->ws_counts;
    if (T == 0) return cudaMemsetAsync(counts, 0, 3 * sizeof(int32_t), st) == cudaSuccess ? SPICE_OK : SPICE_ERR_CUDA;
    if (!w || !w->w_router || !w->slot_of_expert || !w->slot_q_gate_up || !w->slot_s_gate_up || !w->slot_q_down || !w->slot_s_down ||
        !w->shared_q_gate_up || !w->shared_s_gate_up || !w->shared_q_down || !w->shared_s_down || !w->lore_A || !w->lore_B)
        return SPICE_ERR_INVALID_ARG;
    if (!aligned16(w->w_router) || !aligned16(w->slot_q_gate_up) || !aligned16(w->slot_q_down) || !aligned16(w->shared_q_gate_up) ||
        !aligned16(w->shared_q_down) || !aligned16(w->lore_A) || !aligned16(w->lore_B))
        return SPICE_ERR_INVALID_ARG;
    if (!h || !conf || !y || !aligned16(h) || !aligned16(y)) return SPICE_ERR_INVALID_ARG;
    if ((y_cpu_residual && !aligned16(y_cpu_residual)) || (x_resid && !aligned16(x_resid))) return SPICE_ERR_INVALID_ARG;
    const Dims dm = dims_of(ctx, T);
    if (T > 32 || T > ctx->dtc_tokens || !decode_tc_supported(dm, ctx->cfg.conf_stride, (size_t)ctx->max_smem_optin, true))
        return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (!idx) idx = ctx->ws_idx;
    if (!gate) gate = ctx->ws_gate;
    if (!cls) cls = ctx->ws_cls;
    if (!(resid_tok && resid_k && resid_expert && resid_gate)) resid_tok = resid_k = resid_expert = nullptr, resid_gate = nullptr;
    DecodeParams p = decode_params_of(ctx, dm);
    p.h = reinterpret_cast<const __nv_bfloat16 *>(h);
    p.conf = conf;
    p.w = spice_layer_weights{};
    p.w.w_router = w->w_router;
    p.w.slot_of_expert = w->slot_of_expert;
    p.w.lore_A = w->lore_A;
    p.w.lore_B = w->lore_B;
    p.idx = idx;
    p.gate = gate;
    p.cls = cls;
    p.counts = counts;
    p.resid_tok = resid_tok;
    p.resid_k = resid_k;
    p.resid_expert = resid_expert;
    p.resid_gate = resid_gate;
    p.y16 = reinterpret_cast<__nv_bfloat16 *>(y);
    p.y_cpu = y_cpu_residual;
    p.x_resid = reinterpret_cast<__nv_bfloat16 *>(x_resid);
    Fp8Layer f8{w->slot_q_gate_up, w->slot_q_down, w->shared_q_gate_up, w->shared_q_down,
                w->slot_s_gate_up, w->slot_s_down, w->shared_s_gate_up, w->shared_s_down,
                ctx->x8_h, ctx->act8_hit, ctx->act8_sh};
    const int n = launch_decode_tc(p, ctx->part_split, ctx->n_sms, ctx->max_smem_optin, st, &f8);
    if (n < 0) return SPICE_ERR_CUDA;
    ctx->launches += n;
    return SPICE_OK;
}

}  // extern "C"

namespace {

// the layer on the kernels for batches and shapes the fused decode kernels do not take
spice_status layer_general_path(spice_ctx *ctx, const spice_layer_weights *w, const __nv_bfloat16 *hb, const float *conf, int32_t T,
                                const float *y_cpu_residual, spice_bf16 *x_resid, spice_bf16 *y, int32_t *idx, float *gate,
                                uint8_t *cls, int32_t *counts, int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                                float *resid_gate, cudaStream_t st) {
    const Dims dm = dims_of(ctx, T);
    const bool tc_path = ctx->opt_path != 1 && ctx->opt_path != 3 && ctx->tc_ok && tc_shape_ok(dm);
    // The shared expert needs nothing but h: it runs on the context's side stream beside the routing chain (router,
    // classification, grouping, gather occupy few SMs) and joins before the combine.  Both event edges are ordinary
    // stream dependencies, so the call can still be captured into a CUDA graph.  Once the side stream has been forked
    // off, every way out of this function -- an error return included -- joins it back into the caller's stream: a
    // capture of that stream would otherwise be left with an unjoined branch.
    bool forked = false;
    spice_status rc = SPICE_OK;
    // (a failed launch ends the sequence; the join below still runs)
#define SPICE_STEP(expr)                          \
    do {                                          \
        if (rc == SPICE_OK) {                     \
            int n_ = (expr);                      \
            if (n_ < 0) rc = SPICE_ERR_CUDA;      \
            else ctx->launches += n_;             \
        }                                         \
    } while (0)
    if (tc_path) {
        if (ctx->side && cudaEventRecord(ctx->ev_fork, st) == cudaSuccess &&
            cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) == cudaSuccess) {
            forked = true;
            SPICE_STEP(launch_tc_shared(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, ctx->side));
        } else {
            cudaGetLastError();
        }
    }
    if (tc_path && T > 64 && tc_router_ok(dm)) {
        // large batch: the logits are a GEMM of their own (a status word of the GEMM is the tables' one)
        SPICE_STEP(launch_tc_router_logits(dm, hb, reinterpret_cast<const __nv_bfloat16 *>(w->w_router), ctx->route_logits,
                                           ctx->tcb, ctx->n_sms, st));
        SPICE_STEP(launch_topk_from_logits(dm, ctx->cfg.norm_topk, ctx->route_logits, idx, gate, st));
    } else {
        SPICE_STEP(launch_route_topk(dm, ctx->cfg.norm_topk, hb, reinterpret_cast<const __nv_bfloat16 *>(w->w_router), idx,
                                     gate, nullptr, st));
    }
    SPICE_STEP(launch_classify_group(dm, ctx->cfg.conf_stride, ctx->cfg.tau, idx, gate, w->slot_of_expert, conf, cls,
                                     ctx->ws_slot, counts, resid_tok, resid_k, resid_expert, resid_gate, ctx->tb, st, &ctx->gsc));
    if (tc_path) {
        // batches the decode kernel does not take: exact experts, shared expert and LoRE down-projection on the
        // tensor cores (grouped GEMM kernel), LoRE up-projection on lore_b_kernel
        // the LoRE groups need the grouping, not the routed experts: on the side stream they run beside the routed GEMMs
        cudaStream_t ls = st;
        if (forked && rc == SPICE_OK) {
            if (cudaEventRecord(ctx->ev_grouped, st) != cudaSuccess || cudaStreamWaitEvent(ctx->side, ctx->ev_grouped, 0) != cudaSuccess)
                rc = SPICE_ERR_CUDA;
            ls = ctx->side;
        }
        SPICE_STEP(launch_tc_routed(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, st, gate));
        if (!forked) SPICE_STEP(launch_tc_shared(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, st));
        if (tc_lore_ok(dm)) {
            SPICE_STEP(launch_tc_lore_a(dm, *w, hb, ctx->tb, ctx->tcb, ctx->n_sms, ls));
            SPICE_STEP(launch_lore_b(dm, *w, ctx->tb, 1, ls));
        } else {
            SPICE_STEP(launch_lore_a(dm, *w, hb, ctx->tb, ls));
            SPICE_STEP(launch_lore_b(dm, *w, ctx->tb, 0, ls));
        }
    } else {
        SPICE_STEP(launch_gateup(dm, KIND_SHARED | KIND_HIT, *w, hb, ctx->tb, st));
        SPICE_STEP(launch_lore_a(dm, *w, hb, ctx->tb, st));
        SPICE_STEP(launch_down(dm, KIND_SHARED | KIND_HIT | KIND_LOW, *w, ctx->tb, st));
    }
    if (forked) {   // join, whatever happened above (after whatever ran on the side stream)
        if (cudaEventRecord(ctx->ev_join, ctx->side) != cudaSuccess || cudaStreamWaitEvent(st, ctx->ev_join, 0) != cudaSuccess) {
            cudaGetLastError();
            if (rc == SPICE_OK) rc = SPICE_ERR_CUDA;
        }
    }
    CombineArgs ca{KIND_SHARED | KIND_HIT | KIND_LOW, 0, gate, cls, nullptr, reinterpret_cast<__nv_bfloat16 *>(y),
                   y_cpu_residual, reinterpret_cast<__nv_bfloat16 *>(x_resid)};
    ca.hit_rows_gated16 = tc_path ? 1 : 0;
    SPICE_STEP(launch_combine(dm, ca, ctx->tb, st));
#undef SPICE_STEP
    return rc;
}

}  // namespace
