/*
 * spice.h -- C ABI of the B200 (sm_100a) MoE-layer forward for SPICE-style offloaded decoding.
 *
 * One call of spice_moe_layer_fwd computes the GPU part of one offloaded-MoE layer as the
 * paper states it:
 *     S_t = TopK(Router(h_t), K)                                   (Eq. 1, Sec. 2.2)
 *     shared experts always on, routed outputs gate-weighted        (Sec. 2.1)
 *     resident (prefetched) expert      -> executed exactly         (Sec. 4.2, runtime policy)
 *     missing, confidence < tau         -> S(h) + B_e A_e h         (Sec. 4.2, LoRE surrogate)
 *     missing, otherwise                -> listed for exact recovery (Sec. 4.3, set M)
 *     y_t = s_t + sum_{HIT} g_k E_{e_k}(h_t) + sum_{LOWCONF} g_k ( s_t + B_{e_k} A_{e_k} h_t )
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless it says "host".
 *   - bf16 tensors are passed as spice_bf16* (raw 16-bit patterns), row-major, 16-byte aligned,
 *     weights in [out, in] order.  Expert FFNs are SwiGLU: E(x) = W_d ( silu(W_g x) * (W_u x) ).
 *   - All calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default stream)
 *     and return without synchronising (spice_moe_layer_fwd can therefore be captured into a CUDA
 *     graph; pointers are baked in at capture time).  The library allocates device memory only in
 *     spice_create; per call it allocates nothing.  A ctx must not be used by two streams at once.
 *     For batches above 64 tokens spice_moe_layer_fwd runs the shared expert and the LoRE groups on a
 *     stream the ctx owns, forked from and joined back to `stream` by events inside the call: the
 *     caller sees stream order, and a capture of `stream` takes the fork in as edges of the graph.
 *   - Errors found on the host return a code and launch nothing.  Conditions found on the device
 *     (expert id out of range, slot index >= n_slots, an expired bounded wait) never trap: the
 *     entry is treated as an exact-recovery miss or skipped, a status word is set, and
 *     spice_get_device_status reports it.
 *   - T = 0 is SPICE_OK and launches nothing.
 *   - Class codes: 0 = HIT, 1 = MISS_EXACT, 2 = LOWCONF.  LOWCONF iff the expert is not resident
 *     and confidence < tau (strict; NaN compares false, i.e. exact recovery).
 *   - Top-k order: decreasing logit, equal logits towards the smaller expert index.
 */
#ifndef SPICE_H_
#define SPICE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint16_t spice_bf16;
typedef struct spice_ctx spice_ctx;

typedef enum {
    SPICE_OK = 0,
    SPICE_ERR_INVALID_ARG = 1,       /* NULL / misaligned pointer, T < 0, T > max_tokens            */
    SPICE_ERR_UNSUPPORTED_SHAPE = 2, /* a dimension the kernels do not cover (see spice_create)      */
    SPICE_ERR_WORKSPACE = 3,         /* workspace allocation failed                                  */
    SPICE_ERR_CUDA = 4,              /* a CUDA runtime call failed                                   */
    SPICE_ERR_BAD_TABLE = 5,         /* device: slot_of_expert entry >= n_slots, or expert id bad    */
    SPICE_ERR_TIMEOUT = 6            /* device: a bounded wait expired                               */
} spice_status;

enum { SPICE_HIT = 0, SPICE_MISS_EXACT = 1, SPICE_LOWCONF = 2 };

/* Static shape of one layer (notation of the paper: K of Eq. 1, r and d of the LoRE factors,
 * tau of Sec. 4.1/4.2). */
typedef struct {
    int32_t d;            /* hidden width; multiple of 8                                  */
    int32_t n_experts;    /* N routed experts, 1..1024                                    */
    int32_t top_k;        /* K, 1..min(N,32)                                              */
    int32_t inter;        /* I, routed SwiGLU intermediate width; multiple of 8           */
    int32_t inter_shared; /* I_s, width of the fused shared expert; multiple of 8         */
    int32_t lore_rank;    /* r; multiple of 8                                             */
    int32_t n_slots;      /* S, resident expert slots, 1..1024                            */
    int32_t norm_topk;    /* 1: gates = softmax over the K winners; 0: full-softmax probs */
    int32_t conf_stride;  /* N: conf is [T,N] per (token, expert); 0: conf is [T]         */
    float tau;            /* confidence threshold                                         */
} spice_layer_cfg;

/* Weights of one layer.  The slot pool holds the resident experts; LoRE factors and the shared
 * expert are resident for every expert (Sec. 3, scenario 2). */
typedef struct {
    const spice_bf16 *w_router;         /* [N, d]                                          */
    const spice_bf16 *slot_w_gate_up;   /* [S, 2I, d]: I gate rows, then I up rows         */
    const spice_bf16 *slot_w_down;      /* [S, d, I]                                       */
    const int32_t *slot_of_expert;      /* [N]; slot index, or -1 when not resident        */
    const spice_bf16 *shared_w_gate_up; /* [2 I_s, d]: I_s gate rows, then I_s up rows     */
    const spice_bf16 *shared_w_down;    /* [d, I_s]                                        */
    const spice_bf16 *lore_A;           /* [N, r, d]   A_e of Delta_e(h) = B_e A_e h       */
    const spice_bf16 *lore_B;           /* [N, d, r]   B_e                                 */
} spice_layer_weights;

/* Library version (major*10000 + minor*100 + patch).  Host only. */
int32_t spice_version(void);

/* Create a context for layers of shape *cfg on CUDA device `device`, able to process up to
 * max_tokens tokens per call.  Allocates the workspace (its size is reported by
 * spice_workspace_bytes).  Returns SPICE_ERR_UNSUPPORTED_SHAPE when a dimension breaks the
 * limits stated in spice_layer_cfg, SPICE_ERR_WORKSPACE / SPICE_ERR_CUDA on allocation failure.
 * The ctx is owned by the caller and released with spice_destroy. */
spice_status spice_create(spice_ctx **ctx, int32_t device, const spice_layer_cfg *cfg, int32_t max_tokens);
spice_status spice_destroy(spice_ctx *ctx);
spice_status spice_workspace_bytes(const spice_ctx *ctx, size_t *bytes /* host */);

/* Router + TopK + gate scores (Eq. 1; the routing result the runtime policy of Sec. 4.2 starts from).
 *   h [T,d] bf16, w_router [N,d] bf16  ->  idx [T,K] int32, gate [T,K] fp32,
 *   logits [T,N] fp32 (optional, may be NULL).
 * Logits are accumulated in fp32; selection is done on logits, never on exponentials. */
spice_status spice_route_topk(spice_ctx *ctx, const spice_bf16 *h, const spice_bf16 *w_router, int32_t T,
                              int32_t *idx, float *gate, float *logits, void *stream);

/* Hit / miss / low-confidence classification of every selected expert against the slot table and
 * the draft model's confidences (runtime policy of Sec. 4.2), and the residual-miss list
 * (set M of Sec. 4.3) in ascending (t*K + k) order.
 *   idx [T,K], gate [T,K], slot_of_expert [N], conf [T,N] fp32 (or [T] when conf_stride == 0)
 *   -> cls [T,K] uint8, slot [T,K] int32 (slot index for HIT, else -1),
 *      counts [3] int32 (entries per class code),
 *      resid_tok / resid_k / resid_expert [T*K] int32 and resid_gate [T*K] fp32: the first
 *      counts[1] entries are valid.  Any of the four resid arrays may be NULL (then none is written). */
spice_status spice_classify_misses(spice_ctx *ctx, const int32_t *idx, const float *gate,
                                   const int32_t *slot_of_expert, const float *conf, int32_t T,
                                   uint8_t *cls, int32_t *slot, int32_t *counts,
                                   int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                                   float *resid_gate, void *stream);

/* Exact execution of the resident experts (Sec. 4.2: an expert found on the GPU is run as it is):
 *   y[t,:] += sum over k with cls[t,k] == HIT of gate[t,k] * E_{slot[t,k]}(h[t,:]),   y [T,d] fp32.
 * Tokens are grouped by slot so that each resident expert's weights are read once. */
spice_status spice_grouped_expert_ffn(spice_ctx *ctx, const spice_layer_weights *w /* host struct */,
                                      const spice_bf16 *h, const int32_t *idx, const float *gate,
                                      const uint8_t *cls, const int32_t *slot, int32_t T, float *y,
                                      void *stream);

/* Shared expert plus LoRE substitution for low-confidence misses (Sec. 4.2, y~_e = S(h) + B_e A_e h):
 *   y[t,:] += (1 + sum_{LOWCONF} gate[t,k]) * S(h[t,:]) + sum_{LOWCONF} gate[t,k] * B_e A_e h[t,:],  y fp32. */
spice_status spice_lore_surrogate(spice_ctx *ctx, const spice_layer_weights *w /* host struct */,
                                  const spice_bf16 *h, const int32_t *idx, const float *gate,
                                  const uint8_t *cls, int32_t T, float *y, void *stream);

/* The whole layer: route -> classify -> resident experts + shared/LoRE -> combine.
 *   h [T,d] bf16, conf as in spice_classify_misses.
 *   y_cpu_residual [T,d] fp32, optional: outputs of exactly recovered experts computed elsewhere
 *       (Sec. 4.3: the GPU result and the experts recovered on the host are summed into one output); added before rounding.
 *   x_resid [T,d] bf16, optional, in/out: residual stream, x_resid <- x_resid + y.
 *   y [T,d] bf16 out.  idx, gate, cls, counts, resid_*: as above; each may be NULL when not wanted.
 * Equals spice_route_topk, spice_classify_misses, y = 0, spice_grouped_expert_ffn,
 * spice_lore_surrogate applied in turn, up to fp32 summation order and the final bf16 rounding.
 * Batches of more than 64 tokens take their router logits from a tensor-core GEMM (fp32 accumulation, truncated after
 * every 16 terms): the selection rule is the same, the logits differ from spice_route_topk's by up to ~1e-5, so idx
 * agrees with it whenever a token's K-th and (K+1)-th logits are further apart than that; gates agree to 4e-6. */
spice_status spice_moe_layer_fwd(spice_ctx *ctx, const spice_layer_weights *w /* host struct */,
                                 const spice_bf16 *h, const float *conf, int32_t T,
                                 const float *y_cpu_residual, spice_bf16 *x_resid, spice_bf16 *y,
                                 int32_t *idx, float *gate, uint8_t *cls, int32_t *counts,
                                 int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                                 float *resid_gate, void *stream);

/* Draft-router confidence (Sec. 4.1): the producer of the `conf` input above.
 *   pi_hat[t,:] = softmax over all N experts of  h_hat[t,:] . w_draft_router[e,:]      (predicted routing distribution)
 *   idx_hat[t,0..K-1] = TopK(pi_hat[t,:], K)                                          (Eq. 2; same order and tie rule as Eq. 1)
 *   conf[t] = sum_{i in idx_hat[t,:]} pi_hat[t,i]                                      (Eq. 5), summed in k order
 * h_hat [T,d] bf16: hidden states the draft predictor hands to the layer's router copy; w_draft_router [N,d] bf16.
 * idx_hat [T,K] int32 out; conf [T] fp32 out: the per-token confidence (the conf_stride = 0 layout of
 * spice_classify_misses / spice_moe_layer_fwd); pi_hat [T,N] fp32 out, optional (NULL: not wanted): the
 * per-(token, expert) layout (conf_stride = N).  The logits use the arithmetic of spice_route_topk, so idx_hat equals
 * what spice_route_topk returns for the same inputs, and pi_hat[t, idx_hat[t,k]] equals its gate with norm_topk = 0. */
spice_status spice_draft_confidence(spice_ctx *ctx, const spice_bf16 *h_hat, const spice_bf16 *w_draft_router,
                                    int32_t T, int32_t *idx_hat, float *pi_hat, float *conf, void *stream);

/* Speculative prefetch rollout (Algorithm 1, Sec. 4.1) for a batch of tokens, all depths on the device.
 * For depth l = 1 .. l_max, for every token that still speculates, with h^(0) = x_current:
 *     pi^(l) = softmax(router^(l)(h^(l-1))),  S^(l) = TopK(pi^(l), K) is enqueued,  C^(l) = sum_{i in S^(l)} pi^(l)_i;
 *     if l >= l_min and C^(l) < tau the token stops here (this prediction is kept, deeper ones are not made);
 *     h^(l) = h^(l-1) + sum_{i in S^(l)} pi^(l)_i * ( S^(l)(h^(l-1)) + B_i A_i h^(l-1) ).
 * Readings of the paper: the attention term of the projection, which the paper does not define for a single state, is the
 * identity; the state is held in bf16 between depths; a NaN confidence does not stop a token.
 *   w: HOST array of l_max structs, w[l-1] = weights of the layer at depth l; only w_router, shared_w_gate_up,
 *      shared_w_down, lore_A and lore_B are read (of w[l_max-1] only w_router).
 *   x_current [T,d] bf16.  1 <= l_min <= l_max <= 64.  tau: the threshold of Algorithm 1 (need not be cfg.tau).
 *   idx_hat [l_max,T,K] int32 out: predicted sets, -1 past a token's last depth.  conf [l_max,T] fp32 out, 0 there.
 *   depth [T] int32 out: number of predictions enqueued for the token (>= min(l_min, l_max)).
 *   h_final [T,d] bf16 out, optional: the draft state after the last projection made for each token.
 *   prefetch_mask [l_max, N] uint8 out, optional: the prefetch intents of Eq. 3 for the batch, kept per depth because
 *       depth l names experts of the layer l ahead: prefetch_mask[l-1, e] = 1 iff some token enqueues expert e at depth l.
 * Issuing the copies is the host runtime's job.  Decode batches the fused kernel takes run one launch per projecting
 * depth plus four small ones for the last depth and the prefetch set; other shapes run about 8 general-shape kernels per
 * depth.  Either way the call is bound by launch latency, not bandwidth. */
spice_status spice_prefetch_rollout(spice_ctx *ctx, const spice_layer_weights *w /* host array */,
                                    const spice_bf16 *x_current, int32_t T, int32_t l_min, int32_t l_max, float tau,
                                    int32_t *idx_hat, float *conf, int32_t *depth, spice_bf16 *h_final,
                                    uint8_t *prefetch_mask, void *stream);

/* Eq. 4 (host arithmetic, no device work): H_min = ceil(P * M_e / (B_PCIe * T_comp)), the lookahead depth needed to hide the
 * transfer of n_prefetch experts of expert_bytes each per layer behind t_comp_s seconds of compute per layer over a link of
 * pcie_bytes_per_s.  Returns -1 on a non-positive bandwidth or compute window. */
int32_t spice_min_lookahead_depth(int32_t n_prefetch, double expert_bytes, double pcie_bytes_per_s, double t_comp_s);

/* LoRE calibration of one (layer, expert) pair (Sec. 4.2): the rank-r residual module Delta(h) = B A h that minimises
 *     sum over the calibration tokens h routed to the expert of  || E(h) - S(h) - B A h ||_2^2 .
 * The paper trains the factors on this objective; it is a reduced-rank regression with a closed-form minimiser, which this
 * call computes on the device in fp32 (offline path, a few hundred small launches): G = H^T H + ridge * mean(diag G) * I,
 * C = H^T R, G = L L^T, Z = L^-1 C, V = the r leading eigenvectors of Z^T Z (block subspace iteration, `iterations` steps:
 * the objective is within 2 % of its minimum after 5 to 30 steps and within 1e-4 after 100 when neighbouring singular values
 * differ by 10 %), B = V, A = (G^-1 C V)^T.
 *   h_cal [n_tokens, d] bf16: calibration hidden states;  resid [n_tokens, d] fp32: targets E(h) - S(h) (e.g. from
 *   spice_grouped_expert_ffn and spice_lore_surrogate with zero factors);  A_out [rank, d], B_out [d, rank] bf16 out, in
 *   the layout of one expert's slice of spice_layer_weights.lore_A / lore_B.
 *   1 <= rank <= d / 2 (the surrogate is low-rank by construction: r << d).
 *   ridge >= 0: relative Tikhonov term; needed when n_tokens < d or the tokens are collinear (0 otherwise).
 *   loss_out: optional device float[2]: { objective at the bf16 factors written, sum ||resid||^2 }.
 *   device_status: device int32, out: 0, or 1 when a Cholesky pivot was not positive (G singular: raise ridge).
 *   workspace: device buffer of at least spice_lore_calibrate_workspace_bytes(d, n_tokens, rank) bytes, owned by the
 *   caller (the call allocates nothing); 256-byte aligned is best.  No spice_ctx is needed; the GPU is the calling
 *   thread's current device.  The factors are unique only up to an invertible r x r change of basis; B A is what is fitted. */
size_t spice_lore_calibrate_workspace_bytes(int32_t d, int32_t n_tokens, int32_t rank);
spice_status spice_lore_calibrate(int32_t d, int32_t n_tokens, int32_t rank, float ridge, int32_t iterations,
                                  const spice_bf16 *h_cal, const float *resid, spice_bf16 *A_out, spice_bf16 *B_out,
                                  float *loss_out, int32_t *device_status, void *workspace, size_t workspace_bytes,
                                  void *stream);

/* ---- Second weight precision: 8-bit expert weights (the paper reports every result at BF16 and at one quantised
 * precision, Sec. 5.1 and Table 1, and names that format without defining it).  Reading taken by this library: the
 * matrices of the routed experts and of the shared expert are stored as E4M3 bytes (1 sign, 4 exponent bits with bias 7,
 * 3 fraction bits; no infinities, S.1111.111 is NaN, largest value 448) with ONE fp32 scale per output row; the weight
 * the layer computes with is scale[row] * value(code).  Router and LoRE factors keep bf16, so routing and classification
 * do not depend on the precision.  Activations stay bf16 (inputs, the intermediate silu(g)*u, outputs): the layer at this
 * precision is, by definition, spice_moe_layer_fwd on the dequantised weights.  Half the weight bytes cross HBM. */
typedef struct {
    const spice_bf16 *w_router;         /* [N, d] bf16                                       */
    const uint8_t *slot_q_gate_up;      /* [S, 2I, d] E4M3: I gate rows, then I up rows      */
    const float *slot_s_gate_up;        /* [S, 2I] row scales                                */
    const uint8_t *slot_q_down;         /* [S, d, I] E4M3                                    */
    const float *slot_s_down;           /* [S, d]                                            */
    const int32_t *slot_of_expert;      /* [N]; slot index, or -1 when not resident          */
    const uint8_t *shared_q_gate_up;    /* [2 I_s, d] E4M3                                   */
    const float *shared_s_gate_up;      /* [2 I_s]                                           */
    const uint8_t *shared_q_down;       /* [d, I_s] E4M3                                     */
    const float *shared_s_down;         /* [d]                                               */
    const spice_bf16 *lore_A;           /* [N, r, d] bf16                                    */
    const spice_bf16 *lore_B;           /* [N, d, r] bf16                                    */
} spice_layer_weights_fp8;

/* Quantiser of that format: for each of `rows` rows of the bf16 matrix w [rows, cols] (cols a multiple of 8)
 *     scale[r] = 2^ceil(log2(max_j |w[r,j]| / 448))   (1 for an all-zero row),
 *     q[r,j]   = the E4M3 value nearest to w[r,j] / scale[r], ties to the even code, magnitudes above 448 saturate.
 * w, q [rows, cols] uint8 and scale [rows] fp32 are device pointers owned by the caller (q, scale: out; 16-byte aligned
 * w and q).  No ctx: the GPU is the calling thread's current device.  Any positive finite scales are accepted by the
 * layer call; the powers of two written here make the dequantised weights exact in fp32 (and in bf16). */
spice_status spice_quantize_e4m3_rows(const spice_bf16 *w, int64_t rows, int32_t cols, uint8_t *q, float *scale,
                                      void *stream);

/* spice_moe_layer_fwd at the 8-bit weight precision; every other argument, every output and every rule (top-k order,
 * classes, residual list, optional residual inputs) as there.  Covers decode batches: T <= 32, and d, inter and
 * inter_shared multiples of 128 (SPICE_ERR_UNSUPPORTED_SHAPE otherwise; there is no second kernel path behind it, and
 * SPICE_ERR_CUDA is returned when the device refuses the cooperative launch).  One launch: inside the kernel the input
 * activations and later the intermediate ones are written as the sum of three E5M2 terms (exact for bf16 magnitudes from
 * 2^-7 to 57344; smaller ones to 2^-17 absolute, larger ones saturate), and the tensor cores multiply E4M3 weights with
 * those terms (kind::f8f6f4), fp32 accumulation, row scale in the epilogue. */
spice_status spice_moe_layer_fwd_fp8(spice_ctx *ctx, const spice_layer_weights_fp8 *w /* host struct */,
                                     const spice_bf16 *h, const float *conf, int32_t T,
                                     const float *y_cpu_residual, spice_bf16 *x_resid, spice_bf16 *y,
                                     int32_t *idx, float *gate, uint8_t *cls, int32_t *counts,
                                     int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                                     float *resid_gate, void *stream);

/* The resident-expert FFN for callers that cannot allocate (the paper has no counterpart: this is
 * a packaging variant of spice_grouped_expert_ffn, not a step of the method).
 *
 * Every other call needs a spice_ctx, and spice_create obtains the workspace with cudaMalloc.  A
 * host that is not allowed to do that -- a server that gives each component a fixed arena and
 * forbids driver allocations after start-up, a process whose memory cap works by failing cudaMalloc
 * -- can use this entry point instead.  It needs no ctx and allocates nothing, on the host or on
 * the device: the scratch of the kernels (group table, permutation, activations, un-gated rows)
 * lives in one fixed device array of spice_static_scratch_bytes() = 8 MiB that every GPU loading
 * the library holds until the process exits.
 *
 *   y[t,:] += sum over k with cls[t,k] == HIT of gate[t,k] * E_{slot[t,k]}(h[t,:]),   y [T,d] fp32
 *
 * with the arguments of spice_grouped_expert_ffn; cfg is a host struct (only d, n_experts, top_k,
 * inter, n_slots are used), the GPU used is the calling thread's current device.
 *   device_status: optional device int32; receives SPICE_OK or SPICE_ERR_BAD_TABLE for this call.
 * Limits and behaviour:
 *   - A call needs about T*K*(inter + d)*4 bytes of the array (e.g. 96 (t,k) entries of a
 *     DeepSeek-V2-Lite-shaped layer: 1.3 MB).  A call that does not fit returns
 *     SPICE_ERR_WORKSPACE and launches nothing.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress, no
 *     allocation).  Make that first call before any stream capture is begun on the device.
 *   - All calls on a device share the array and it keeps the previous call's contents; what must
 *     start from zero is cleared by the call itself.  Two calls that overlap on the GPU (different
 *     streams, or different threads without ordering) race on it: keep them ordered. */
spice_status spice_grouped_expert_ffn_static(const spice_layer_cfg *cfg /* host */,
                                             const spice_layer_weights *w /* host struct */, const spice_bf16 *h,
                                             const int32_t *idx, const float *gate, const uint8_t *cls,
                                             const int32_t *slot, int32_t T, float *y, int32_t *device_status,
                                             void *stream);
size_t spice_static_scratch_bytes(void);

/* Synchronises the device work issued through ctx so far and returns the sticky device status
 * (SPICE_OK, SPICE_ERR_BAD_TABLE or SPICE_ERR_TIMEOUT) in *code (host), then clears it. */
spice_status spice_get_device_status(spice_ctx *ctx, int32_t *code /* host */);

/* Number of kernels the library has launched through ctx since it was created (host counter). */
spice_status spice_launch_count(const spice_ctx *ctx, int64_t *launches /* host */);

/* Knobs (host only).  SPICE_OPT_PATH: 0 = choose the kernel path by batch size (default),
 * 1 = always use the general-shape kernels, 2 = never use a fused decode kernel (tensor-core
 * grouped GEMM for the experts at any batch size), 3 = for small batches use the fused decode
 * kernel built on mma.sync instead of the tcgen05 one.  SPICE_OPT_SPIN_LIMIT: number of polls after which a
 * dependency wait inside the fused decode kernel gives up and reports SPICE_ERR_TIMEOUT
 * (default 2^20; a poll takes 0.1 to 1 us).  SPICE_OPT_TC_WAIT_LIMIT: the same for the pipeline waits (shared-memory
 * barriers between the copy, tensor-core and epilogue roles) of the grouped GEMM kernel that batches above 64 tokens
 * run on (default 2^22 polls).  A wait that gives up ends its thread block early: the call's outputs are then
 * undefined, SPICE_ERR_TIMEOUT is recorded in the status word, nothing stays in flight, and the next call on the
 * ctx starts clean (dependency counters are reset by the kernel that gave up; the status word stays set until
 * spice_get_device_status reads it). */
enum { SPICE_OPT_PATH = 0, SPICE_OPT_SPIN_LIMIT = 1, SPICE_OPT_TC_WAIT_LIMIT = 2 };
spice_status spice_set_option(spice_ctx *ctx, int32_t option, int64_t value);

/* Text for a status code (static storage, never NULL). */
const char *spice_status_string(spice_status s);

#ifdef __cplusplus
}
#endif
#endif /* SPICE_H_ */
