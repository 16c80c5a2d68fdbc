// Internal declarations shared by the translation units of libspice (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spice.h"

namespace spice {

constexpr int KIND_SHARED = 1;  // the fused shared expert, all T tokens
constexpr int KIND_HIT = 2;     // one resident slot and the (t,k) entries routed to it
constexpr int KIND_LOW = 4;     // one non-resident expert and its low-confidence entries

// One unit of grouped work: m rows that all use the same weight matrices.
struct GroupDesc {
    int32_t kind;  // KIND_*
    int32_t id;    // slot index (HIT), expert index (LOW), 0 (SHARED)
    int32_t off;   // first position in perm_hit / perm_low (0 for SHARED)
    int32_t m;     // number of rows
};

// Header words written by the grouping kernel.
enum { HDR_N_GROUPS = 0, HDR_N_HIT_GROUPS, HDR_N_LOW_GROUPS, HDR_N_HIT, HDR_N_LOW, HDR_WORDS = 8 };

// Device-side view of the per-call tables that live in the ctx workspace.
struct Tables {
    GroupDesc *groups;     // [1 + S + N]  group 0 is always the shared expert
    int32_t *hdr;          // [HDR_WORDS]
    int32_t *perm_hit;     // [Tm*K] entry ids (t*K+k) grouped by slot
    int32_t *perm_low;     // [Tm*K] entry ids grouped by expert
    int32_t *pos_of_entry; // [Tm*K] position of the entry in perm_hit / perm_low, -1 if none
    float *coef_shared;    // [Tm] 1 + sum of LOWCONF gates
    float *act_hit;        // [Tm*K, I]   silu(gate)*up of HIT entries, perm_hit order
    float *act_shared;     // [Tm, I_s]
    float *z_low;          // [Tm*K, r]   A_e h of LOWCONF entries, perm_low order
    float *part;           // [Tm*K, d]   down-projected row of entry t*K+k (un-gated)
    float *part_shared;    // [Tm, d]
    int32_t *status;       // sticky device status word
};

struct Dims {
    int32_t T, d, N, K, I, Is, r, S;
};

// ---- kernels launchers (each returns the number of kernels it launched, or -1 on launch error)
int launch_route_topk(const Dims &dm, int norm_topk, const __nv_bfloat16 *h, const __nv_bfloat16 *w_router,
                      int32_t *idx, float *gate, float *logits, cudaStream_t st);

// draft-router confidence: route with full-softmax gates, then the per-token sum and (optionally) the distribution
int launch_draft_confidence(const Dims &dm, const __nv_bfloat16 *h_hat, const __nv_bfloat16 *w_draft, int32_t *idx_hat,
                            float *gate_ws, float *logits_ws, float *pi_hat, float *conf, cudaStream_t st);

// scratch of the multi-CTA classify / group kernels (large batches); without it the single-CTA kernels run
struct GroupScratch {
    int32_t *cnt;        // [4096]: entries per slot [0,1024) and per expert [1024,2048), then the cursors [2048,4096)
    int32_t *off;        // [2048]: first position of each slot's / expert's group
    int32_t *blk_miss;   // [ceil(Tm*K / 1024)]: exact-recovery misses per chunk of 1024 entries
};

int launch_classify(const Dims &dm, int conf_stride, float tau, const int32_t *idx, const float *gate,
                    const int32_t *slot_of_expert, const float *conf, uint8_t *cls, int32_t *slot,
                    int32_t *counts, int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                    float *resid_gate, int32_t *status, cudaStream_t st, const GroupScratch *scratch = nullptr);

int launch_group(const Dims &dm, const int32_t *idx, const float *gate, const uint8_t *cls,
                 const int32_t *slot, const Tables &tb, cudaStream_t st, const GroupScratch *scratch = nullptr);

// classification and grouping of one call: one launch while a single CTA builds the tables, else the launches above
int launch_classify_group(const Dims &dm, int conf_stride, float tau, const int32_t *idx, const float *gate,
                          const int32_t *slot_of_expert, const float *conf, uint8_t *cls, int32_t *slot, int32_t *counts,
                          int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert, float *resid_gate, const Tables &tb,
                          cudaStream_t st, const GroupScratch *scratch = nullptr);

// Reference ("v1") expert path: warp-per-row GEMV kernels for any shape.
int launch_gateup(const Dims &dm, int kind_mask, const spice_layer_weights &w, const __nv_bfloat16 *h,
                  const Tables &tb, cudaStream_t st);
int launch_lore_a(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                  cudaStream_t st);
int launch_down(const Dims &dm, int kind_mask, const spice_layer_weights &w, const Tables &tb, cudaStream_t st);
int launch_lore_b(const Dims &dm, const spice_layer_weights &w, const Tables &tb, int z_after_hits, cudaStream_t st);   // LOW groups only

struct CombineArgs {
    int kind_mask;              // which terms enter
    int accumulate;             // 1: y32 += ..., 0: y = ...
    const float *gate;          // [T,K]
    const uint8_t *cls;         // [T,K]
    float *y32;                 // fp32 output / accumulator or NULL
    __nv_bfloat16 *y16;         // bf16 output or NULL
    const float *y_cpu;         // optional fp32 addend
    __nv_bfloat16 *x_resid;     // optional bf16 in/out residual stream
    int shared_coef_low_sum;    // 1: the shared expert enters with sum of LOWCONF gates (no "1 +"): rollout projection
    int hit_rows_gated16;       // 1: rows of HIT entries in tb.part are bf16 and already multiplied by their gate
};
int launch_combine(const Dims &dm, const CombineArgs &a, const Tables &tb, cudaStream_t st);

// ---- speculative prefetch rollout, Algorithm 1 (rollout.cu); w: host array of l_max structs
int launch_rollout(const Dims &dm, const spice_layer_weights *w, int l_min, int l_max, float tau, __nv_bfloat16 *h_state,
                   __nv_bfloat16 *y_scratch, int32_t *idx_ws, float *gate_ws, uint8_t *cls_ws, float *conf_ws, float *logits_ws,
                   int32_t *active_ws, const Tables &tb, int32_t *idx_hat, float *conf, int32_t *depth, cudaStream_t st);

int launch_prefetch_set(const Dims &dm, int l_max, const int32_t *idx_hat, uint8_t *mask, cudaStream_t st);
int launch_rollout_mask(const Dims &dm, int depth, int l_min, int l_max, float tau, const float *conf_l, int32_t *active,
                        const int32_t *idx_ws, int32_t *idx_out, float *conf_out, uint8_t *cls, int32_t *depth_out,
                        cudaStream_t st);

// ---- LoRE calibration (calibrate.cu): closed-form rank-r fit of the residual E(h) - S(h) over calibration tokens
size_t lore_calibrate_workspace_bytes(int d, int n, int r);
int launch_lore_calibrate(int d, int n, int r, float ridge, int iters, const __nv_bfloat16 *h_cal, const float *resid,
                          __nv_bfloat16 *A_out, __nv_bfloat16 *B_out, float *loss_out, int32_t *flag, void *workspace,
                          cudaStream_t st);

// ---- fused decode kernel (decode.cu)
// words of the dependency-counter array
enum { SY_ABORT = 0, SY_TEAMS_DONE, SY_R1_DONE, SY_ROUTE_DONE, SY_P2_DONE, SY_P1_ALL, SY_NEXT_TASK, SY_H8_DONE, SY_GROUP0 = 8 };

struct DecodeParams {
    Dims dm;
    int32_t norm_topk, conf_stride;
    float tau;
    int32_t n_r1;         // router tasks
    int32_t spin_limit;   // iterations after which a dependency wait gives up
    int32_t sync_words;   // length of sync[]
    const __nv_bfloat16 *h;
    const float *conf;
    spice_layer_weights w;
    int32_t *idx;
    float *gate;
    uint8_t *cls;
    int32_t *counts;
    int32_t *resid_tok, *resid_k, *resid_expert;
    float *resid_gate;
    // the context's own [Tm*K] arrays: where the tcgen05 decode kernel exchanges the routing of a batch that it spreads
    // over the grid (the caller's idx / gate / cls may be mapped host memory and are only ever written)
    int32_t *x_idx;
    float *x_gate;
    uint8_t *x_cls;
    __nv_bfloat16 *y16;
    const float *y_cpu;
    __nv_bfloat16 *x_resid;
    Tables tb;
    float *logits;                 // [T,N]
    __nv_bfloat16 *act_hit16;      // [Tm*K, I]  perm_hit order
    __nv_bfloat16 *act_shared16;   // [Tm, I_s]
    __nv_bfloat16 *z16;            // [Tm*K, r]  perm_low order
    int32_t *sync;                 // [sync_words] zero between launches
    // Rollout mode of the tcgen05 decode kernel (Algorithm 1, one depth per launch; 0 = ordinary layer call): the
    // classes come from the halting rule instead of residency and confidences -- every selected expert of a token that
    // continues is a low-confidence miss, nothing is added for a token that stops -- and the shared expert is weighted
    // by the sum of the gates alone.
    int32_t roll_depth, roll_l_min;
    float roll_tau;
    const int32_t *roll_active_in;   // [T] 1 while the token still speculates (ignored at depth 1)
    int32_t *roll_active_out;        // [T] the same after this depth
    int32_t *roll_idx_out;           // [T,K] predicted set of this depth, -1 for tokens that stopped earlier
    float *roll_conf_out;            // [T]
    int32_t *roll_depth_out;         // [T]
};
size_t decode_smem_bytes(const Dims &dm);
bool decode_supported(const Dims &dm, size_t max_smem);
int decode_prepare(int max_smem_optin);
int launch_decode(const DecodeParams &p, int n_ctas, cudaStream_t st);

// ---- fused decode kernel on tcgen05 / TMA (decode_tc.cu); shares DecodeParams and the counter words
// The layer at the 8-bit weight precision: E4M3 codes and fp32 row scales of the expert matrices (layouts of
// spice_layer_weights_fp8), and the ctx buffers that hold activations as three E5M2 planes.
struct Fp8Layer {
    const uint8_t *q_slot_gu, *q_slot_d, *q_sh_gu, *q_sh_d;
    const float *s_slot_gu, *s_slot_d, *s_sh_gu, *s_sh_d;
    uint8_t *x8_h;       // [3][T][d]
    uint8_t *act8_hit;   // [group][3][T][I]
    uint8_t *act8_sh;    // [3][T][Is]
};
bool decode_tc_supported(const Dims &dm, int conf_stride, size_t max_smem, bool f8 = false);
int decode_tc_nsplit(const Dims &dm, bool f8 = false);   // K ranges of the shared expert's down projection (rows of part_split)
int decode_tc_prepare(int max_smem_optin);
int launch_decode_tc(const DecodeParams &p, float *part_split, int n_ctas, int max_smem_optin, cudaStream_t st,
                     const Fp8Layer *f8 = nullptr);

// ---- 8-bit formats (fp8.cu)
// per-row power-of-two scale and E4M3 codes of a bf16 matrix [rows, cols]
int launch_quantize_e4m3_rows(const __nv_bfloat16 *w, size_t rows, int cols, uint8_t *q, float *scale, cudaStream_t st);


// ---- tensor-core path for large batches (tc_gemm.cu)
// One m-tile of the grouped problem: rows [row0, row0+rows) of the gathered activation buffer, all of
// which use the weights of slot `slot`.
struct MTile {
    int32_t slot, row0, rows, pad;
};
struct TcBuffers {
    __nv_bfloat16 *x_perm;        // [Tm*K, d]   tokens gathered in perm_hit order
    __nv_bfloat16 *act16;         // [Tm*K, I]   silu(gate)*up of HIT entries
    __nv_bfloat16 *act_shared16;  // [Tm, I_s]
    MTile *mtiles, *mtiles_shared, *mtiles_low;   // tile lists: routed (also the router's), shared expert, LOW groups
    int32_t *n_mtiles, *n_mtiles_shared, *n_mtiles_low;
    int32_t *status;              // sticky device status word of the ctx
    uint32_t wait_limit;          // polls after which a pipeline wait of the GEMM kernel gives up (0: the default)
};
bool tc_available();
int tc_prepare();
bool tc_shape_ok(const Dims &dm);
// gate16 != NULL: the down projection writes gate[entry] * row as bf16 into the first half of the entry's row of tb.part
// (CombineArgs::hit_rows_gated16 tells the combine); NULL: plain fp32 rows
int launch_tc_routed(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                     const TcBuffers &b, int n_sms, cudaStream_t st, const float *gate16 = nullptr);
int launch_tc_shared(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                     const TcBuffers &b, int n_sms, cudaStream_t st);
// out[M,N] fp32 (ld) = A[M,K] B[N,K]^T on the tensor cores; bf16 operands with row pitch ldk (multiple of 8, zero padded)
int launch_tc_plain(const __nv_bfloat16 *A, int M, const __nv_bfloat16 *B, int N, int K, int ldk, float *out, int ld, MTile *mtiles,
                    int32_t *n_mtiles, int n_sms, cudaStream_t st);
// the same cut into n_split ranges of k_split reduction elements; partial results at out + s * M * ld (tile list built once)
int launch_tc_splitk_tiles(int M, int n_split, MTile *mtiles, int32_t *n_mtiles, cudaStream_t st);
int launch_tc_plain_splitk(const __nv_bfloat16 *A, int M, const __nv_bfloat16 *B, int N, int k_split, int ldk, float *out, int ld,
                           const MTile *mtiles, const int32_t *n_mtiles, int n_sms, cudaStream_t st);
// router logits of a large batch as a GEMM, then Top-K from the stored logits (route.cu)
bool tc_router_ok(const Dims &dm);
int launch_tc_router_logits(const Dims &dm, const __nv_bfloat16 *h, const __nv_bfloat16 *w_router, float *logits,
                            const TcBuffers &b, int n_sms, cudaStream_t st);
// LoRE of a large batch: z = A_e h through the GEMM kernel (rows n_hit + p of tb.z_low), then lore_b_kernel
bool tc_lore_ok(const Dims &dm);
int launch_tc_lore_a(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb, const TcBuffers &b,
                     int n_sms, cudaStream_t st);
int launch_topk_from_logits(const Dims &dm, int norm_topk, const float *logits, int32_t *idx, float *gate, cudaStream_t st);

// ---- small device helpers
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// bf16 pair packed in a 32-bit word -> two fp32 (exact)
__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

__device__ __forceinline__ uint4 ldg_stream(const void *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + __expf(-v)); }

}  // namespace spice
