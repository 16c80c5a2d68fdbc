// Router logits, Top-K and gate scores (Eq. 1 of the paper; "selected experts and their gate
// scores", Sec. 4.2).  One CTA owns TPC tokens: its warps share the router rows (each warp takes a
// few experts at a time), logits are accumulated in fp32 in a fixed order and parked in shared
// memory, then one warp per token selects the K winners (ties -> smaller expert index).
#include "route_device.cuh"
#include "spice_internal.cuh"

namespace spice {

template <int TPC>
__global__ void route_topk_kernel(const __nv_bfloat16 *__restrict__ h, const __nv_bfloat16 *__restrict__ wr,
                                  int T, int d, int N, int K, int norm_topk, int32_t *__restrict__ idx,
                                  float *__restrict__ gate, float *__restrict__ logits_out) {
    extern __shared__ __align__(16) float smem[];
    float *hs = smem;                   // [TPC][d] fp32 copy of the tokens
    float *lg = smem + (size_t)TPC * d; // [TPC][N]
    float *sel_val = lg + (size_t)TPC * N;                       // [nwarps][32]
    int *sel_idx = reinterpret_cast<int *>(sel_val + 32 * 32);   // [nwarps][32]
    const int t0 = blockIdx.x * TPC;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;

    // stage the tokens (8 bf16 per thread-step), zero rows past T
    for (int v = threadIdx.x; v < TPC * (d >> 3); v += blockDim.x) {
        int tt = v / (d >> 3), c = v - tt * (d >> 3);
        uint4 u = make_uint4(0, 0, 0, 0);
        if (t0 + tt < T) u = *reinterpret_cast<const uint4 *>(h + (size_t)(t0 + tt) * d + c * 8);
        float *dst = hs + (size_t)tt * d + c * 8;
        reinterpret_cast<float4 *>(dst)[0] = make_float4(bf_lo(u.x), bf_hi(u.x), bf_lo(u.y), bf_hi(u.y));
        reinterpret_cast<float4 *>(dst)[1] = make_float4(bf_lo(u.z), bf_hi(u.z), bf_lo(u.w), bf_hi(u.w));
    }
    __syncthreads();

    // Each warp takes EPW experts at a time so that every token slice read from shared memory feeds
    // EPW fmaf chains; per (expert, token) the arithmetic is exactly lane_dot_f32's.
    constexpr int EPW = (TPC >= 4) ? 4 : 1;
    for (int e0 = warp * EPW; e0 < N; e0 += nwarps * EPW) {
        float acc[EPW][TPC];
#pragma unroll
        for (int ee = 0; ee < EPW; ++ee)
#pragma unroll
            for (int tt = 0; tt < TPC; ++tt) acc[ee][tt] = 0.f;
        for (int k = lane * 8; k < d; k += 256) {
            uint4 u[EPW];
#pragma unroll
            for (int ee = 0; ee < EPW; ++ee)
                u[ee] = (e0 + ee < N) ? *reinterpret_cast<const uint4 *>(wr + (size_t)(e0 + ee) * d + k) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int tt = 0; tt < TPC; ++tt) {
                const float4 a = *reinterpret_cast<const float4 *>(hs + (size_t)tt * d + k);
                const float4 b = *reinterpret_cast<const float4 *>(hs + (size_t)tt * d + k + 4);
#pragma unroll
                for (int ee = 0; ee < EPW; ++ee) acc[ee][tt] += slice_dot(u[ee], a, b);
            }
        }
#pragma unroll
        for (int ee = 0; ee < EPW; ++ee)
#pragma unroll
            for (int tt = 0; tt < TPC; ++tt) {
                const float s = warp_sum(acc[ee][tt]);
                if (lane == 0 && e0 + ee < N) lg[tt * N + e0 + ee] = s;
            }
    }
    __syncthreads();

    for (int tt = warp; tt < TPC; tt += nwarps) {
        const int t = t0 + tt;
        if (t >= T) continue;   // warp-uniform
        if (N <= 256)
            warp_topk_gates(lg + tt * N, N, K, norm_topk, lane, idx + (size_t)t * K, gate + (size_t)t * K,
                            logits_out ? logits_out + (size_t)t * N : nullptr, sel_idx + warp * 32, sel_val + warp * 32);
        else
            warp_topk_gates_rounds(lg + tt * N, N, K, norm_topk, lane, idx + (size_t)t * K, gate + (size_t)t * K,
                                   logits_out ? logits_out + (size_t)t * N : nullptr);
    }
}

// Draft-router confidence (Sec. 4.1, Eq. 5) from the logits, winners and full-softmax gates that
// route_topk_kernel produced with norm_topk = 0: conf[t] = sum of the K gates in k order; optionally the whole
// distribution pi_hat = exp(l - l_max) / denom, with the denominator summed exactly as the gates' was
// (lane-strided partial sums, xor-shuffle tree), so pi_hat[t, idx[t,k]] equals gate[t,k] bit for bit.
// One warp per token; lp holds the logits on entry and, when pi_out == lp, the distribution on exit.
__global__ void __launch_bounds__(256) draft_confidence_kernel(const float *lp, const int32_t *__restrict__ idx,
                                                               const float *__restrict__ gate, int T, int N, int K,
                                                               float *pi_out, float *__restrict__ conf) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= T) return;   // warp-uniform
    if (lane == 0) {
        float c = 0.f;
        for (int k = 0; k < K; ++k) c += gate[(size_t)t * K + k];
        conf[t] = c;
    }
    if (!pi_out) return;
    const float *l = lp + (size_t)t * N;
    float m = l[idx[(size_t)t * K]];
    if (!(m == m)) m = -INFINITY;
    float s = 0.f;
#pragma unroll 1
    for (int e = lane; e < N; e += 32) s += expf(l[e] - m);
    const float denom = warp_sum(s);
    __syncwarp();   // every lane has read its logits before the row is overwritten in place
#pragma unroll 1
    for (int e = lane; e < N; e += 32) pi_out[(size_t)t * N + e] = expf(l[e] - m) / denom;
}

// Top-K and gates from logits that another kernel left in global memory ([T, N] fp32): one warp per token, the row
// is copied to shared memory first.  Used for large batches, whose logits come from the tensor cores.
__global__ void __launch_bounds__(256) topk_from_logits_kernel(const float *__restrict__ logits, int T, int N, int K, int norm_topk,
                                                               int32_t *__restrict__ idx, float *__restrict__ gate) {
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    float *row = smem + (size_t)warp * N;
    float *sel_val = smem + (size_t)nwarps * N + warp * 32;
    int *sel_idx = reinterpret_cast<int *>(smem + (size_t)nwarps * N + nwarps * 32) + warp * 32;
    const int t = blockIdx.x * nwarps + warp;
    if (t >= T) return;   // warp-uniform; no block-wide barrier below
#pragma unroll 1
    for (int e = lane; e < N; e += 32) row[e] = logits[(size_t)t * N + e];
    __syncwarp();
    if (N <= 256) warp_topk_gates(row, N, K, norm_topk, lane, idx + (size_t)t * K, gate + (size_t)t * K, nullptr, sel_idx, sel_val);
    else warp_topk_gates_rounds(row, N, K, norm_topk, lane, idx + (size_t)t * K, gate + (size_t)t * K, nullptr);
}

int launch_topk_from_logits(const Dims &dm, int norm_topk, const float *logits, int32_t *idx, float *gate, cudaStream_t st) {
    const int nwarps = 8;
    const size_t smem = ((size_t)nwarps * dm.N + 2 * nwarps * 32) * sizeof(float);
    if (smem > 48 * 1024) return -1;
    topk_from_logits_kernel<<<(dm.T + nwarps - 1) / nwarps, nwarps * 32, smem, st>>>(logits, dm.T, dm.N, dm.K, norm_topk, idx, gate);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_draft_confidence(const Dims &dm, const __nv_bfloat16 *h_hat, const __nv_bfloat16 *w_draft, int32_t *idx_hat,
                            float *gate_ws, float *logits_ws, float *pi_hat, float *conf, cudaStream_t st) {
    // logits land in pi_hat when the caller wants the distribution (converted in place), else in the workspace
    float *lp = pi_hat ? pi_hat : logits_ws;
    int n = launch_route_topk(dm, /*norm_topk=*/0, h_hat, w_draft, idx_hat, gate_ws, lp, st);
    if (n < 0) return -1;
    const int wpb = 8;
    draft_confidence_kernel<<<(dm.T + wpb - 1) / wpb, wpb * 32, 0, st>>>(lp, idx_hat, gate_ws, dm.T, dm.N, dm.K, pi_hat, conf);
    return cudaGetLastError() == cudaSuccess ? n + 1 : -1;
}

template <int TPC>
static int launch_tpc(const Dims &dm, int norm_topk, const __nv_bfloat16 *h, const __nv_bfloat16 *w_router,
                      int32_t *idx, float *gate, float *logits, int threads, cudaStream_t st) {
    size_t smem = ((size_t)TPC * dm.d + (size_t)TPC * dm.N + 2 * 32 * 32) * sizeof(float);
    if (smem > 220 * 1024) return -1;
    if (cudaFuncSetAttribute(route_topk_kernel<TPC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return -1;
    int grid = (dm.T + TPC - 1) / TPC;
    route_topk_kernel<TPC><<<grid, threads, smem, st>>>(h, w_router, dm.T, dm.d, dm.N, dm.K, norm_topk, idx, gate,
                                                        logits);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_route_topk(const Dims &dm, int norm_topk, const __nv_bfloat16 *h, const __nv_bfloat16 *w_router,
                      int32_t *idx, float *gate, float *logits, cudaStream_t st) {
    // few tokens: one token per CTA with many warps across the experts;
    // many tokens: several tokens per CTA share each router row read.
    if (dm.T <= 64) return launch_tpc<1>(dm, norm_topk, h, w_router, idx, gate, logits, dm.N >= 32 ? 1024 : 256, st);
    if ((size_t)8 * (dm.d + dm.N) * sizeof(float) <= 160 * 1024)
        return launch_tpc<8>(dm, norm_topk, h, w_router, idx, gate, logits, 256, st);
    if ((size_t)2 * (dm.d + dm.N) * sizeof(float) <= 200 * 1024)
        return launch_tpc<2>(dm, norm_topk, h, w_router, idx, gate, logits, 256, st);
    return launch_tpc<1>(dm, norm_topk, h, w_router, idx, gate, logits, 256, st);
}

}  // namespace spice
