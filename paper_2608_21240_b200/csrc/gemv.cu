// General-shape expert path: warp-per-row GEMV kernels with 128-bit bf16 weight loads and fp32
// accumulation, for any token count and any dimensions that are multiples of 8.
//   gate/up + SwiGLU   a = silu(W_g x) * (W_u x)            exact expert E_e of Sec. 4.2 (and shared S)
//   LoRE down-project  z = A_e x                            Delta_e(h) = B_e A_e h, Sec. 4.2
//   down-projection    part = W_d a   (or B_e z)            un-gated rows, one per (t,k) entry
//   combine            y_t = c_t * S(h_t) + sum_k g_k part  weighted aggregation of Sec. 2.1 with the
//                                                            surrogate substituted as in Sec. 4.2
// A CTA owns (group, block of output rows); it walks the group's rows MT tokens at a time and the
// reduction dimension KC elements at a time, with the token chunk staged in shared memory as fp32.
#include "spice_internal.cuh"

namespace spice {

constexpr int GT = 256;        // threads per CTA
constexpr int GW = GT / 32;    // warps
constexpr int MT = 4;          // tokens per pass
constexpr int KC = 2048;       // reduction chunk (elements)

__device__ __forceinline__ void fma8(const uint4 u, const float *x, float &acc) {
    const float4 a = *reinterpret_cast<const float4 *>(x);
    const float4 b = *reinterpret_cast<const float4 *>(x + 4);
    float s = acc;
    s = fmaf(bf_lo(u.x), a.x, s); s = fmaf(bf_hi(u.x), a.y, s);
    s = fmaf(bf_lo(u.y), a.z, s); s = fmaf(bf_hi(u.y), a.w, s);
    s = fmaf(bf_lo(u.z), b.x, s); s = fmaf(bf_hi(u.z), b.y, s);
    s = fmaf(bf_lo(u.w), b.z, s); s = fmaf(bf_hi(u.w), b.w, s);
    acc = s;
}

// stage xs[m][0..len) for the mt tokens of this pass; rows >= mt are zero-filled
template <bool SRC_BF16>
__device__ __forceinline__ void stage_chunk(float *xs, const void *const *rows /* smem [MT] */, int mt, int k0,
                                            int len) {
    const int vec = len >> 3;
    for (int v = threadIdx.x; v < MT * vec; v += GT) {
        const int m = v / vec, c = v - m * vec;
        float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
        if (m < mt) {
            if (SRC_BF16) {
                const uint4 u = *reinterpret_cast<const uint4 *>(static_cast<const __nv_bfloat16 *>(rows[m]) + k0 + c * 8);
                lo = make_float4(bf_lo(u.x), bf_hi(u.x), bf_lo(u.y), bf_hi(u.y));
                hi = make_float4(bf_lo(u.z), bf_hi(u.z), bf_lo(u.w), bf_hi(u.w));
            } else {
                const float *p = static_cast<const float *>(rows[m]) + k0 + c * 8;
                lo = *reinterpret_cast<const float4 *>(p);
                hi = *reinterpret_cast<const float4 *>(p + 4);
            }
        }
        reinterpret_cast<float4 *>(xs + (size_t)m * KC + c * 8)[0] = lo;
        reinterpret_cast<float4 *>(xs + (size_t)m * KC + c * 8)[1] = hi;
    }
}

// ---------------------------------------------------------------------------------------------
// MODE 0: gate/up + SwiGLU (SHARED and HIT groups);  MODE 1: plain rows z = A x (LOW groups)
template <int MODE>
__global__ void __launch_bounds__(GT) rows_from_h_kernel(Dims dm, int kind_mask, spice_layer_weights w,
                                                         const __nv_bfloat16 *__restrict__ h, Tables tb) {
    __shared__ __align__(16) float xs[MT * KC];
    __shared__ const void *rows[MT];
    // when only the low-confidence groups are wanted they are addressed directly (they follow the hit groups)
    const int g = blockIdx.y + (kind_mask == KIND_LOW ? 1 + tb.hdr[HDR_N_HIT_GROUPS] : 0);
    if (g >= tb.hdr[HDR_N_GROUPS]) return;
    const GroupDesc grp = tb.groups[g];
    if (!(grp.kind & kind_mask)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = dm.d;
    int n_out;                      // output rows of this group (I, I_s or r)
    const __nv_bfloat16 *W0, *W1;   // row i of W0 (and of W1 for gate/up)
    float *out;                     // out[(p)*n_out + i]
    const int32_t *perm = nullptr;
    if (MODE == 0) {
        if (grp.kind == KIND_SHARED) {
            n_out = dm.Is;
            W0 = reinterpret_cast<const __nv_bfloat16 *>(w.shared_w_gate_up);
            out = tb.act_shared;
        } else {
            n_out = dm.I;
            W0 = reinterpret_cast<const __nv_bfloat16 *>(w.slot_w_gate_up) + (size_t)grp.id * 2 * dm.I * d;
            out = tb.act_hit + (size_t)grp.off * dm.I;
            perm = tb.perm_hit + grp.off;
        }
        W1 = W0 + (size_t)n_out * d;
    } else {
        n_out = dm.r;
        W0 = reinterpret_cast<const __nv_bfloat16 *>(w.lore_A) + (size_t)grp.id * dm.r * d;
        W1 = W0;
        out = tb.z_low + (size_t)grp.off * dm.r;
        perm = tb.perm_low + grp.off;
    }
    const int i = blockIdx.x * GW + warp;   // this warp's output row
    if (blockIdx.x * GW >= n_out) return;
    const bool active = i < n_out;
    const __nv_bfloat16 *r0 = W0 + (size_t)(active ? i : 0) * d;
    const __nv_bfloat16 *r1 = W1 + (size_t)(active ? i : 0) * d;

    for (int p0 = 0; p0 < grp.m; p0 += MT) {
        const int mt = min(MT, grp.m - p0);
        __syncthreads();
        if (threadIdx.x < MT) {
            const int p = p0 + threadIdx.x;
            int t = 0;
            if (p < grp.m) t = perm ? perm[p] / dm.K : p;
            rows[threadIdx.x] = h + (size_t)t * d;
        }
        float ag[MT], au[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) ag[m] = au[m] = 0.f;
        for (int k0 = 0; k0 < d; k0 += KC) {
            const int len = min(KC, d - k0);
            __syncthreads();
            stage_chunk<true>(xs, rows, mt, k0, len);
            __syncthreads();
            if (active) {
                for (int k = lane * 8; k < len; k += 256) {
                    const uint4 ug = ldg_stream(r0 + k0 + k);
                    uint4 uu = ug;
                    if (MODE == 0) uu = ldg_stream(r1 + k0 + k);
#pragma unroll
                    for (int m = 0; m < MT; ++m) {
                        fma8(ug, xs + (size_t)m * KC + k, ag[m]);
                        if (MODE == 0) fma8(uu, xs + (size_t)m * KC + k, au[m]);
                    }
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float sg = warp_sum(ag[m]);
            const float su = (MODE == 0) ? warp_sum(au[m]) : 0.f;
            if (active && lane == 0 && m < mt) {
                const float v = (MODE == 0) ? silu_f(sg) * su : sg;
                out[(size_t)(p0 + m) * n_out + i] = v;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// down-projection of every group: part[row, j] = sum_i W[j,i] * a[p,i]
__global__ void __launch_bounds__(GT) down_kernel(Dims dm, int kind_mask, spice_layer_weights w, Tables tb) {
    __shared__ __align__(16) float xs[MT * KC];
    __shared__ const void *rows[MT];
    __shared__ float *outs[MT];
    const int g = blockIdx.y + (kind_mask == KIND_LOW ? 1 + tb.hdr[HDR_N_HIT_GROUPS] : 0);
    if (g >= tb.hdr[HDR_N_GROUPS]) return;
    const GroupDesc grp = tb.groups[g];
    if (!(grp.kind & kind_mask)) return;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int d = dm.d;
    int kd;                      // reduction length (I_s, I or r)
    const __nv_bfloat16 *W;      // [d, kd]
    const float *src;            // [m, kd]
    const int32_t *perm = nullptr;
    if (grp.kind == KIND_SHARED) {
        kd = dm.Is;
        W = reinterpret_cast<const __nv_bfloat16 *>(w.shared_w_down);
        src = tb.act_shared;
    } else if (grp.kind == KIND_HIT) {
        kd = dm.I;
        W = reinterpret_cast<const __nv_bfloat16 *>(w.slot_w_down) + (size_t)grp.id * d * dm.I;
        src = tb.act_hit + (size_t)grp.off * dm.I;
        perm = tb.perm_hit + grp.off;
    } else {
        kd = dm.r;
        W = reinterpret_cast<const __nv_bfloat16 *>(w.lore_B) + (size_t)grp.id * d * dm.r;
        src = tb.z_low + (size_t)grp.off * dm.r;
        perm = tb.perm_low + grp.off;
    }
    const int j = blockIdx.x * GW + warp;
    const bool active = j < d;
    const __nv_bfloat16 *r0 = W + (size_t)(active ? j : 0) * kd;

    for (int p0 = 0; p0 < grp.m; p0 += MT) {
        const int mt = min(MT, grp.m - p0);
        __syncthreads();
        if (threadIdx.x < MT) {
            const int p = min(p0 + (int)threadIdx.x, grp.m - 1);
            rows[threadIdx.x] = src + (size_t)p * kd;
            outs[threadIdx.x] = perm ? tb.part + (size_t)perm[p] * d : tb.part_shared + (size_t)p * d;
        }
        float acc[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0.f;
        for (int k0 = 0; k0 < kd; k0 += KC) {
            const int len = min(KC, kd - k0);
            __syncthreads();
            stage_chunk<false>(xs, rows, mt, k0, len);
            __syncthreads();
            if (active) {
                for (int k = lane * 8; k < len; k += 256) {
                    const uint4 u = ldg_stream(r0 + k0 + k);
#pragma unroll
                    for (int m = 0; m < MT; ++m) fma8(u, xs + (size_t)m * KC + k, acc[m]);
                }
            }
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            const float s = warp_sum(acc[m]);
            if (active && lane == 0 && m < mt) outs[m][j] = s;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// y_t = [y_t +] c_t * part_shared_t + sum_k g_k * part_{t,k} [+ y_cpu_t]; optional residual stream
__global__ void __launch_bounds__(256) combine_kernel(Dims dm, CombineArgs a, Tables tb) {
    const int t = blockIdx.y;
    const int j = (blockIdx.x * 256 + threadIdx.x) * 4;
    if (j >= dm.d) return;
    const int d = dm.d, K = dm.K;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (a.accumulate) acc = *reinterpret_cast<const float4 *>(a.y32 + (size_t)t * d + j);
    if (a.kind_mask & KIND_SHARED) {
        float c = tb.coef_shared[t];
        if (a.shared_coef_low_sum) {   // sum of the LOWCONF gates alone, in k order
            c = 0.f;
            for (int k = 0; k < K; ++k)
                if (a.cls[t * K + k] == SPICE_LOWCONF) c += a.gate[t * K + k];
        }
        const float4 s = *reinterpret_cast<const float4 *>(tb.part_shared + (size_t)t * d + j);
        acc.x = fmaf(c, s.x, acc.x); acc.y = fmaf(c, s.y, acc.y);
        acc.z = fmaf(c, s.z, acc.z); acc.w = fmaf(c, s.w, acc.w);
    }
    for (int k = 0; k < K; ++k) {
        const int i = t * K + k;
        const int c = a.cls[i];
        const bool use = (c == SPICE_HIT && (a.kind_mask & KIND_HIT)) || (c == SPICE_LOWCONF && (a.kind_mask & KIND_LOW));
        if (!use || tb.pos_of_entry[i] < 0) continue;
        if (a.hit_rows_gated16 && c == SPICE_HIT) {   // gate applied by the producer, bf16 row in the fp32 row's first half
            const uint2 u = *reinterpret_cast<const uint2 *>(reinterpret_cast<const __nv_bfloat16 *>(tb.part + (size_t)i * d) + j);
            acc.x += bf_lo(u.x); acc.y += bf_hi(u.x);
            acc.z += bf_lo(u.y); acc.w += bf_hi(u.y);
            continue;
        }
        const float g = a.gate[i];
        const float4 s = *reinterpret_cast<const float4 *>(tb.part + (size_t)i * d + j);
        acc.x = fmaf(g, s.x, acc.x); acc.y = fmaf(g, s.y, acc.y);
        acc.z = fmaf(g, s.z, acc.z); acc.w = fmaf(g, s.w, acc.w);
    }
    if (a.y_cpu) {
        const float4 s = *reinterpret_cast<const float4 *>(a.y_cpu + (size_t)t * d + j);
        acc.x += s.x; acc.y += s.y; acc.z += s.z; acc.w += s.w;
    }
    if (a.y32) *reinterpret_cast<float4 *>(a.y32 + (size_t)t * d + j) = acc;
    if (a.y16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
        *reinterpret_cast<uint2 *>(a.y16 + (size_t)t * d + j) = pk;
    }
    if (a.x_resid) {
        uint2 xr = *reinterpret_cast<const uint2 *>(a.x_resid + (size_t)t * d + j);
        __nv_bfloat162 lo = __floats2bfloat162_rn(bf_lo(xr.x) + acc.x, bf_hi(xr.x) + acc.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(bf_lo(xr.y) + acc.z, bf_hi(xr.y) + acc.w);
        uint2 pk = make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
        *reinterpret_cast<uint2 *>(a.x_resid + (size_t)t * d + j) = pk;
    }
}

// ---------------------------------------------------------------------------------------------
// LoRE up-projection alone (LOW groups only): part[entry, j] = sum_k B_e[j,k] z[p,k].  The reduction is only r long,
// so a warp per output row would leave most lanes idle; here a THREAD owns output column j, streams its row of B_e
// (r bf16) and applies it to LB tokens at a time whose z rows sit in shared memory (all threads read the same word:
// a broadcast).  Groups are walked with a stride, so a launch that finds no LOW group costs a few small CTAs.
constexpr int LB = 8;        // tokens per pass
constexpr int LB_GROUPS = 32;

__global__ void __launch_bounds__(256) lore_b_kernel(Dims dm, spice_layer_weights w, Tables tb, int z_after_hits) {
    extern __shared__ __align__(16) float zs[];   // [LB][r]
    const int r = dm.r, d = dm.d;
    const int j = blockIdx.x * 256 + threadIdx.x;
    const int first = 1 + tb.hdr[HDR_N_HIT_GROUPS], n_groups = tb.hdr[HDR_N_GROUPS];
    for (int g = first + blockIdx.y; g < n_groups; g += gridDim.y) {
        const GroupDesc grp = tb.groups[g];
        if (grp.kind != KIND_LOW) continue;   // (uniform)
        const __nv_bfloat16 *row = reinterpret_cast<const __nv_bfloat16 *>(w.lore_B) + ((size_t)grp.id * d + (j < d ? j : 0)) * r;
        // (z rows are numbered like the low entries, or behind the hit entries when the GEMM path produced them)
        const float *z = tb.z_low + (size_t)(grp.off + (z_after_hits ? tb.hdr[HDR_N_HIT] : 0)) * r;
        const int32_t *perm = tb.perm_low + grp.off;
        for (int p0 = 0; p0 < grp.m; p0 += LB) {
            const int mt = min(LB, grp.m - p0);
            __syncthreads();
            for (int v = threadIdx.x; v < LB * r; v += 256) zs[v] = v < mt * r ? z[(size_t)p0 * r + v] : 0.f;
            __syncthreads();
            float acc[LB];
#pragma unroll
            for (int m = 0; m < LB; ++m) acc[m] = 0.f;
            if (j < d) {
#pragma unroll 2
                for (int k = 0; k < r; k += 8) {
                    const uint4 u = *reinterpret_cast<const uint4 *>(row + k);
#pragma unroll
                    for (int m = 0; m < LB; ++m) fma8(u, zs + m * r + k, acc[m]);
                }
#pragma unroll
                for (int m = 0; m < LB; ++m)
                    if (m < mt) tb.part[(size_t)perm[p0 + m] * d + j] = acc[m];
            }
        }
    }
}

static inline int max_groups(const Dims &dm) {
    const int n = dm.T * dm.K;
    return 1 + min(dm.S, n) + min(dm.N, n);
}

int launch_gateup(const Dims &dm, int kind_mask, const spice_layer_weights &w, const __nv_bfloat16 *h,
                  const Tables &tb, cudaStream_t st) {
    const int rows = max((kind_mask & KIND_SHARED) ? dm.Is : 0, (kind_mask & KIND_HIT) ? dm.I : 0);
    dim3 grid((rows + GW - 1) / GW, max_groups(dm));
    rows_from_h_kernel<0><<<grid, GT, 0, st>>>(dm, kind_mask, w, h, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_lore_a(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                  cudaStream_t st) {
    dim3 grid((dm.r + GW - 1) / GW, min(dm.N, dm.T * dm.K));
    rows_from_h_kernel<1><<<grid, GT, 0, st>>>(dm, KIND_LOW, w, h, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_down(const Dims &dm, int kind_mask, const spice_layer_weights &w, const Tables &tb, cudaStream_t st) {
    dim3 grid((dm.d + GW - 1) / GW, kind_mask == KIND_LOW ? min(dm.N, dm.T * dm.K) : max_groups(dm));
    down_kernel<<<grid, GT, 0, st>>>(dm, kind_mask, w, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_lore_b(const Dims &dm, const spice_layer_weights &w, const Tables &tb, int z_after_hits, cudaStream_t st) {
    const size_t smem = (size_t)LB * dm.r * sizeof(float);
    if (smem > 48 * 1024) return z_after_hits ? -1 : launch_down(dm, KIND_LOW, w, tb, st);
    dim3 grid((dm.d + 255) / 256, min(LB_GROUPS, min(dm.N, dm.T * dm.K)));
    lore_b_kernel<<<grid, 256, smem, st>>>(dm, w, tb, z_after_hits);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_combine(const Dims &dm, const CombineArgs &a, const Tables &tb, cudaStream_t st) {
    dim3 grid((dm.d / 4 + 255) / 256, dm.T);
    combine_kernel<<<grid, 256, 0, st>>>(dm, a, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace spice
