// Device routines shared by the stand-alone router kernel and the fused decode kernel, so that
// both produce bit-identical logits, selections and gates (Eq. 1 of the paper; gate scores of
// Sec. 4.2).  The arithmetic order is fixed: each lane accumulates its 8-element slices of the
// row in increasing k with fmaf, then the 32 lane sums are combined by an xor-shuffle tree.
#pragma once
#include "spice_internal.cuh"

namespace spice {

// acc += sum over this lane's slices of w_row[k] * x[k];  x is an fp32 row in shared memory
__device__ __forceinline__ float lane_dot_f32(const __nv_bfloat16 *__restrict__ w_row, const float *x, int d, int lane) {
    float s = 0.f;
    for (int k = lane * 8; k < d; k += 256) {
        const uint4 u = *reinterpret_cast<const uint4 *>(w_row + k);
        const float4 a = *reinterpret_cast<const float4 *>(x + k);
        const float4 b = *reinterpret_cast<const float4 *>(x + k + 4);
        s = fmaf(bf_lo(u.x), a.x, s); s = fmaf(bf_hi(u.x), a.y, s);
        s = fmaf(bf_lo(u.y), a.z, s); s = fmaf(bf_hi(u.y), a.w, s);
        s = fmaf(bf_lo(u.z), b.x, s); s = fmaf(bf_hi(u.z), b.y, s);
        s = fmaf(bf_lo(u.w), b.z, s); s = fmaf(bf_hi(u.w), b.w, s);
    }
    return s;
}

// same sum with the activation row held as bf16 in shared memory (values are identical after
// the exact bf16 -> fp32 widening, so the result equals lane_dot_f32 bit for bit)
__device__ __forceinline__ float lane_dot_bf16(const __nv_bfloat16 *__restrict__ w_row, const __nv_bfloat16 *x, int d,
                                               int lane) {
    float s = 0.f;
    for (int k = lane * 8; k < d; k += 256) {
        const uint4 u = *reinterpret_cast<const uint4 *>(w_row + k);
        const uint4 v = *reinterpret_cast<const uint4 *>(x + k);
        s = fmaf(bf_lo(u.x), bf_lo(v.x), s); s = fmaf(bf_hi(u.x), bf_hi(v.x), s);
        s = fmaf(bf_lo(u.y), bf_lo(v.y), s); s = fmaf(bf_hi(u.y), bf_hi(v.y), s);
        s = fmaf(bf_lo(u.z), bf_lo(v.z), s); s = fmaf(bf_hi(u.z), bf_hi(v.z), s);
        s = fmaf(bf_lo(u.w), bf_lo(v.w), s); s = fmaf(bf_hi(u.w), bf_hi(v.w), s);
    }
    return s;
}

// One warp selects the K largest of l[0..N) (ties -> smaller index), writes idx_out[0..K) in
// decreasing order and the gates: softmax over the winners (norm_topk) or full-softmax values.
// N <= 1024, K <= 32.  l may live in shared memory; it is not modified.
__device__ __forceinline__ void warp_topk_gates(const float *l, int N, int K, int norm_topk, int lane,
                                                int32_t *idx_out, float *gate_out, float *logits_out) {
    if (logits_out)
        for (int e = lane; e < N; e += 32) logits_out[e] = l[e];
    uint32_t taken = 0;     // bit i: expert lane + 32*i already selected (N <= 1024)
    float m = 0.f, denom = 0.f, my_val = 0.f;
    int my_idx = 0;
    for (int k = 0; k < K; ++k) {
        float bv = -INFINITY;
        int be = 0x7fffffff;
        for (int i = 0, e = lane; e < N; ++i, e += 32) {
            if ((taken >> i) & 1u) continue;
            float v = l[e];
            if (!(v == v)) v = -INFINITY;   // NaN never wins
            if (be == 0x7fffffff || v > bv) { bv = v; be = e; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            int oe = __shfl_xor_sync(0xffffffffu, be, o);
            if (ov > bv || (ov == bv && oe < be)) { bv = ov; be = oe; }
        }
        if ((be & 31) == lane) taken |= 1u << (be >> 5);
        if (k == 0) {
            m = bv;
            if (!norm_topk) {   // full-softmax denominator
                float s = 0.f;
                for (int e = lane; e < N; e += 32) s += expf(l[e] - m);
                denom = warp_sum(s);
            }
        }
        if (lane == k) { my_val = bv; my_idx = be; }
    }
    float p = (lane < K) ? expf(my_val - m) : 0.f;
    if (norm_topk) {
        // sum the K numerators in k order on every lane (deterministic, matches the definition)
        float s = 0.f;
        for (int k = 0; k < K; ++k) s += __shfl_sync(0xffffffffu, p, k);
        denom = s;
    }
    if (lane < K) {
        idx_out[lane] = my_idx;
        gate_out[lane] = p / denom;
    }
}

}  // namespace spice
