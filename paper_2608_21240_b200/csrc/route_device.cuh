// Device routines shared by the stand-alone router kernel and the fused decode kernel, so that
// both produce bit-identical logits, selections and gates (Eq. 1 of the paper; gate scores of
// Sec. 4.2).  The arithmetic order is fixed: each lane reduces every 8-element slice it owns with
// an fmaf chain from zero, adds the slice sums in increasing k, then the 32 lane sums are
// combined by an xor-shuffle tree.
#pragma once
#include "spice_internal.cuh"

namespace spice {

// 8 products of one 128-bit slice, accumulated in index order starting from zero
__device__ __forceinline__ float slice_dot(const uint4 u, const float4 a, const float4 b) {
    float q = 0.f;
    q = fmaf(bf_lo(u.x), a.x, q); q = fmaf(bf_hi(u.x), a.y, q);
    q = fmaf(bf_lo(u.y), a.z, q); q = fmaf(bf_hi(u.y), a.w, q);
    q = fmaf(bf_lo(u.z), b.x, q); q = fmaf(bf_hi(u.z), b.y, q);
    q = fmaf(bf_lo(u.w), b.z, q); q = fmaf(bf_hi(u.w), b.w, q);
    return q;
}
__device__ __forceinline__ float slice_dot(const uint4 u, const uint4 v) {
    return slice_dot(u, make_float4(bf_lo(v.x), bf_hi(v.x), bf_lo(v.y), bf_hi(v.y)),
                     make_float4(bf_lo(v.z), bf_hi(v.z), bf_lo(v.w), bf_hi(v.w)));
}

// This lane's share of dot(w_row, x): slices k = lane*8 + 256*i, each reduced by slice_dot, the
// slice sums added in increasing i.  x is an fp32 row in shared memory.
__device__ __forceinline__ float lane_dot_f32(const __nv_bfloat16 *__restrict__ w_row, const float *x, int d, int lane) {
    float s = 0.f;
    for (int k = lane * 8; k < d; k += 256) {
        const uint4 u = *reinterpret_cast<const uint4 *>(w_row + k);
        s += slice_dot(u, *reinterpret_cast<const float4 *>(x + k), *reinterpret_cast<const float4 *>(x + k + 4));
    }
    return s;
}

// same sum with the activation row held as bf16 (the bf16 -> fp32 widening is exact, so the
// result equals lane_dot_f32 bit for bit)
__device__ __forceinline__ float lane_dot_bf16(const __nv_bfloat16 *__restrict__ w_row, const __nv_bfloat16 *x, int d,
                                               int lane) {
    float s = 0.f;
#pragma unroll 8
    for (int k = lane * 8; k < d; k += 256) {
        const uint4 u = *reinterpret_cast<const uint4 *>(w_row + k);
        s += slice_dot(u, *reinterpret_cast<const uint4 *>(x + k));
    }
    return s;
}

// One warp selects the K largest of l[0..N) (ties -> smaller index), writes idx_out[0..K) in
// decreasing order and the gates: softmax over the winners (norm_topk) or full-softmax values.
// N <= 1024, K <= 32.  l may live in shared memory; it is not modified.  sel_idx / sel_val:
// K-entry scratch rows in shared memory owned by this warp.
// The winners are found by ranking: element e has rank #{j : l[j] > l[e] or (l[j] == l[e] and j < e)}
// and is the rank-th winner when rank < K.  Ranks are a permutation, so every output slot is written
// exactly once; the result is the same as K rounds of arg-max with ties to the smaller index.
__device__ __forceinline__ void warp_topk_gates(const float *l, int N, int K, int norm_topk, int lane,
                                                int32_t *idx_out, float *gate_out, float *logits_out,
                                                int *sel_idx, float *sel_val) {
    if (logits_out) {
#pragma unroll 1
        for (int e = lane; e < N; e += 32) logits_out[e] = l[e];
    }
#pragma unroll 1
    for (int e = lane; e < N; e += 32) {
        float v = l[e];
        if (!(v == v)) v = -INFINITY;   // NaN never wins
        int rank = 0;
#pragma unroll 4
        for (int j = 0; j < N; ++j) {
            float u = l[j];
            if (!(u == u)) u = -INFINITY;
            rank += (u > v) || (u == v && j < e);
        }
        if (rank < K) {
            sel_idx[rank] = e;
            sel_val[rank] = v;
        }
    }
    __syncwarp();
    const float m = sel_val[0];
    float denom = 0.f;
    if (!norm_topk) {   // full-softmax denominator
        float s = 0.f;
#pragma unroll 1
        for (int e = lane; e < N; e += 32) s += expf(l[e] - m);
        denom = warp_sum(s);
    }
    const float p = (lane < K) ? expf(sel_val[lane] - m) : 0.f;
    if (norm_topk) {
        // sum the K numerators in k order on every lane (deterministic, matches the definition)
        float s = 0.f;
#pragma unroll 1
        for (int k = 0; k < K; ++k) s += __shfl_sync(0xffffffffu, p, k);
        denom = s;
    }
    if (lane < K) {
        idx_out[lane] = sel_idx[lane];
        gate_out[lane] = p / denom;
    }
    __syncwarp();
}

// The same selection by K rounds of a shuffle arg-max; used when N is large (ranking is O(N^2)).
__device__ __forceinline__ void warp_topk_gates_rounds(const float *l, int N, int K, int norm_topk, int lane,
                                                int32_t *idx_out, float *gate_out, float *logits_out) {
    if (logits_out)
#pragma unroll 1
        for (int e = lane; e < N; e += 32) logits_out[e] = l[e];
    uint32_t taken = 0;     // bit i: expert lane + 32*i already selected (N <= 1024)
    float m = 0.f, denom = 0.f, my_val = 0.f;
    int my_idx = 0;
#pragma unroll 1
    for (int k = 0; k < K; ++k) {
        float bv = -INFINITY;
        int be = 0x7fffffff;
#pragma unroll 1
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
#pragma unroll 1
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
#pragma unroll 1
        for (int k = 0; k < K; ++k) s += __shfl_sync(0xffffffffu, p, k);
        denom = s;
    }
    if (lane < K) {
        idx_out[lane] = my_idx;
        gate_out[lane] = p / denom;
    }
}

}  // namespace spice
