// The 8-bit weight format of the layer's second precision.
//
// The paper reports every result at BF16 and at one quantised weight precision (Sec. 5.1, Table 1) without defining the
// latter.  Here: E4M3 codes (1-4-3 bits, bias 7, no infinities, largest value 448) with one power-of-two scale per
// output row, s_r = 2^ceil(log2(max_j |W_rj| / 448)) (1 for an all-zero row), q_rj = nearest E4M3 value of W_rj / s_r,
// ties to even, saturating.  The conversions are the hardware's (cvt.rn.satfinite); the scale is found with integer
// arithmetic on the exponent, no logarithm.
#include <cuda_fp8.h>

#include "spice_internal.cuh"

namespace spice {

namespace {

// one warp per row: maximum magnitude, scale, codes
__global__ void __launch_bounds__(256) quantize_e4m3_rows_kernel(const __nv_bfloat16 *__restrict__ w, size_t rows, int cols,
                                                                 uint8_t *__restrict__ q, float *__restrict__ scale) {
    const int lane = threadIdx.x & 31;
    const size_t warps = (size_t)gridDim.x * (blockDim.x >> 5);
    for (size_t r = (size_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < rows; r += warps) {
        const uint4 *src = reinterpret_cast<const uint4 *>(w + r * cols);
        const int nv = cols >> 3;
        uint32_t amax_bits = 0;   // bf16 magnitude bits compare like integers
        for (int v = lane; v < nv; v += 32) {
            const uint4 u = src[v];
            const uint32_t x[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                amax_bits = max(amax_bits, x[j] & 0x7fffu);
                amax_bits = max(amax_bits, (x[j] >> 16) & 0x7fffu);
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) amax_bits = max(amax_bits, __shfl_xor_sync(0xffffffffu, amax_bits, o));
        const float amax = __uint_as_float(amax_bits << 16);
        // amax / 448 = m * 2^e with m in [0.5, 1): the scale is 2^e, or 2^(e-1) when m is exactly 0.5
        float s = 1.0f;
        if (amax > 0.0f) {
            int e;
            const float m = frexpf(amax / 448.0f, &e);   // (448 = 7 * 2^6: the division is exact up to one rounding of a
            s = ldexpf(1.0f, m == 0.5f ? e - 1 : e);      //  value with 8 significant bits; m == 0.5 only for amax = 448 * 2^k)
        }
        if (lane == 0) scale[r] = s;
        const float inv = 1.0f / s;                      // exact: a power of two
        uint2 *dst = reinterpret_cast<uint2 *>(q + r * cols);
        for (int v = lane; v < nv; v += 32) {
            const uint4 u = src[v];
            const uint32_t x[4] = {u.x, u.y, u.z, u.w};
            uint32_t out[2] = {0u, 0u};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t lo = __nv_cvt_float_to_fp8(bf_lo(x[j]) * inv, __NV_SATFINITE, __NV_E4M3);
                const uint32_t hi = __nv_cvt_float_to_fp8(bf_hi(x[j]) * inv, __NV_SATFINITE, __NV_E4M3);
                out[j >> 1] |= (lo | (hi << 8)) << (16 * (j & 1));
            }
            dst[v] = make_uint2(out[0], out[1]);
        }
    }
}

}  // namespace

int launch_quantize_e4m3_rows(const __nv_bfloat16 *w, size_t rows, int cols, uint8_t *q, float *scale, cudaStream_t st) {
    if (rows == 0) return 0;
    const size_t blocks = (rows + 7) / 8;
    quantize_e4m3_rows_kernel<<<(unsigned)(blocks < 4096 ? blocks : 4096), 256, 0, st>>>(w, rows, cols, q, scale);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace spice
