// LoRE calibration of one (layer, expert) pair (Sec. 4.2 of the paper): fit the rank-r residual module
//     Delta(h) = B A h,   A: r x d,  B: d x r,
// that minimises  sum_{h in D} || E(h) - S(h) - B A h ||_2^2  over the calibration tokens routed to the expert.
// The paper states this objective and names no optimiser; the objective is a reduced-rank
// regression and has a closed-form minimiser, which is what is computed here (in fp32, offline path):
//     G = H^T H (+ ridge),  C = H^T R          H [n,d] hidden states, R [n,d] targets E(h) - S(h)
//     G = L L^T,  Z = L^-1 C                   (then the fitted values satisfy  Yhat^T Yhat = Z^T Z)
//     V = r leading eigenvectors of Z^T Z      block subspace iteration, orthonormalised by Cholesky QR (twice)
//     B = V,   A = ( L^-T Z V )^T = ( W V )^T  with W = G^-1 C the least-squares map
// The two Gram products, 2 n d^2 multiply-adds each and a third of the work, run on the tensor cores: H is bf16, so
// H^T H is a bf16 x bf16 product with fp32 accumulation and nothing is lost; the fp32 targets are written as the sum of
// three bf16 terms (24 significant bits), so H^T R is three such products added in a fixed order.  The operands are
// transposed copies (reduction index contiguous) and the kernel is the plain mode of the grouped GEMM of large batches.
// Everything else is dense fp32 linear algebra on d x d matrices built from tiled SGEMMs (split over the reduction,
// with the slices summed in a fixed order, where a product has too few output tiles to fill the GPU), 64 x 64 Cholesky /
// triangular-solve blocks and a few element-wise kernels, launched in order on one stream; nothing synchronises
// with the host.  The caller provides the workspace (spice_lore_calibrate_workspace_bytes).
#include "spice_internal.cuh"

namespace spice {

namespace {

constexpr int TB = 64;    // block size of the factorisations and tile of the SGEMM
constexpr int BK = 16;

__host__ __device__ inline int pad64(int v) { return (v + 63) / 64 * 64; }

// C[M,N] = alpha * op(A) * op(B) + beta * C, row-major.  TA: A is stored [K,M] (lda); TB_: B is stored [N,K] (ldb).
template <bool TA, bool TB_>
__global__ void __launch_bounds__(256) sgemm_kernel(int M, int N, int K, float alpha, const float *__restrict__ A, int lda,
                                                    const float *__restrict__ B, int ldb, float beta, float *__restrict__ C,
                                                    int ldc, int kchunk, float *__restrict__ part) {
    __shared__ float As[BK][TB + 4], Bs[BK][TB + 4];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const int m0 = blockIdx.y * TB, n0 = blockIdx.x * TB;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    // blockIdx.z takes the reduction range [z kchunk, (z+1) kchunk): products with few output tiles are split over
    // the reduction so that they fill the machine; the slices are summed in z order by splitk_reduce_kernel
    const int kb = blockIdx.z * kchunk;
    K = min(K, kb + kchunk);
    for (int k0 = kb; k0 < K; k0 += BK) {
        for (int e = threadIdx.x; e < BK * TB; e += 256) {
            int kk, mm;
            if (TA) { kk = e / TB; mm = e % TB; } else { mm = e / BK; kk = e % BK; }
            const int gm = m0 + mm, gk = k0 + kk;
            As[kk][mm] = (gm < M && gk < K) ? (TA ? A[(size_t)gk * lda + gm] : A[(size_t)gm * lda + gk]) : 0.f;
            int kb, nn;
            if (TB_) { nn = e / BK; kb = e % BK; } else { kb = e / TB; nn = e % TB; }
            const int gn = n0 + nn, gkb = k0 + kb;
            Bs[kb][nn] = (gn < N && gkb < K) ? (TB_ ? B[(size_t)gn * ldb + gkb] : B[(size_t)gkb * ldb + gn]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
            if (gm < M && gn < N) {
                if (part) {
                    part[((size_t)blockIdx.z * M + gm) * N + gn] = acc[i][j];
                } else {
                    float *c = C + (size_t)gm * ldc + gn;
                    *c = alpha * acc[i][j] + (beta != 0.f ? beta * *c : 0.f);
                }
            }
        }
}

// C = alpha * (sum over the nz slices of part, in slice order) + beta * C
__global__ void splitk_reduce_kernel(int M, int N, int nz, float alpha, const float *__restrict__ part, float beta,
                                     float *__restrict__ C, int ldc) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)M * N) return;
    float s = 0.f;
    for (int z = 0; z < nz; ++z) s += part[(size_t)z * M * N + i];
    float *c = C + (i / N) * (size_t)ldc + (i % N);
    *c = alpha * s + (beta != 0.f ? beta * *c : 0.f);
}

// scratch for the split products (set by launch_lore_calibrate for the duration of a call)
thread_local float *t_splitk_ws = nullptr;
thread_local size_t t_splitk_floats = 0;

template <bool TA, bool TB_>
int gemm(int M, int N, int K, float alpha, const float *A, int lda, const float *B, int ldb, float beta, float *C, int ldc,
         cudaStream_t st) {
    if (M <= 0 || N <= 0) return 0;
    dim3 grid((N + TB - 1) / TB, (M + TB - 1) / TB);
    const int tiles = (int)(grid.x * grid.y);
    int nz = 1;
    if (t_splitk_ws && tiles < 74 && K >= 512) {
        nz = min(min(148 / tiles, K / 256), 32);
        while (nz > 1 && (size_t)nz * M * N > t_splitk_floats) --nz;
    }
    if (nz <= 1) {
        sgemm_kernel<TA, TB_><<<grid, 256, 0, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, K, nullptr);
        return cudaGetLastError() == cudaSuccess ? 1 : -1;
    }
    const int kchunk = ((K + nz - 1) / nz + BK - 1) / BK * BK;
    grid.z = (K + kchunk - 1) / kchunk;
    sgemm_kernel<TA, TB_><<<grid, 256, 0, st>>>(M, N, K, alpha, A, lda, B, ldb, beta, C, ldc, kchunk, t_splitk_ws);
    splitk_reduce_kernel<<<(unsigned)(((size_t)M * N + 255) / 256), 256, 0, st>>>(M, N, (int)grid.z, alpha, t_splitk_ws, beta, C, ldc);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

// dst[c, r] = src[r, c] for a bf16 matrix [rows, cols]; dst is [cols_pad, ld] with zeros outside (32 x 32 tiles)
__global__ void __launch_bounds__(256) transpose_bf16_kernel(const __nv_bfloat16 *__restrict__ src, int rows, int cols,
                                                             __nv_bfloat16 *__restrict__ dst, int cols_pad, int ld) {
    __shared__ __nv_bfloat16 t[32][33];
    const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        t[i][tx] = (r < rows && c < cols) ? src[(size_t)r * cols + c] : __float2bfloat16(0.f);
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;
        if (c < cols_pad && r < ld) dst[(size_t)c * ld + r] = t[tx][i];
    }
}

// the same for an fp32 matrix, written as three bf16 planes whose sum is the value to 24 bits: x1 = bf16(x),
// x2 = bf16(x - x1), x3 = bf16(x - x1 - x2); plane p at dst + p * cols_pad * ld
__global__ void __launch_bounds__(256) transpose_split3_kernel(const float *__restrict__ src, int rows, int cols,
                                                               __nv_bfloat16 *__restrict__ dst, int cols_pad, int ld) {
    __shared__ float t[32][33];
    const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        t[i][tx] = (r < rows && c < cols) ? src[(size_t)r * cols + c] : 0.f;
    }
    __syncthreads();
    const size_t plane = (size_t)cols_pad * ld;
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;
        if (c < cols_pad && r < ld) {
            float x = t[tx][i];
            const __nv_bfloat16 x1 = __float2bfloat16(x);
            x -= __bfloat162float(x1);
            const __nv_bfloat16 x2 = __float2bfloat16(x);
            x -= __bfloat162float(x2);
            const size_t o = (size_t)c * ld + r;
            dst[o] = x1;
            dst[plane + o] = x2;
            dst[2 * plane + o] = __float2bfloat16(x);
        }
    }
}

// Operands of the subspace iteration's two products on the tensor cores.  An fp32 value is written as x1 + x2 with
// x1 = bf16(x), x2 = bf16(x - x1) (16 significant bits), and a product Z Q as Z1 Q1 + Z1 Q2 + Z2 Q1 (the dropped term
// Z2 Q2 is 2^-16 of the result): ONE product with the three pairs laid side by side along the reduction index,
// [Z1 | Z1 | Z2] [Q1 | Q2 | Q1]^T, so that the accumulator in tensor memory adds them.
// dst [n, 3 n] from the fp32 matrix src [n, n] (ld): row i = (row i of src, or column i when TRANS) as [x1 | x1 | x2]
template <bool TRANS>
__global__ void __launch_bounds__(256) split2_cat_matrix_kernel(const float *__restrict__ src, int n, int ld, __nv_bfloat16 *__restrict__ dst) {
    __shared__ float t[32][33];
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;   // tile of dst rows r0.., reduction index c0..
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        // want v(r, c) = TRANS ? src[c][r] : src[r][c]; read coalesced along the contiguous index of src
        const int a = TRANS ? c0 + i : r0 + i, b = TRANS ? r0 + tx : c0 + tx;
        t[i][tx] = (a < n && b < n) ? src[(size_t)a * ld + b] : 0.f;
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        if (r < n && c < n) {
            const float x = TRANS ? t[tx][i] : t[i][tx];
            const __nv_bfloat16 x1 = __float2bfloat16(x), x2 = __float2bfloat16(x - __bfloat162float(x1));
            __nv_bfloat16 *row = dst + (size_t)r * 3 * n;
            row[c] = x1;
            row[n + c] = x1;
            row[2 * n + c] = x2;
        }
    }
}
// dst [cols, 3 n] from the fp32 block src [n, cols] (ld = cols): row j = column j of src as [x1 | x2 | x1]
__global__ void __launch_bounds__(256) split2_cat_block_kernel(const float *__restrict__ src, int n, int cols, __nv_bfloat16 *__restrict__ dst) {
    __shared__ float t[32][33];
    const int k0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    for (int i = ty; i < 32; i += 8) {
        const int k = k0 + i, j = j0 + tx;
        t[i][tx] = (k < n && j < cols) ? src[(size_t)k * cols + j] : 0.f;
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int j = j0 + i, k = k0 + tx;
        if (j < cols && k < n) {
            const float x = t[tx][i];
            const __nv_bfloat16 x1 = __float2bfloat16(x), x2 = __float2bfloat16(x - __bfloat162float(x1));
            __nv_bfloat16 *row = dst + (size_t)j * 3 * n;
            row[k] = x1;
            row[n + k] = x2;
            row[2 * n + k] = x1;
        }
    }
}

// c = (a + b) + c3, element-wise over a [rows, ld] matrix
__global__ void sum3_kernel(float *__restrict__ a, const float *__restrict__ b, const float *__restrict__ c3, size_t n) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) a[i] = (a[i] + b[i]) + c3[i];
}

// bf16 [rows, cols] -> fp32 [rows, ld] with zero columns cols..ld-1
__global__ void widen_pad_kernel(const __nv_bfloat16 *__restrict__ src, int rows, int cols, float *__restrict__ dst, int ld) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)rows * ld) return;
    const int r = (int)(i / ld), c = (int)(i % ld);
    dst[i] = c < cols ? __bfloat162float(src[(size_t)r * cols + c]) : 0.f;
}

// scal[0] = trace of the leading d x d block / d
__global__ void mean_diag_kernel(const float *__restrict__ G, int ld, int d, float *scal) {
    __shared__ float red[256];
    float s = 0.f;
    for (int i = threadIdx.x; i < d; i += 256) s += G[(size_t)i * ld + i];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) scal[0] = red[0] / (float)d;
}

// diagonal: G[i,i] += ridge * scal[0] for i < d; padding rows / columns i >= d become the identity
__global__ void regularise_kernel(float *G, int ld, int d, int dp, float ridge, const float *scal) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)dp * dp) return;
    const int r = (int)(i / dp), c = (int)(i % dp);
    float *g = G + (size_t)r * ld + c;
    if (r >= d || c >= d) *g = (r == c) ? 1.f : 0.f;
    else if (r == c) *g += ridge * scal[0];
}

// Cholesky of one 64 x 64 diagonal block in place (lower triangle; the strict upper triangle is zeroed).
// A pivot that is not positive is replaced by a tiny positive number and flagged.
__global__ void __launch_bounds__(256) potrf64_kernel(float *A, int ld, int32_t *flag) {
    __shared__ float a[TB][TB + 1];
    // 256 threads: thread (t, part) owns row t and the columns c = part (mod 4) of the trailing update
    const int t = threadIdx.x & 63, part = threadIdx.x >> 6;
#pragma unroll 4
    for (int r = part; r < TB; r += 4) a[r][t] = A[(size_t)r * ld + t];
    __syncthreads();
    for (int j = 0; j < TB; ++j) {
        if (threadIdx.x == j) {
            float p = a[j][j];
            if (!(p > 0.f)) {
                p = 1e-20f;
                atomicOr(flag, 1);
            }
            a[j][j] = sqrtf(p);
        }
        __syncthreads();
        const float piv = a[j][j];
        if (part == 0 && t > j) a[t][j] /= piv;
        __syncthreads();
        // trailing update: row t, columns j+1 .. t
        if (t > j) {
            const float ltj = a[t][j];
            for (int c = j + 1 + ((part - (j + 1)) & 3); c <= t; c += 4) a[t][c] -= ltj * a[c][j];
        }
        __syncthreads();
    }
#pragma unroll 4
    for (int r = part; r < TB; r += 4) A[(size_t)r * ld + t] = t <= r ? a[r][t] : 0.f;
}

// X <- X L^-T for a panel of rows (one CTA of 64 threads takes 64 rows): X [rows, 64] (ldx), L 64 x 64 lower (ldl)
__global__ void __launch_bounds__(64) trsm_right_lt_kernel(float *X, int ldx, int rows, const float *__restrict__ L, int ldl) {
    __shared__ float l[TB][TB + 1];
    const int t = threadIdx.x;
#pragma unroll 8
    for (int r = 0; r < TB; ++r) l[r][t] = L[(size_t)r * ldl + t];
    __syncthreads();
    const int row = blockIdx.x * TB + t;
    if (row >= rows) return;
    float x[TB];
#pragma unroll
    for (int c = 0; c < TB; ++c) x[c] = X[(size_t)row * ldx + c];
    // solve y L^T = x: y_c = (x_c - sum_{q<c} y_q L[c][q]) / L[c][c]   (fully unrolled: x stays in registers)
#pragma unroll
    for (int c = 0; c < TB; ++c) {
        float s = x[c];
#pragma unroll
        for (int qq = 0; qq < c; ++qq) s -= x[qq] * l[c][qq];
        x[c] = s / l[c][c];
    }
#pragma unroll
    for (int c = 0; c < TB; ++c) X[(size_t)row * ldx + c] = x[c];
}

// X <- L^-1 X (TRANS = false) or L^-T X (TRANS = true) for a block row X [64, cols] (ldx); one thread per column
template <bool TRANS>
__global__ void __launch_bounds__(64) trsm_left_kernel(float *X, int ldx, int cols, const float *__restrict__ L, int ldl) {
    __shared__ float l[TB][TB + 1];
    const int t = threadIdx.x;
    for (int r = 0; r < TB; ++r) l[r][t] = L[(size_t)r * ldl + t];
    __syncthreads();
    const int col = blockIdx.x * TB + t;
    if (col >= cols) return;
    float x[TB];
#pragma unroll
    for (int r = 0; r < TB; ++r) x[r] = X[(size_t)r * ldx + col];
    if (!TRANS) {
#pragma unroll 1
        for (int r = 0; r < TB; ++r) {
            float s = x[r];
            for (int qq = 0; qq < r; ++qq) s -= l[r][qq] * x[qq];
            x[r] = s / l[r][r];
        }
    } else {
#pragma unroll 1
        for (int r = TB - 1; r >= 0; --r) {
            float s = x[r];
            for (int qq = r + 1; qq < TB; ++qq) s -= l[qq][r] * x[qq];
            x[r] = s / l[r][r];
        }
    }
#pragma unroll
    for (int r = 0; r < TB; ++r) X[(size_t)r * ldx + col] = x[r];
}

// deterministic start block for the subspace iteration: a hash of (row, column) mapped to (-1, 1)
__global__ void init_block_kernel(float *Q, int rows, int ld, int cols) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)rows * ld) return;
    const int r = (int)(i / ld), c = (int)(i % ld);
    uint32_t h = (uint32_t)r * 2654435761u ^ ((uint32_t)c + 0x9e3779b9u) * 2246822519u;
    h ^= h >> 15; h *= 2246822519u; h ^= h >> 13; h *= 3266489917u; h ^= h >> 16;
    Q[i] = c < cols ? ((float)(h >> 8) * (1.0f / 8388608.0f) - 1.0f) : 0.f;
}

// S (rp x rp): padding rows / columns >= r become the identity.  In the first pass of the Cholesky QR a small multiple of
// the largest diagonal entry is added to the diagonal: the columns of a power-iterated block can be dependent to working
// precision, and the factorisation must not break down on directions that carry no weight (the second pass restores
// orthonormality of what is left).
__global__ void fix_gram_kernel(float *S, int rp, int r, float jitter) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rp * rp) return;
    const int a = i / rp, b = i % rp;
    if (a >= r || b >= r) {
        S[i] = (a == b) ? 1.f : 0.f;
    } else if (a == b && jitter > 0.f) {
        float mx = 0.f;
        for (int q = 0; q < r; ++q) mx = fmaxf(mx, S[q * rp + q]);   // (reads diagonal entries other threads may be updating:
        S[i] += jitter * mx;                                          //  the bound only has to be of the right magnitude)
    }
}

// ---- one Cholesky-QR pass of a block of 64 columns in three launches (the general path below takes six)
// (1) Gram matrix of one 64-row slab of Q [rows, 64]: part[b] = Q_b^T Q_b
__global__ void __launch_bounds__(256) qr_gram_slab_kernel(const float *__restrict__ Q, int rows, float *__restrict__ part) {
    __shared__ float q[TB][TB + 1];
    const int r0 = blockIdx.x * TB;
    for (int e = threadIdx.x; e < TB * TB; e += 256) {
        const int k = e / TB, c = e % TB;
        q[k][c] = r0 + k < rows ? Q[(size_t)(r0 + k) * TB + c] : 0.f;
    }
    __syncthreads();
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 8
    for (int k = 0; k < TB; ++k) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = q[k][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = q[k][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    float *out = part + (size_t)blockIdx.x * TB * TB;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) out[(ty * 4 + i) * TB + tx * 4 + j] = acc[i][j];
}

// (2) S = sum of the slabs' Gram matrices in slab order; rows / columns >= r become the identity; in the first pass a
// small multiple of the largest diagonal entry is added to the diagonal (see fix_gram_kernel); Cholesky in place in shared
// memory; L (lower, strict upper triangle zero) to global memory.  One CTA.
__global__ void __launch_bounds__(256) qr_factor_kernel(const float *__restrict__ part, int n_slabs, int r, float jitter,
                                                        float *__restrict__ L, int32_t *flag) {
    __shared__ float a[TB][TB + 1];
    __shared__ float s_max;
    // (four consecutive elements per thread and step, sixteen slabs' loads in flight; the sum stays in slab order)
    for (int e = threadIdx.x * 4; e < TB * TB; e += 256 * 4) {
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int b0 = 0; b0 < n_slabs; b0 += 16) {
            float4 v[16];
#pragma unroll
            for (int u = 0; u < 16; ++u)
                v[u] = b0 + u < n_slabs ? __ldcg(reinterpret_cast<const float4 *>(part + (size_t)(b0 + u) * TB * TB + e))
                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                s.x += v[u].x;
                s.y += v[u].y;
                s.z += v[u].z;
                s.w += v[u].w;
            }
        }
        const int i = e / TB, j = e % TB;   // (j is a multiple of 4: the four elements share row i)
        a[i][j] = (i >= r || j >= r) ? (i == j ? 1.f : 0.f) : s.x;
        a[i][j + 1] = (i >= r || j + 1 >= r) ? (i == j + 1 ? 1.f : 0.f) : s.y;
        a[i][j + 2] = (i >= r || j + 2 >= r) ? (i == j + 2 ? 1.f : 0.f) : s.z;
        a[i][j + 3] = (i >= r || j + 3 >= r) ? (i == j + 3 ? 1.f : 0.f) : s.w;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float mx = 0.f;
        for (int i = 0; i < r; ++i) mx = fmaxf(mx, a[i][i]);
        s_max = mx;
    }
    __syncthreads();
    if (jitter > 0.f && (int)threadIdx.x < r) a[threadIdx.x][threadIdx.x] += jitter * s_max;
    __syncthreads();
    // Right-looking Cholesky by the first 64 threads, thread t holding row t of the lower triangle in registers.  Step j:
    // every thread publishes its entry of column j, one barrier (the column buffers alternate, so a fast thread's next
    // column cannot overwrite what a slow one still reads), then each thread scales by the same 1 / sqrt(pivot) -- its own
    // entry and the entries of the rows above it -- and updates its row.  One barrier of two warps per step instead of three
    // CTA-wide ones.
    __shared__ float col[2][TB];
    if (threadIdx.x < TB) {
        const int t = threadIdx.x;
        float row[TB];
#pragma unroll
        for (int c = 0; c < TB; ++c) row[c] = a[t][c];
#pragma unroll
        for (int j = 0; j < TB; ++j) {
            float *cb = col[j & 1];
            if (t >= j) cb[t] = row[j];
            asm volatile("bar.sync 2, 64;" ::: "memory");
            float p = cb[j];
            if (!(p > 0.f)) {
                p = 1e-20f;
                if (t == j) atomicOr(flag, 1);
            }
            const float inv = 1.0f / sqrtf(p);
            if (t >= j) row[j] *= inv;   // (row j's own entry becomes sqrt(pivot) up to rounding)
            const float ltj = row[j];
#pragma unroll
            for (int c = j + 1; c < TB; ++c)
                if (c <= t) row[c] -= ltj * (cb[c] * inv);
        }
#pragma unroll
        for (int c = 0; c < TB; ++c) a[t][c] = row[c];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < TB * TB; e += 256) {
        const int i = e / TB, j = e % TB;
        L[e] = j <= i ? a[i][j] : 0.f;
    }
}

__global__ void write_factors_kernel(const float *__restrict__ V, const float *__restrict__ X, int ld, int d, int r,
                                     __nv_bfloat16 *__restrict__ A, __nv_bfloat16 *__restrict__ B) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (size_t)d * r) return;
    const int j = (int)(i / r), qq = (int)(i % r);
    B[(size_t)j * r + qq] = __float2bfloat16(V[(size_t)j * ld + qq]);      // B [d, r]
    A[(size_t)qq * d + j] = __float2bfloat16(X[(size_t)j * ld + qq]);      // A [r, d] = X^T
}

// out[0] += sum (R - T)^2, out[1] += sum R^2 over a slice
__global__ void __launch_bounds__(256) loss_kernel(const float *__restrict__ R, int ldr, const float *__restrict__ T, int ldt, int n,
                                                   int d, float *out) {
    __shared__ float r0[256], r1[256];
    float a = 0.f, b = 0.f;
    const size_t total = (size_t)n * d;
    for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < total; i += (size_t)gridDim.x * 256) {
        const int row = (int)(i / d), c = (int)(i % d);
        const float rv = R[(size_t)row * ldr + c], dv = rv - T[(size_t)row * ldt + c];
        a += dv * dv;
        b += rv * rv;
    }
    r0[threadIdx.x] = a;
    r1[threadIdx.x] = b;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            r0[threadIdx.x] += r0[threadIdx.x + o];
            r1[threadIdx.x] += r1[threadIdx.x + o];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        atomicAdd(out, r0[0]);
        atomicAdd(out + 1, r1[0]);
    }
}

__global__ void widen_kernel(const __nv_bfloat16 *__restrict__ src, size_t n, float *__restrict__ dst) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = __bfloat162float(src[i]);
}

#define CK(expr)                 \
    do {                         \
        int k_ = (expr);         \
        if (k_ < 0) return -1;   \
        launches += k_;          \
    } while (0)
#define CKL()                                             \
    do {                                                  \
        if (cudaGetLastError() != cudaSuccess) return -1; \
        ++launches;                                       \
    } while (0)

// in-place blocked Cholesky of the leading np x np block (np a multiple of 64), lower triangle
int cholesky(float *G, int ld, int np, int32_t *flag, cudaStream_t st) {
    int launches = 0;
    for (int k = 0; k < np; k += TB) {
        float *diag = G + (size_t)k * ld + k;
        potrf64_kernel<<<1, 256, 0, st>>>(diag, ld, flag);
        CKL();
        const int rem = np - k - TB;
        if (rem > 0) {
            float *panel = G + (size_t)(k + TB) * ld + k;
            trsm_right_lt_kernel<<<rem / TB, 64, 0, st>>>(panel, ld, rem, diag, ld);
            CKL();
            CK((gemm<false, true>(rem, rem, TB, -1.f, panel, ld, panel, ld, 1.f, G + (size_t)(k + TB) * ld + (k + TB), ld, st)));
        }
    }
    return launches;
}

// Y [np, cols] <- Y L^-T with L np x np lower (np a multiple of 64): column blocks left to right
int solve_right_lt(float *Y, int ldy, int rows, const float *L, int ldl, int np, cudaStream_t st) {
    int launches = 0;
    for (int j = 0; j < np; j += TB) {
        if (j > 0)   // Y_j -= Y_{<j} L[j, <j]^T
            CK((gemm<false, true>(rows, TB, j, -1.f, Y, ldy, L + (size_t)j * ldl, ldl, 1.f, Y + j, ldy, st)));
        trsm_right_lt_kernel<<<(rows + TB - 1) / TB, 64, 0, st>>>(Y + j, ldy, rows, L + (size_t)j * ldl + j, ldl);
        CKL();
    }
    return launches;
}

// Q [dp, rp] <- orthonormal basis of its columns by Cholesky QR, twice
int orthonormalise(float *Q, int dp, int rp, int r, float *S, int32_t *flag, cudaStream_t st) {
    int launches = 0;
    if (rp == TB && t_splitk_ws && (size_t)(dp / TB) * TB * TB <= t_splitk_floats) {
        // a block of 64 columns: slab Gram matrices, one CTA that sums and factorises them, the triangular solve
        for (int pass = 0; pass < 2; ++pass) {
            qr_gram_slab_kernel<<<dp / TB, 256, 0, st>>>(Q, dp, t_splitk_ws);
            CKL();
            qr_factor_kernel<<<1, 256, 0, st>>>(t_splitk_ws, dp / TB, r, pass == 0 ? 1e-6f : 0.f, S, flag);
            CKL();
            trsm_right_lt_kernel<<<dp / TB, 64, 0, st>>>(Q, rp, dp, S, rp);
            CKL();
        }
        return launches;
    }
    for (int pass = 0; pass < 2; ++pass) {
        CK((gemm<true, false>(rp, rp, dp, 1.f, Q, rp, Q, rp, 0.f, S, rp, st)));
        fix_gram_kernel<<<(rp * rp + 255) / 256, 256, 0, st>>>(S, rp, r, pass == 0 ? 1e-6f : 0.f);
        CKL();
        CK(cholesky(S, rp, rp, flag, st));
        CK(solve_right_lt(Q, rp, dp, S, rp, rp, st));
    }
    return launches;
}

// tensor-core Gram products: transposed bf16 copies of H (1 plane) and R (3 planes), [dp, n8] each, two more [dp, dp] fp32
// outputs, and the GEMM's tile list
size_t gram_tc_bytes(size_t dp, size_t n) {
    const size_t n8 = (n + 7) / 8 * 8;
    return 4 * dp * n8 * sizeof(__nv_bfloat16) + 2 * dp * dp * sizeof(float) + (dp / 128 + 2) * sizeof(MTile) + 1024;
}
// tensor-core products of the subspace iteration (blocks of 64 columns): [Z1|Z1|Z2] and its transposed twin, the block's
// operand, the partial results of the ranges of the reduction, the tile list
constexpr int IT_SPLIT = 8;
size_t iter_tc_bytes(size_t dp) {
    return 2 * dp * 3 * dp * sizeof(__nv_bfloat16) + TB * 3 * dp * sizeof(__nv_bfloat16) + IT_SPLIT * dp * TB * sizeof(float) +
           (IT_SPLIT * (dp / 128 + 1) + 2) * sizeof(MTile) + 1024;
}

}  // namespace

size_t lore_calibrate_workspace_bytes(int d, int n, int r) {
    const size_t dp = pad64(d), rp = pad64(r);
    // H32 / T2 [n, dp], G [dp, dp], C [dp, dp], Q, P, Y [dp, rp] each, S [rp, rp], T1 [n, rp], A32 [rp, dp], B32 [dp, rp], scalars
    size_t f = (size_t)n * dp + 2 * dp * dp + 3 * dp * rp + rp * rp + (size_t)n * rp + 2 * dp * rp + 64;
    f += 8 * dp * rp;   // slices of the products that are split over their reduction
    return f * sizeof(float) + 256 + gram_tc_bytes(dp, (size_t)n) + iter_tc_bytes(dp);
}


int launch_lore_calibrate(int d, int n, int r, float ridge, int iters, const __nv_bfloat16 *h_cal, const float *resid,
                          __nv_bfloat16 *A_out, __nv_bfloat16 *B_out, float *loss_out, int32_t *flag, void *workspace,
                          cudaStream_t st) {
    int launches = 0;
    const int dp = pad64(d), rp = pad64(r);
    float *w = reinterpret_cast<float *>((reinterpret_cast<uintptr_t>(workspace) + 255) & ~uintptr_t(255));
    float *H32 = w;                      w += (size_t)n * dp;
    float *G = w;                        w += (size_t)dp * dp;
    float *C = w;                        w += (size_t)dp * dp;
    float *Q = w;                        w += (size_t)dp * rp;
    float *P = w;                        w += (size_t)dp * rp;
    float *Y = w;                        w += (size_t)dp * rp;
    float *S = w;                        w += (size_t)rp * rp;
    float *T1 = w;                       w += (size_t)n * rp;
    float *A32 = w;                      w += (size_t)rp * dp;
    float *B32 = w;                      w += (size_t)dp * rp;
    float *scal = w;                     w += 64;
    t_splitk_ws = w;                     w += (size_t)8 * dp * rp;
    t_splitk_floats = (size_t)8 * dp * rp;
    // buffers of the tensor-core Gram products
    const size_t n8 = ((size_t)n + 7) / 8 * 8;
    float *C2 = w;                       w += (size_t)dp * dp;
    float *C3 = w;                       w += (size_t)dp * dp;
    __nv_bfloat16 *Ht16 = reinterpret_cast<__nv_bfloat16 *>((reinterpret_cast<uintptr_t>(w) + 255) & ~uintptr_t(255));
    __nv_bfloat16 *Rt16 = Ht16 + (size_t)dp * n8;                 // three planes
    MTile *mt = reinterpret_cast<MTile *>((reinterpret_cast<uintptr_t>(Rt16 + 3 * (size_t)dp * n8) + 255) & ~uintptr_t(255));
    int32_t *n_mt = reinterpret_cast<int32_t *>(mt + dp / 128 + 1);
    // buffers of the tensor-core products of the subspace iteration
    __nv_bfloat16 *Zcat = reinterpret_cast<__nv_bfloat16 *>((reinterpret_cast<uintptr_t>(n_mt + 4) + 255) & ~uintptr_t(255));
    __nv_bfloat16 *Ztcat = Zcat + (size_t)dp * 3 * dp;
    __nv_bfloat16 *Bcat = Ztcat + (size_t)dp * 3 * dp;
    float *it_part = reinterpret_cast<float *>((reinterpret_cast<uintptr_t>(Bcat + (size_t)TB * 3 * dp) + 255) & ~uintptr_t(255));
    MTile *it_mt = reinterpret_cast<MTile *>(it_part + (size_t)IT_SPLIT * dp * TB);
    int32_t *it_n_mt = reinterpret_cast<int32_t *>(it_mt + IT_SPLIT * (dp / 128 + 1));
    int32_t *qr_flag = reinterpret_cast<int32_t *>(scal + 8);   // pivots clamped inside the Cholesky QR are not an error
    if (cudaMemsetAsync(flag, 0, sizeof(int32_t), st) != cudaSuccess) return -1;
    widen_pad_kernel<<<(unsigned)(((size_t)n * dp + 255) / 256), 256, 0, st>>>(h_cal, n, d, H32, dp);
    CKL();
    // G = H^T H, C = H^T R (columns >= d of C stay zero)
    int n_sms = 0, dev = 0;
    const bool tc = tc_available() && tc_prepare() == 0 && cudaGetDevice(&dev) == cudaSuccess &&
                    cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n_sms > 0;
    if (tc) {
        // on the tensor cores: transposed copies (the token index becomes the contiguous reduction index), H as it is
        // (bf16), R as three bf16 planes; padded rows and columns are zero
        dim3 tg((unsigned)((n8 + 31) / 32), (unsigned)((dp + 31) / 32));
        transpose_bf16_kernel<<<tg, 256, 0, st>>>(h_cal, n, d, Ht16, dp, (int)n8);
        CKL();
        transpose_split3_kernel<<<tg, 256, 0, st>>>(resid, n, d, Rt16, dp, (int)n8);
        CKL();
        CK(launch_tc_plain(Ht16, dp, Ht16, dp, n, (int)n8, G, dp, mt, n_mt, n_sms, st));
        float *outs[3] = {C, C2, C3};
        for (int pl = 0; pl < 3; ++pl)
            CK(launch_tc_plain(Ht16, dp, Rt16 + (size_t)pl * dp * n8, dp, n, (int)n8, outs[pl], dp, mt, n_mt, n_sms, st));
        sum3_kernel<<<(unsigned)(((size_t)dp * dp + 255) / 256), 256, 0, st>>>(C, C2, C3, (size_t)dp * dp);
        CKL();
    } else {
        CK((gemm<true, false>(dp, dp, n, 1.f, H32, dp, H32, dp, 0.f, G, dp, st)));
        if (cudaMemsetAsync(C, 0, sizeof(float) * (size_t)dp * dp, st) != cudaSuccess) return -1;
        CK((gemm<true, false>(dp, d, n, 1.f, H32, dp, resid, d, 0.f, C, dp, st)));
    }
    mean_diag_kernel<<<1, 256, 0, st>>>(G, dp, d, scal);
    CKL();
    regularise_kernel<<<(unsigned)(((size_t)dp * dp + 255) / 256), 256, 0, st>>>(G, dp, d, dp, ridge, scal);
    CKL();
    CK(cholesky(G, dp, dp, flag, st));
    // Z = L^-1 C, block rows top to bottom (in place in C)
    for (int k = 0; k < dp; k += TB) {
        trsm_left_kernel<false><<<dp / TB, 64, 0, st>>>(C + (size_t)k * dp, dp, dp, G + (size_t)k * dp + k, dp);
        CKL();
        const int rem = dp - k - TB;
        if (rem > 0)
            CK((gemm<false, false>(rem, dp, TB, -1.f, G + (size_t)(k + TB) * dp + k, dp, C + (size_t)k * dp, dp, 1.f,
                                   C + (size_t)(k + TB) * dp, dp, st)));
    }
    float *Z = C;
    // r leading eigenvectors of Z^T Z by block subspace iteration
    init_block_kernel<<<(unsigned)(((size_t)dp * rp + 255) / 256), 256, 0, st>>>(Q, dp, rp, r);
    CKL();
    CK(orthonormalise(Q, dp, rp, r, S, qr_flag, st));
    const bool tc_iter = tc && rp == TB && iters > 0;
    const int k_split = ((3 * dp + IT_SPLIT - 1) / IT_SPLIT + 63) / 64 * 64;
    if (tc_iter) {
        dim3 mg((unsigned)((dp + 31) / 32), (unsigned)((dp + 31) / 32));
        split2_cat_matrix_kernel<false><<<mg, 256, 0, st>>>(Z, dp, dp, Zcat);
        CKL();
        split2_cat_matrix_kernel<true><<<mg, 256, 0, st>>>(Z, dp, dp, Ztcat);
        CKL();
        CK(launch_tc_splitk_tiles(dp, IT_SPLIT, it_mt, it_n_mt, st));
    }
    for (int it = 0; it < iters; ++it) {
        if (tc_iter) {
            // P = Z Q and Q <- Z^T P on the tensor cores (two-term operands, see split2_cat_matrix_kernel), each cut into
            // IT_SPLIT ranges of the reduction whose partial results are added in range order
            dim3 bg((unsigned)((dp + 31) / 32), (unsigned)((rp + 31) / 32));
            const unsigned rb = (unsigned)(((size_t)dp * rp + 255) / 256);
            split2_cat_block_kernel<<<bg, 256, 0, st>>>(Q, dp, rp, Bcat);
            CKL();
            CK(launch_tc_plain_splitk(Zcat, dp, Bcat, rp, k_split, 3 * dp, it_part, rp, it_mt, it_n_mt, n_sms, st));
            splitk_reduce_kernel<<<rb, 256, 0, st>>>(dp, rp, IT_SPLIT, 1.f, it_part, 0.f, P, rp);
            CKL();
            split2_cat_block_kernel<<<bg, 256, 0, st>>>(P, dp, rp, Bcat);
            CKL();
            CK(launch_tc_plain_splitk(Ztcat, dp, Bcat, rp, k_split, 3 * dp, it_part, rp, it_mt, it_n_mt, n_sms, st));
            splitk_reduce_kernel<<<rb, 256, 0, st>>>(dp, rp, IT_SPLIT, 1.f, it_part, 0.f, Q, rp);
            CKL();
        } else {
            CK((gemm<false, false>(dp, rp, dp, 1.f, Z, dp, Q, rp, 0.f, P, rp, st)));     // P = Z Q
            CK((gemm<true, false>(dp, rp, dp, 1.f, Z, dp, P, rp, 0.f, Y, rp, st)));      // Y = Z^T P
            if (cudaMemcpyAsync(Q, Y, sizeof(float) * (size_t)dp * rp, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return -1;
        }
        CK(orthonormalise(Q, dp, rp, r, S, qr_flag, st));
    }
    // B = V = Q;  A^T = W V = L^-T (Z V): block rows bottom to top (in place in P)
    CK((gemm<false, false>(dp, rp, dp, 1.f, Z, dp, Q, rp, 0.f, P, rp, st)));
    for (int k = dp - TB; k >= 0; k -= TB) {
        trsm_left_kernel<true><<<rp / TB, 64, 0, st>>>(P + (size_t)k * rp, rp, rp, G + (size_t)k * dp + k, dp);
        CKL();
        if (k > 0)   // P_{<k} -= L[k, <k]^T P_k
            CK((gemm<true, false>(k, rp, TB, -1.f, G + (size_t)k * dp, dp, P + (size_t)k * rp, rp, 1.f, P, rp, st)));
    }
    write_factors_kernel<<<(unsigned)(((size_t)d * r + 255) / 256), 256, 0, st>>>(Q, P, rp, d, r, A_out, B_out);
    CKL();
    if (loss_out) {
        // objective at the bf16 factors that were written: T2 = (H A^T) B^T, loss = sum (R - T2)^2
        widen_kernel<<<(unsigned)(((size_t)r * d + 255) / 256), 256, 0, st>>>(A_out, (size_t)r * d, A32);
        CKL();
        widen_kernel<<<(unsigned)(((size_t)d * r + 255) / 256), 256, 0, st>>>(B_out, (size_t)d * r, B32);
        CKL();
        CK((gemm<false, true>(n, r, d, 1.f, H32, dp, A32, d, 0.f, T1, rp, st)));      // T1 = H A^T  [n, r]
        CK((gemm<false, true>(n, d, r, 1.f, T1, rp, B32, r, 0.f, H32, dp, st)));      // T2 = T1 B^T [n, d], over H32 (no longer needed)
        if (cudaMemsetAsync(loss_out, 0, 2 * sizeof(float), st) != cudaSuccess) return -1;
        loss_kernel<<<512, 256, 0, st>>>(resid, d, H32, dp, n, d, loss_out);
        CKL();
    }
    t_splitk_ws = nullptr;
    return launches;
}

}  // namespace spice
