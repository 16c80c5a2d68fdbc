// Grouped expert GEMMs for large batches on the 5th-generation tensor cores (tcgen05 + TMEM), fed
// by TMA.  This is the compute-bound regime of the exact resident experts E_e of Sec. 4.2 and of
// the shared expert S of Sec. 2.1: once an expert sees hundreds of tokens the contraction is a
// dense GEMM (arithmetic intensity ~330 FLOP/B at 4096 tokens of a DeepSeek-V2-Lite-shaped layer).
//
//   MODE_ACT : act[row, i]        = silu(X W_g^T)[row,i] * (X W_u^T)[row,i]      (bf16 out)
//   MODE_OUT : out[orow(row), j]  = (act W_d^T)[row, j]                          (fp32 out)
//   MODE_GATED: out[orow(row), j] = gate[orow(row)] * (act W_d^T)[row, j]        (bf16 out: the routed down projection
//              of large batches, whose 6 rows per token the combine then only adds; half the bytes of fp32 rows)
//
// C[M,N] = A[M,K] B[N,K]^T with both operands K-major.  A rows are tokens (gathered so that every
// group is a contiguous row range), B rows are weight rows.  One persistent CTA per SM:
//   warp 0   TMA producer: 128 x 64 A box + 256 rows of B (gate box + up box, or one 256-row box)
//            per k-block into a 4-stage shared-memory ring (128-byte swizzle), mbarrier complete_tx
//   warp 1   issues tcgen05.mma (M=128, N=256, K=16, bf16 -> fp32) on the staged tiles; the
//            accumulator (256 TMEM columns) is double-buffered so the epilogue of tile i overlaps
//            the main loop of tile i+1; tcgen05.commit releases ring stages / publishes accumulators
//   warps 2-5 epilogue: tcgen05.ld 32 lanes x 32 columns at a time, SwiGLU or plain; every warp turns its
//            32 x 32 piece through a private shared-memory buffer so that its global stores are whole
//            16-byte pieces of consecutive columns (a store then touches 4-8 lines instead of 32)
// The same kernel (plain mode) computes the router logits of batches of more than 64 tokens.
// Every wait is bounded: on expiry the CTA records SPICE_ERR_TIMEOUT, stops, drains its own copies
// in flight (again bounded), frees its TMEM and returns.  No load uses cluster multicast.
#include <cuda.h>

#include "spice_internal.cuh"
#include "tc_device.cuh"

namespace spice {

namespace {

using namespace tcdev;

constexpr int BM = 128, BK = 64, BN2 = 256;          // CTA tile: 128 rows x 256 accumulator columns
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN2 * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int TC_THREADS = 192;
constexpr int STG_WARP_BYTES = 32 * 144;             // an epilogue warp's transposition buffer

constexpr uint32_t IDESC = make_idesc(BM, BN2);

// SiLU with the fast reciprocal: the result is rounded to bf16 right after, and under the power cap every
// instruction the epilogue does not issue is clock for the tensor pipe
__device__ __forceinline__ float silu_x(float x) { return __fdividef(x, 1.0f + __expf(-x)); }

struct TcShared {
    alignas(8) unsigned long long full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], mma_drain;
    uint32_t tmem_base;
    int abort_flag;
};

}  // namespace

struct TcGemmArgs {
    const MTile *mtiles;        // device
    const int32_t *n_mtiles;    // device scalar
    int32_t n_ntiles;           // column tiles per m-tile
    int32_t K;                  // reduction length
    int32_t b_rows_per_slot;    // rows of B per slot (2I for gate/up, d for down)
    int32_t b_second_off;       // MODE_ACT: row offset of the second (up) block inside a slot, = I
    int32_t n_cols;             // valid output columns (I or d)
    // epilogue
    __nv_bfloat16 *out16;       // MODE_ACT: [rows, ld]
    float *out32;               // MODE_OUT: [orows, ld]
    const int32_t *row_map;     // MODE_OUT: output row of A row r (entry id), or null for identity
    const float *row_scale;     // MODE_GATED: factor of output row orow (the entry's gate)
    int32_t split_rows;         // plain fp32 mode, product split over its reduction: rows of one partial result (MTile::pad = range)
    int32_t ld;
    int32_t *status;
    uint32_t wait_limit;        // polls after which a pipeline wait gives up (SPICE_OPT_TC_WAIT_LIMIT)
};

template <int MODE>   // 0 = gate/up + SwiGLU, 1 = plain fp32, 2 = plain, scaled per output row, bf16
__global__ void __launch_bounds__(TC_THREADS, 1) tc_grouped_gemm_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                        const __grid_constant__ CUtensorMap map_b,
                                                                        const TcGemmArgs g) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    // ring first (1024-byte aligned tiles), control block after it
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    TcShared *sh = reinterpret_cast<TcShared *>(ring + STAGES * STAGE_BYTES);
    unsigned char *stage_base = ring + STAGES * STAGE_BYTES + 256;   // (TcShared is smaller than 256 bytes)
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh->abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->tmem_full[b]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[b]), 4);
        }
        mbar_init(smem_u32(&sh->mma_drain), 1);
        sh->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const uint32_t wl = g.wait_limit;
    if (warp == 1) {   // TMEM: all 512 columns (two 256-column accumulators)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    const int n_mt = *g.n_mtiles;
    const int n_tiles = n_mt * g.n_ntiles;
    const int kblocks = (g.K + BK - 1) / BK;

    if (warp == 0) {
        // ---------------- TMA producer (one lane)
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const MTile mt = g.mtiles[tile / g.n_ntiles];
                const int nt = tile % g.n_ntiles;
                const int b_row = mt.slot * g.b_rows_per_slot + nt * (MODE == 0 ? 128 : BN2);
                const int k_off = mt.pad * g.K;   // a tile of a product that is split over its reduction takes range `pad`
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(smem_u32(&sh->empty[s]), ((it / STAGES) & 1) ^ 1, abort_flag, wl)) { ok = false; break; }
                    const uint32_t full = smem_u32(&sh->full[s]);
                    const uint32_t dst = smem_u32(ring + s * STAGE_BYTES);
                    mbar_expect_tx(full, STAGE_BYTES);
                    tma_load_2d(dst, &map_a, k_off + kb * BK, mt.row0, full);
                    if (MODE == 0) {
                        tma_load_2d(dst + A_BYTES, &map_b, k_off + kb * BK, b_row, full);                              // gate rows
                        tma_load_2d(dst + A_BYTES + B_BYTES / 2, &map_b, k_off + kb * BK, b_row + g.b_second_off, full);  // up rows
                    } else {
                        tma_load_2d(dst + A_BYTES, &map_b, k_off + kb * BK, b_row, full);
                        tma_load_2d(dst + A_BYTES + B_BYTES / 2, &map_b, k_off + kb * BK, b_row + 128, full);
                    }
                }
            }
            // drain: every stage that was armed must have landed before the CTA may end (also after an abort)
            for (uint32_t j = (it > STAGES ? it - STAGES : 0); j < it; ++j)
                mbar_drain(smem_u32(&sh->full[j % STAGES]), (j / STAGES) & 1);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane)
        if (lane == 0) {
            uint32_t it = 0, tcount = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++tcount) {
                const int buf = tcount & 1;
                if (!mbar_wait(smem_u32(&sh->tmem_empty[buf]), ((tcount >> 1) & 1) ^ 1, abort_flag, wl)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN2;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!mbar_wait(smem_u32(&sh->full[s]), (it / STAGES) & 1, abort_flag, wl)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a0 = smem_u32(ring + s * STAGE_BYTES), b0 = a0 + A_BYTES;
                    const uint64_t da = make_desc(a0), db = make_desc(b0);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)   // 16 bf16 = 32 bytes = 2 descriptor units per step
                        tc_mma(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | k) ? 1u : 0u);
                    tc_commit(smem_u32(&sh->empty[s]));   // stage free once these MMAs have read it
                }
                if (ok) tc_commit(smem_u32(&sh->tmem_full[buf]));
            }
            // every MMA this thread issued must be over before the TMEM columns are given back
            tc_commit(smem_u32(&sh->mma_drain));
            mbar_drain(smem_u32(&sh->mma_drain), 0);
        }
    } else {
        // ---------------- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 = rows of the tile
        const int q = warp & 3;
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, ++tcount) {
            const int buf = tcount & 1;
            const MTile mt = g.mtiles[tile / g.n_ntiles];
            const int nt = tile % g.n_ntiles;
            bool ok = true;
            if (lane == 0) ok = mbar_wait(smem_u32(&sh->tmem_full[buf]), (tcount >> 1) & 1, abort_flag, wl);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            tc_fence_after();
            const int r = q * 32 + lane;                       // row inside the tile
            const bool row_ok = r < mt.rows;
            const uint32_t t0 = tmem_base + buf * BN2 + ((uint32_t)(q * 32) << 16);
            // A thread holds one row of the tile, so a warp-wide store of its registers would touch 32 lines with a
            // few bytes each.  Each warp instead passes 32 columns of its 32 rows through a private piece of shared
            // memory (row pitch chosen so that the 16-byte accesses do not collide) and writes them out with whole
            // 16-byte pieces of consecutive columns per lane: a store then covers 8 (bf16) or 4 (fp32) rows' runs.
            unsigned char *stg = stage_base + (warp - 2) * STG_WARP_BYTES;
            if (MODE == 0) {
                const int col0 = nt * 128;
                constexpr int PITCH = 80;   // 64 B of bf16 per row + 16
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t gv[32], uv[32];
                    tc_ld32(t0 + c, gv);
                    tc_ld32(t0 + 128 + c, uv);
                    tc_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        const float a0 = silu_x(__uint_as_float(gv[j])) * __uint_as_float(uv[j]);
                        const float a1 = silu_x(__uint_as_float(gv[j + 1])) * __uint_as_float(uv[j + 1]);
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(a0, a1);
                        pk[j >> 1] = *reinterpret_cast<uint32_t *>(&b2);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<uint4 *>(stg + lane * PITCH + k * 16) = make_uint4(pk[4 * k], pk[4 * k + 1], pk[4 * k + 2], pk[4 * k + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rr = i * 8 + (lane >> 2), part = lane & 3;
                        const int col = col0 + c + part * 8;
                        const uint4 val = *reinterpret_cast<const uint4 *>(stg + rr * PITCH + part * 16);
                        if (q * 32 + rr < mt.rows && col < g.n_cols)   // (n_cols is a multiple of 8)
                            *reinterpret_cast<uint4 *>(g.out16 + (size_t)(mt.row0 + q * 32 + rr) * g.ld + col) = val;
                    }
                    __syncwarp();
                }
            } else if (MODE == 2) {
                const int col0 = nt * BN2;
                const int out_r = row_ok ? (g.row_map ? g.row_map[mt.row0 + r] : mt.row0 + r) : -1;
                const float sc = out_r >= 0 ? g.row_scale[out_r] : 0.f;
                constexpr int PITCH = 80;   // 64 B of bf16 per row + 16
#pragma unroll 1
                for (int c = 0; c < BN2; c += 32) {
                    uint32_t v[32];
                    tc_ld32(t0 + c, v);
                    tc_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) {
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(sc * __uint_as_float(v[j]), sc * __uint_as_float(v[j + 1]));
                        pk[j >> 1] = *reinterpret_cast<uint32_t *>(&b2);
                    }
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        *reinterpret_cast<uint4 *>(stg + lane * PITCH + k * 16) = make_uint4(pk[4 * k], pk[4 * k + 1], pk[4 * k + 2], pk[4 * k + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int rr = i * 8 + (lane >> 2), part = lane & 3;
                        const int col = col0 + c + part * 8;
                        const int orow = __shfl_sync(0xffffffffu, out_r, rr);
                        const uint4 val = *reinterpret_cast<const uint4 *>(stg + rr * PITCH + part * 16);
                        if (orow >= 0 && col < g.n_cols)   // (n_cols is a multiple of 8)
                            *reinterpret_cast<uint4 *>(g.out16 + (size_t)orow * g.ld + col) = val;
                    }
                    __syncwarp();
                }
            } else {
                const int col0 = nt * BN2;
                const int out_r = row_ok ? (g.row_map ? g.row_map[mt.row0 + r] : mt.row0 + r + mt.pad * g.split_rows) : -1;
                constexpr int PITCH = 144;   // 128 B of fp32 per row + 16
#pragma unroll 1
                for (int c = 0; c < BN2; c += 32) {
                    uint32_t v[32];
                    tc_ld32(t0 + c, v);
                    tc_wait_ld();
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        *reinterpret_cast<uint4 *>(stg + lane * PITCH + k * 16) = make_uint4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int rr = i * 4 + (lane >> 3), part = lane & 7;
                        const int col = col0 + c + part * 4;
                        const int orow = __shfl_sync(0xffffffffu, out_r, rr);
                        const uint4 val = *reinterpret_cast<const uint4 *>(stg + rr * PITCH + part * 16);
                        if (orow >= 0 && col < g.n_cols)   // (n_cols is a multiple of 4)
                            *reinterpret_cast<uint4 *>(g.out32 + (size_t)orow * g.ld + col) = val;
                    }
                    __syncwarp();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[buf]));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && sh->abort_flag && g.status) atomicMax(g.status, (int)SPICE_ERR_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
    }
}

// ---------------------------------------------------------------------------------------------
// helpers around the GEMMs

// x_perm[p, :] = h[perm_hit[p] / K, :]  (rows of one slot become contiguous)
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16 *__restrict__ h, const int32_t *__restrict__ perm,
                                                          const int32_t *__restrict__ hdr, int K, int d,
                                                          __nv_bfloat16 *__restrict__ out) {
    const int n_hit = hdr[HDR_N_HIT];
    const int vec = d >> 3;
    for (int p = blockIdx.x; p < n_hit; p += gridDim.x) {
        const int t = perm[p] / K;
        const uint4 *src = reinterpret_cast<const uint4 *>(h + (size_t)t * d);
        uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)p * d);
        for (int v = threadIdx.x; v < vec; v += blockDim.x) dst[v] = src[v];
    }
}

// m-tiles of the hit groups (group list order), 128 rows each; one warp, a group per lane
__global__ void build_mtiles_kernel(const GroupDesc *__restrict__ groups, const int32_t *__restrict__ hdr, MTile *mtiles,
                                    int32_t *n_mtiles) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    const int n_hg = hdr[HDR_N_HIT_GROUPS];
    int base = 0;
    for (int g0 = 0; g0 < n_hg; g0 += 32) {
        const int gi = 1 + g0 + lane;
        GroupDesc grp{0, 0, 0, 0};
        if (g0 + lane < n_hg) grp = groups[gi];
        const int nt = (grp.m + BM - 1) / BM;
        int inc = nt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        const int first = base + inc - nt;
        for (int j = 0; j < nt; ++j) mtiles[first + j] = MTile{grp.id, grp.off + j * BM, min(BM, grp.m - j * BM), 0};
        base += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) *n_mtiles = base;
}

// m-tiles of the shared expert: all T rows, "slot" 0
__global__ void build_shared_mtiles_kernel(int T, MTile *mtiles, int32_t *n_mtiles) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int n = 0;
    for (int r = 0; r < T; r += BM) mtiles[n++] = MTile{0, r, min(BM, T - r), 0};
    *n_mtiles = n;
}

// ---------------------------------------------------------------------------------------------
// host side
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor [rows, cols] (cols contiguous), box = box_rows x 64 columns, 128-byte swizzle, zero fill
bool make_map(CUtensorMap *m, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// 5-D tensor map (bf16, or bytes) with explicit extents, byte strides (dimensions 1..4) and box; 128-byte swizzle, zero
// fill.  The innermost box extent must be one swizzle span: 64 bf16 elements or 128 bytes.
bool tc_encode_map5(CUtensorMap *m, const void *base, const uint64_t dims[5], const uint64_t strides[4], const uint32_t box[5],
                    int elem_bytes) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t gd[5], gs[4];
    cuuint32_t bx[5], estr[5] = {1, 1, 1, 1, 1};
    for (int i = 0; i < 5; ++i) {
        gd[i] = dims[i];
        bx[i] = box[i];
    }
    for (int i = 0; i < 4; ++i) gs[i] = strides[i];
    return fn(m, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), gd,
              gs, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

namespace {

static_assert(sizeof(TcShared) <= 256, "control block");
constexpr size_t TC_SMEM = STAGES * STAGE_BYTES + 256 + 4 * STG_WARP_BYTES + 1024;

}  // namespace

bool tc_available() { return encode_fn() != nullptr; }

int tc_prepare() {
    if (cudaFuncSetAttribute(tc_grouped_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM) != cudaSuccess)
        return -1;
    if (cudaFuncSetAttribute(tc_grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM) != cudaSuccess)
        return -1;
    if (cudaFuncSetAttribute(tc_grouped_gemm_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM) != cudaSuccess)
        return -1;
    return 0;
}

bool tc_shape_ok(const Dims &dm) {
    // TMA: row pitches must be multiples of 16 bytes (dims are multiples of 8: yes); nothing else is required,
    // partial tiles are zero-filled on load and masked on store
    return dm.d % 8 == 0 && dm.I % 8 == 0 && dm.Is % 8 == 0;
}

// Router logits of a large batch (Eq. 1) as one GEMM on the tensor cores: logits[T, N] = h W_r^T, fp32 out.  The
// router matrix plays the weight operand of "slot" 0 (rows past N are zero-filled by the tensor map).
bool tc_router_ok(const Dims &dm) { return tc_shape_ok(dm) && dm.N <= BN2 && dm.N % 4 == 0; }

int launch_tc_router_logits(const Dims &dm, const __nv_bfloat16 *h, const __nv_bfloat16 *w_router, float *logits,
                            const TcBuffers &b, int n_sms, cudaStream_t st) {
    const uint32_t wait_limit = b.wait_limit ? b.wait_limit : WAIT_LIMIT;
    CUtensorMap ma, mb;
    // (the tile list of the routed experts is free until the grouping has run; the shared expert's list may be in
    // use on the side stream)
    build_shared_mtiles_kernel<<<1, 32, 0, st>>>(dm.T, b.mtiles, b.n_mtiles);
    if (!make_map(&ma, h, dm.T, dm.d, BM) || !make_map(&mb, w_router, dm.N, dm.d, 128)) return -1;
    TcGemmArgs g{};
    g.mtiles = b.mtiles;
    g.n_mtiles = b.n_mtiles;
    g.n_ntiles = 1;
    g.K = dm.d;
    g.b_rows_per_slot = 0;
    g.b_second_off = 0;
    g.n_cols = dm.N;
    g.out32 = logits;
    g.row_map = nullptr;
    g.ld = dm.N;
    g.status = b.status;
    g.wait_limit = wait_limit;
    tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

// A plain product on the tensor cores: out[M, N] (fp32, leading dimension ld) = A[M, K] B[N, K]^T, both operands bf16,
// K-major with row pitch ldk elements (a multiple of 8).  mtiles: room for ceil(M / 128) entries, n_mtiles: one int.
int launch_tc_plain(const __nv_bfloat16 *A, int M, const __nv_bfloat16 *B, int N, int K, int ldk, float *out, int ld, MTile *mtiles,
                    int32_t *n_mtiles, int n_sms, cudaStream_t st) {
    CUtensorMap ma, mb;
    build_shared_mtiles_kernel<<<1, 32, 0, st>>>(M, mtiles, n_mtiles);
    // (make_map takes the row pitch as the column count; columns past K are zero by construction of the callers' buffers)
    if (!make_map(&ma, A, M, ldk, BM) || !make_map(&mb, B, N, ldk, 128)) return -1;
    TcGemmArgs g{};
    g.mtiles = mtiles;
    g.n_mtiles = n_mtiles;
    g.n_ntiles = (N + BN2 - 1) / BN2;
    g.K = K;
    g.b_rows_per_slot = 0;
    g.b_second_off = 0;
    g.n_cols = N;
    g.out32 = out;
    g.row_map = nullptr;
    g.ld = ld;
    g.status = nullptr;
    g.wait_limit = WAIT_LIMIT;
    tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

// tile list of a product split over its reduction: for every range s, the m-tiles of all M rows
__global__ void build_splitk_mtiles_kernel(int M, int n_split, MTile *mtiles, int32_t *n_mtiles) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    int n = 0;
    for (int s = 0; s < n_split; ++s)
        for (int r = 0; r < M; r += BM) mtiles[n++] = MTile{0, r, min(BM, M - r), s};
    *n_mtiles = n;
}

// The same product cut into n_split ranges of k_split reduction elements (a multiple of 64): range s writes its partial
// result to out + s * M * ld (the caller adds them, in range order).  For products with few output tiles: M / 128 tiles
// would leave most SMs idle.  mtiles: room for n_split * ceil(M / 128) entries, built by launch_tc_splitk_tiles.
int launch_tc_splitk_tiles(int M, int n_split, MTile *mtiles, int32_t *n_mtiles, cudaStream_t st) {
    build_splitk_mtiles_kernel<<<1, 32, 0, st>>>(M, n_split, mtiles, n_mtiles);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}
int launch_tc_plain_splitk(const __nv_bfloat16 *A, int M, const __nv_bfloat16 *B, int N, int k_split, int ldk, float *out, int ld,
                           const MTile *mtiles, const int32_t *n_mtiles, int n_sms, cudaStream_t st) {
    CUtensorMap ma, mb;
    if (!make_map(&ma, A, M, ldk, BM) || !make_map(&mb, B, N, ldk, 128)) return -1;
    TcGemmArgs g{};
    g.mtiles = mtiles;
    g.n_mtiles = n_mtiles;
    g.n_ntiles = (N + BN2 - 1) / BN2;
    g.K = k_split;
    g.n_cols = N;
    g.out32 = out;
    g.ld = ld;
    g.split_rows = M;
    g.wait_limit = WAIT_LIMIT;
    tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

// ---- LoRE down-projection z = A_e h of the LOW groups of a large batch, through the same GEMM kernel.
// The low entries' tokens are gathered behind the hit entries' rows of x_perm (rows n_hit + p, p in perm_low order),
// lore_A plays the weight operand with the expert index as the "slot" (r rows each), z lands in tb.z_low at the
// same row numbers (fp32), where lore_b_kernel picks it up.
__global__ void __launch_bounds__(256) gather_low_rows_kernel(const __nv_bfloat16 *__restrict__ h, const int32_t *__restrict__ perm,
                                                              const int32_t *__restrict__ hdr, int K, int d,
                                                              __nv_bfloat16 *__restrict__ out) {
    const int n_hit = hdr[HDR_N_HIT], n_low = hdr[HDR_N_LOW];
    const int vec = d >> 3;
    for (int p = blockIdx.x; p < n_low; p += gridDim.x) {
        const int t = perm[p] / K;
        const uint4 *src = reinterpret_cast<const uint4 *>(h + (size_t)t * d);
        uint4 *dst = reinterpret_cast<uint4 *>(out + (size_t)(n_hit + p) * d);
        for (int v = threadIdx.x; v < vec; v += blockDim.x) dst[v] = src[v];
    }
}

// m-tiles of the LOW groups (they follow the hit groups in the group list); one warp, a group per lane
__global__ void build_low_mtiles_kernel(const GroupDesc *__restrict__ groups, const int32_t *__restrict__ hdr, MTile *mtiles,
                                        int32_t *n_mtiles) {
    if (blockIdx.x != 0 || threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    const int n_hg = hdr[HDR_N_HIT_GROUPS], n_lg = hdr[HDR_N_LOW_GROUPS], n_hit = hdr[HDR_N_HIT];
    int base = 0;
    for (int g0 = 0; g0 < n_lg; g0 += 32) {
        GroupDesc grp{0, 0, 0, 0};
        if (g0 + lane < n_lg) grp = groups[1 + n_hg + g0 + lane];
        const int nt = (grp.m + BM - 1) / BM;
        int inc = nt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += v;
        }
        const int first = base + inc - nt;
        for (int j = 0; j < nt; ++j) mtiles[first + j] = MTile{grp.id, n_hit + grp.off + j * BM, min(BM, grp.m - j * BM), 0};
        base += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) *n_mtiles = base;
}

bool tc_lore_ok(const Dims &dm) { return tc_shape_ok(dm) && dm.r <= BN2 && dm.r % 8 == 0; }

int launch_tc_lore_a(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb, const TcBuffers &b0,
                     int n_sms, cudaStream_t st) {
    CUtensorMap ma, mb;
    const size_t cap = (size_t)dm.T * dm.K;
    // (a tile list of its own: on the side stream the routed GEMMs may be reading theirs at the same time)
    TcBuffers b = b0;
    b.mtiles = b0.mtiles_low;
    b.n_mtiles = b0.n_mtiles_low;
    build_low_mtiles_kernel<<<1, 32, 0, st>>>(tb.groups, tb.hdr, b.mtiles, b.n_mtiles);
    gather_low_rows_kernel<<<n_sms * 2, 256, 0, st>>>(h, tb.perm_low, tb.hdr, dm.K, dm.d, b.x_perm);
    if (!make_map(&ma, b.x_perm, cap, dm.d, BM) || !make_map(&mb, w.lore_A, (uint64_t)dm.N * dm.r, dm.d, 128)) return -1;
    TcGemmArgs g{};
    g.mtiles = b.mtiles;
    g.n_mtiles = b.n_mtiles;
    g.n_ntiles = 1;
    g.K = dm.d;
    g.b_rows_per_slot = dm.r;
    g.b_second_off = 0;
    g.n_cols = dm.r;
    g.out32 = tb.z_low;
    g.row_map = nullptr;
    g.ld = dm.r;
    g.status = tb.status;
    g.wait_limit = b0.wait_limit ? b0.wait_limit : WAIT_LIMIT;
    tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    return cudaGetLastError() == cudaSuccess ? 3 : -1;
}

// The exact-expert part of a large batch: gather, grouped gate/up + SwiGLU, grouped down for the hit groups.
// Results land in tb.part (by entry id) (the shared expert's in tb.part_shared, by token) as fp32, exactly where the
// general kernels put them, so the combine kernel is shared with the general path.
int launch_tc_routed(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                     const TcBuffers &b, int n_sms, cudaStream_t st, const float *gate16) {
    CUtensorMap ma, mb;
    int launches = 0;
    const size_t cap = (size_t)dm.T * dm.K;
    TcGemmArgs g{};
    g.status = tb.status;
    g.wait_limit = b.wait_limit ? b.wait_limit : WAIT_LIMIT;
    // ---- routed experts
    build_mtiles_kernel<<<1, 32, 0, st>>>(tb.groups, tb.hdr, b.mtiles, b.n_mtiles);
    gather_rows_kernel<<<n_sms * 4, 256, 0, st>>>(h, tb.perm_hit, tb.hdr, dm.K, dm.d, b.x_perm);
    launches += 2;
    if (!make_map(&ma, b.x_perm, cap, dm.d, BM) || !make_map(&mb, w.slot_w_gate_up, (uint64_t)dm.S * 2 * dm.I, dm.d, 128))
        return -1;
    g.mtiles = b.mtiles;
    g.n_mtiles = b.n_mtiles;
    g.n_ntiles = (dm.I + 127) / 128;
    g.K = dm.d;
    g.b_rows_per_slot = 2 * dm.I;
    g.b_second_off = dm.I;
    g.n_cols = dm.I;
    g.out16 = b.act16;
    g.ld = dm.I;
    tc_grouped_gemm_kernel<0><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    ++launches;
    if (!make_map(&ma, b.act16, cap, dm.I, BM) || !make_map(&mb, w.slot_w_down, (uint64_t)dm.S * dm.d, dm.I, 128)) return -1;
    g.n_ntiles = (dm.d + BN2 - 1) / BN2;
    g.K = dm.I;
    g.b_rows_per_slot = dm.d;
    g.b_second_off = 0;
    g.n_cols = dm.d;
    g.row_map = tb.perm_hit;
    if (gate16) {
        // gated bf16 rows, each in the first half of the entry's fp32 row of tb.part (so rows of other entries, which the
        // LoRE kernels may be writing as fp32 at the same time on another stream, are not touched)
        g.out16 = reinterpret_cast<__nv_bfloat16 *>(tb.part);
        g.out32 = nullptr;
        g.row_scale = gate16;
        g.ld = 2 * dm.d;
        tc_grouped_gemm_kernel<2><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    } else {
        g.out16 = nullptr;
        g.out32 = tb.part;
        g.ld = dm.d;
        tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    }
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

// The shared expert S of a large batch: one group of all T tokens, A is h itself.  It depends on nothing but h, so
// the caller may run it on a second stream beside the routing chain.
int launch_tc_shared(const Dims &dm, const spice_layer_weights &w, const __nv_bfloat16 *h, const Tables &tb,
                     const TcBuffers &b, int n_sms, cudaStream_t st) {
    CUtensorMap ma, mb;
    int launches = 0;
    TcGemmArgs g{};
    g.status = tb.status;
    g.wait_limit = b.wait_limit ? b.wait_limit : WAIT_LIMIT;
    build_shared_mtiles_kernel<<<1, 32, 0, st>>>(dm.T, b.mtiles_shared, b.n_mtiles_shared);
    ++launches;
    if (!make_map(&ma, h, dm.T, dm.d, BM) || !make_map(&mb, w.shared_w_gate_up, (uint64_t)2 * dm.Is, dm.d, 128)) return -1;
    g.mtiles = b.mtiles_shared;
    g.n_mtiles = b.n_mtiles_shared;
    g.n_ntiles = (dm.Is + 127) / 128;
    g.K = dm.d;
    g.b_rows_per_slot = 2 * dm.Is;
    g.b_second_off = dm.Is;
    g.n_cols = dm.Is;
    g.out16 = b.act_shared16;
    g.out32 = nullptr;
    g.row_map = nullptr;
    g.ld = dm.Is;
    tc_grouped_gemm_kernel<0><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    ++launches;
    if (!make_map(&ma, b.act_shared16, dm.T, dm.Is, BM) || !make_map(&mb, w.shared_w_down, dm.d, dm.Is, 128)) return -1;
    g.n_ntiles = (dm.d + BN2 - 1) / BN2;
    g.K = dm.Is;
    g.b_rows_per_slot = dm.d;
    g.b_second_off = 0;
    g.n_cols = dm.d;
    g.out16 = nullptr;
    g.out32 = tb.part_shared;
    g.ld = dm.d;
    tc_grouped_gemm_kernel<1><<<n_sms, TC_THREADS, TC_SMEM, st>>>(ma, mb, g);
    ++launches;
    return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace spice
