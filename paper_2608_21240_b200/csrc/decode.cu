// Fused decode kernel: the whole MoE layer (Eq. 1 routing; Sec. 4.2 hit / low-confidence /
// exact-recovery policy; exact resident experts; shared expert + LoRE surrogate; gate-weighted
// aggregation of Sec. 2.1) in ONE persistent cooperative launch for small batches (T <= 32).
//
// The layer is HBM-bound at these batch sizes: every weight byte is needed once and reused by at
// most T tokens.  The kernel therefore is a weight streamer.  One CTA per SM holds the tokens in
// shared memory and is split into two independent 8-warp teams.  The work is a flat list of
// tasks, dealt round-robin to the teams; dependencies between tasks are counters in global memory
// (release add by the producer, acquire poll by the consumer, every poll bounded):
//
//   A  R1   router logits for a slice of experts              (no dependency)
//      R2   top-k, gates, classification, residual list,
//           grouping of (t,k) entries by slot / expert         (all R1 done)
//      P1s  16 rows of the shared expert's gate/up + SwiGLU    (no dependency)
//   B  P1   16 rows of gate/up of one hit slot, or 16 rows of
//           LoRE A_e of one low-confidence expert              (R2 done)
//   C  P2   16 rows of a down projection (shared / hit slot),
//           or 128 rows of LoRE B_e                            (that group's P1 rows done)
//   D  P3   combine: y_t = c_t S(h_t) + sum_k g_k part_{t,k}   (all P2 done)
//
// A task streams its weight rows with 128-bit loads straight into mma.sync.m16n8k16 A fragments
// (the reduction index is permuted identically for both operands, so no shuffle is needed); the
// tokens (B fragments, 8 per n-tile) come from shared memory (P1) or L2 (P2).  The 8 warps of a
// team split the reduction dimension and add their partial tiles in shared memory in a fixed
// order, so results are bit-reproducible.  Tensor cores are used only because they make the
// per-byte instruction cost negligible; the kernel is bandwidth-bound by construction.
#include <cooperative_groups.h>

#include "route_device.cuh"
#include "spice_internal.cuh"

namespace spice {

namespace {

constexpr int DT = 512;     // threads per CTA
constexpr int TEAM = 256;   // threads per team
constexpr int TW = 8;       // warps per team
constexpr int NT_MAX = 4;   // n-tiles of 8 tokens
constexpr int XPAD = 64;    // row padding (bytes) of the token tile in shared memory

__device__ __forceinline__ int ld_acquire(const int *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed(const int *p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add(int *p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void team_sync(int team) {
    asm volatile("bar.sync %0, %1;" ::"r"(team + 1), "r"(TEAM) : "memory");
}
__device__ __forceinline__ uint4 ldcg128(const void *p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

struct TeamCtx {
    int team, ttid, twarp, lane;
    float *red;        // [TW][2][NT][128] partial tiles of this team
    int *tok;          // [32] token of every B row; orow = tok + 32: output row (position, entry id
                       // or token) of every B row; flag = tok + 64: broadcast slot
    __device__ __forceinline__ int *orow() const { return tok + 32; }
    __device__ __forceinline__ int *flag() const { return tok + 64; }
};

// Bounded wait (leader thread only): true when *ctr >= target, false on abort or when the limit
// expires, in which case the sticky status and the abort flag are set.
__device__ bool wait_ge(const int *ctr, int target, int *sync, int *status, int spin_limit) {
    for (int it = 0; it < spin_limit; ++it) {
        if (ld_acquire(ctr) >= target) return true;
        if (ld_relaxed(sync + SY_ABORT)) return false;
        if (it > 64) __nanosleep(64);
    }
    atomicMax(status, (int)SPICE_ERR_TIMEOUT);
    atomicExch(sync + SY_ABORT, 1);
    return false;
}

__device__ __forceinline__ bool team_wait_ge(const TeamCtx &tc, const int *ctr, int target, const DecodeParams &p) {
    if (tc.ttid == 0) *tc.flag() = wait_ge(ctr, target, p.sync, p.tb.status, p.spin_limit) ? 1 : 0;
    team_sync(tc.team);
    const bool ok = *tc.flag() != 0;
    team_sync(tc.team);
    return ok;
}

// all global stores of the team are done -> publish one unit of progress
__device__ __forceinline__ void team_signal(const TeamCtx &tc, int *ctr) {
    team_sync(tc.team);
    if (tc.ttid == 0) {
        __threadfence();
        red_release_add(ctr, 1);
    }
}

// exclusive scan over the 256 threads of a team
__device__ __forceinline__ int team_excl_scan(const TeamCtx &tc, int v, int *wt /* [TW+1] */, int &total) {
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (tc.lane >= o) inc += n;
    }
    team_sync(tc.team);
    if (tc.lane == 31) wt[tc.twarp] = inc;
    team_sync(tc.team);
    if (tc.ttid == 0) {
        int run = 0;
        for (int w = 0; w < TW; ++w) {
            int x = wt[w];
            wt[w] = run;
            run += x;
        }
        wt[TW] = run;
    }
    team_sync(tc.team);
    total = wt[TW];
    return wt[tc.twarp] + inc - v;
}

// ------------------------------------------------------------------------------------------
// One warp: C[16 x 8*NT] += W[row0 + {g, g+8}][k] * X[token][k] over k-steps [ks0, ks1).
// A k-step covers 32 reduction indices; lane (g = lane/4, c = lane%4) owns indices
// ks*32 + c*8 .. +7 of rows g and g+8 (one 128-bit load each) and of token g of every n-tile.
template <int NT, bool DUAL, bool B_SMEM, int U>
__device__ __forceinline__ void warp_mma_range(const __nv_bfloat16 *__restrict__ W0,
                                               const __nv_bfloat16 *__restrict__ W1, int K, int row_lo, int row_hi,
                                               bool ok_lo, bool ok_hi, int ks0, int ks1,
                                               const unsigned long long (&bptr)[NT], const bool (&bok)[NT],
                                               float (&acc0)[NT][4], float (&acc1)[NT][4], int lane) {
    const int c = lane & 3;
    const __nv_bfloat16 *p0lo = W0 + (size_t)row_lo * K, *p0hi = W0 + (size_t)row_hi * K;
    const __nv_bfloat16 *p1lo = DUAL ? W1 + (size_t)row_lo * K : nullptr, *p1hi = DUAL ? W1 + (size_t)row_hi * K : nullptr;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int ks = ks0; ks < ks1; ks += U) {
        uint4 a0lo[U], a0hi[U], a1lo[U], a1hi[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kb = (ks + u) * 32 + c * 8;
            const bool in = (ks + u < ks1) && (kb < K);
            a0lo[u] = (in && ok_lo) ? ldg_stream(p0lo + kb) : zero;
            a0hi[u] = (in && ok_hi) ? ldg_stream(p0hi + kb) : zero;
            if (DUAL) {
                a1lo[u] = (in && ok_lo) ? ldg_stream(p1lo + kb) : zero;
                a1hi[u] = (in && ok_hi) ? ldg_stream(p1hi + kb) : zero;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kb = (ks + u) * 32 + c * 8;
            const bool in = (ks + u < ks1) && (kb < K);
            if (ks + u < ks1) {   // warp-uniform
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    uint4 b = zero;
                    if (in && bok[nn]) {
                        if (B_SMEM) b = lds128((uint32_t)bptr[nn] + kb * 2);
                        else b = ldcg128(reinterpret_cast<const unsigned char *>(bptr[nn]) + (size_t)kb * 2);
                    }
                    mma_bf16(acc0[nn], a0lo[u].x, a0hi[u].x, a0lo[u].y, a0hi[u].y, b.x, b.y);
                    mma_bf16(acc0[nn], a0lo[u].z, a0hi[u].z, a0lo[u].w, a0hi[u].w, b.z, b.w);
                    if (DUAL) {
                        mma_bf16(acc1[nn], a1lo[u].x, a1hi[u].x, a1lo[u].y, a1hi[u].y, b.x, b.y);
                        mma_bf16(acc1[nn], a1lo[u].z, a1hi[u].z, a1lo[u].w, a1hi[u].w, b.z, b.w);
                    }
                }
            }
        }
    }
}

__device__ __forceinline__ GroupDesc load_group(const GroupDesc *g) {
    const int4 v = __ldcg(reinterpret_cast<const int4 *>(g));
    return GroupDesc{v.x, v.y, v.z, v.w};
}

enum { EPI_ACT = 0, EPI_Z = 1, EPI_PART = 2 };

// One team, one 16-row tile, reduction split over the 8 warps.
//   EPI_ACT : rows of W0 = gate, W1 = up; out16[(orow)*ld_out + row] = silu(g)*u          (P1 shared/hit)
//   EPI_Z   : out16[(orow)*ld_out + row] = sum                                            (P1 LoRE A)
//   EPI_PART: out32[(orow)*ld_out + row] = sum                                            (P2 down)
template <int NT, int EPI, bool B_SMEM>
__device__ __forceinline__ void team_tile_ksplit(const TeamCtx &tc, const __nv_bfloat16 *W0, const __nv_bfloat16 *W1,
                                                 int row0, int n_rows, int K, int m,
                                                 const unsigned long long (&bptr)[NT], const bool (&bok)[NT],
                                                 __nv_bfloat16 *out16, float *out32, int ld_out) {
    constexpr bool DUAL = (EPI == EPI_ACT);
    constexpr int MATS = DUAL ? 2 : 1;
    constexpr int U = DUAL ? (NT == 4 ? 2 : 4) : (NT == 4 ? 4 : 8);
    const int g = tc.lane >> 2;
    const int KS = (K + 31) >> 5;
    const int base = KS / TW, rem = KS % TW;
    const int ks0 = tc.twarp * base + min(tc.twarp, rem);
    const int ks1 = ks0 + base + (tc.twarp < rem ? 1 : 0);
    float acc0[NT][4], acc1[NT][4];
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc0[nn][r] = acc1[nn][r] = 0.f;
    const int rlo = row0 + g, rhi = row0 + g + 8;
    const bool ok_lo = rlo < n_rows, ok_hi = rhi < n_rows;
    warp_mma_range<NT, DUAL, B_SMEM, U>(W0, W1, K, ok_lo ? rlo : 0, ok_hi ? rhi : 0, ok_lo, ok_hi, ks0, ks1, bptr, bok,
                                       acc0, acc1, tc.lane);
    float *red = tc.red;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            red[((tc.twarp * MATS + 0) * NT + nn) * 128 + r * 32 + tc.lane] = acc0[nn][r];
            if (DUAL) red[((tc.twarp * MATS + 1) * NT + nn) * 128 + r * 32 + tc.lane] = acc1[nn][r];
        }
    team_sync(tc.team);
    for (int e = tc.ttid; e < NT * 128; e += TEAM) {
        const int nn = e >> 7, r = (e >> 5) & 3, ln = e & 31;
        const int row = row0 + (ln >> 2) + ((r & 2) ? 8 : 0);
        const int n = nn * 8 + 2 * (ln & 3) + (r & 1);
        float s0 = 0.f, s1 = 0.f;
#pragma unroll
        for (int w = 0; w < TW; ++w) {
            s0 += red[((w * MATS + 0) * NT + nn) * 128 + r * 32 + ln];
            if (DUAL) s1 += red[((w * MATS + 1) * NT + nn) * 128 + r * 32 + ln];
        }
        if (n < m && row < n_rows) {
            const size_t o = (size_t)tc.orow()[n] * ld_out + row;
            if (EPI == EPI_ACT) out16[o] = __float2bfloat16(silu_f(s0) * s1);
            else if (EPI == EPI_Z) out16[o] = __float2bfloat16(s0);
            else out32[o] = s0;
        }
    }
}

// P2 of a LoRE group: part[entry, j] = sum_q B_e[j,q] z[q]; the reduction (r) is short, so each warp
// takes its own 16 rows and nothing is exchanged.
template <int NT>
__device__ __forceinline__ void team_block_rows(const TeamCtx &tc, const __nv_bfloat16 *W, int row0, int n_rows,
                                                int K, int m, const unsigned long long (&bptr)[NT],
                                                const bool (&bok)[NT], float *out32, int ld_out) {
    const int g = tc.lane >> 2, c = tc.lane & 3;
    float acc0[NT][4], acc1[NT][4];
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc0[nn][r] = acc1[nn][r] = 0.f;
    const int r0 = row0 + tc.twarp * 16;
    const int rlo = r0 + g, rhi = r0 + g + 8;
    const bool ok_lo = rlo < n_rows, ok_hi = rhi < n_rows;
    warp_mma_range<NT, false, false, 4>(W, nullptr, K, ok_lo ? rlo : 0, ok_hi ? rhi : 0, ok_lo, ok_hi, 0, (K + 31) >> 5,
                                        bptr, bok, acc0, acc1, tc.lane);
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = (r & 2) ? rhi : rlo;
            const int n = nn * 8 + 2 * c + (r & 1);
            if (n < m && row < n_rows) out32[(size_t)tc.orow()[n] * ld_out + row] = acc0[nn][r];
        }
}

// ------------------------------------------------------------------------------------------
struct Smem {
    unsigned char *xs;   // [T][d*2 + XPAD] tokens, bf16
    int xstride;
    float *red[2];
    int *tok[2];         // per team: tok[32], orow[32], flag[4]
    // R2 scratch
    float *lg;           // [T][N]
    int *s_idx;          // [T*K]
    float *s_gate;       // [T*K]
    int *s_slot;         // [T*K]
    unsigned char *s_cls;// [T*K]
    int *cnt_hit, *cnt_low, *off_hit, *off_low;   // [256] each
    int *wt;             // [TW+1]
    int *s_cnt;          // [4]
};

__host__ __device__ inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

__host__ __device__ inline size_t smem_layout(const Dims &dm, int nt, Smem *s, unsigned char *base) {
    size_t off = 0;
    auto take = [&](size_t bytes) {
        off = align_up(off, 128);
        size_t o = off;
        off += bytes;
        return o;
    };
    const int n = dm.T * dm.K;
    const size_t xstride = (size_t)dm.d * 2 + XPAD;
    size_t o_xs = take((size_t)dm.T * xstride);
    size_t o_red0 = take((size_t)TW * 2 * nt * 128 * 4), o_red1 = take((size_t)TW * 2 * nt * 128 * 4);
    size_t o_small = take(2 * (32 + 32 + 4) * 4);
    size_t o_lg = take((size_t)dm.T * dm.N * 4);
    size_t o_idx = take((size_t)n * 4), o_gate = take((size_t)n * 4), o_slot = take((size_t)n * 4), o_cls = take(n);
    size_t o_hist = take(4 * 256 * 4);
    size_t o_wt = take((TW + 1 + 4) * 4);
    if (s) {
        s->xs = base + o_xs;
        s->xstride = (int)xstride;
        s->red[0] = reinterpret_cast<float *>(base + o_red0);
        s->red[1] = reinterpret_cast<float *>(base + o_red1);
        int *sm = reinterpret_cast<int *>(base + o_small);
        for (int t = 0; t < 2; ++t) s->tok[t] = sm + t * 68;
        s->lg = reinterpret_cast<float *>(base + o_lg);
        s->s_idx = reinterpret_cast<int *>(base + o_idx);
        s->s_gate = reinterpret_cast<float *>(base + o_gate);
        s->s_slot = reinterpret_cast<int *>(base + o_slot);
        s->s_cls = base + o_cls;
        int *hist = reinterpret_cast<int *>(base + o_hist);
        s->cnt_hit = hist;
        s->cnt_low = hist + 256;
        s->off_hit = hist + 512;
        s->off_low = hist + 768;
        s->wt = reinterpret_cast<int *>(base + o_wt);
        s->s_cnt = s->wt + TW + 1;
    }
    return align_up(off, 128);
}

// ------------------------------------------------------------------------------------------
// R1: logits of experts [e0, e1) for all tokens; one warp per expert, router row kept in registers
__device__ __noinline__ void task_r1(const DecodeParams &p, unsigned char *smem_raw, int nt, TeamCtx tc, int task) {
    const Dims &dm = p.dm;
    Smem sm;
    smem_layout(dm, nt, &sm, smem_raw);
    const int per = (dm.N + p.n_r1 - 1) / p.n_r1;
    const int e0 = task * per, e1 = min(dm.N, e0 + per);
    const __nv_bfloat16 *wr = reinterpret_cast<const __nv_bfloat16 *>(p.w.w_router);
    const int nsl = (dm.d + 255) >> 8;   // 8-element slices per lane
    for (int e = e0 + tc.twarp; e < e1; e += TW) {
        const __nv_bfloat16 *row = wr + (size_t)e * dm.d;
        if (nsl <= 16) {
            // keep this lane's slices of the router row in registers; same fmaf order as lane_dot_bf16
            uint4 wreg[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int k = i * 256 + tc.lane * 8;
                wreg[i] = (k < dm.d) ? *reinterpret_cast<const uint4 *>(row + k) : make_uint4(0, 0, 0, 0);
            }
            for (int t = 0; t < dm.T; ++t) {
                const __nv_bfloat16 *x = reinterpret_cast<const __nv_bfloat16 *>(sm.xs + (size_t)t * sm.xstride);
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int k = i * 256 + tc.lane * 8;
                    if (k < dm.d) {
                        const uint4 u = wreg[i];
                        const uint4 v = *reinterpret_cast<const uint4 *>(x + k);
                        s = fmaf(bf_lo(u.x), bf_lo(v.x), s); s = fmaf(bf_hi(u.x), bf_hi(v.x), s);
                        s = fmaf(bf_lo(u.y), bf_lo(v.y), s); s = fmaf(bf_hi(u.y), bf_hi(v.y), s);
                        s = fmaf(bf_lo(u.z), bf_lo(v.z), s); s = fmaf(bf_hi(u.z), bf_hi(v.z), s);
                        s = fmaf(bf_lo(u.w), bf_lo(v.w), s); s = fmaf(bf_hi(u.w), bf_hi(v.w), s);
                    }
                }
                const float tot = warp_sum(s);
                if (tc.lane == 0) p.logits[(size_t)t * dm.N + e] = tot;
            }
        } else {
            for (int t = 0; t < dm.T; ++t) {
                const float s = lane_dot_bf16(row, reinterpret_cast<const __nv_bfloat16 *>(sm.xs + (size_t)t * sm.xstride),
                                              dm.d, tc.lane);
                const float tot = warp_sum(s);
                if (tc.lane == 0) p.logits[(size_t)t * dm.N + e] = tot;
            }
        }
    }
    team_signal(tc, p.sync + SY_R1_DONE);
}

// R2: top-k + gates, classification, residual list, grouping (one team)
__device__ __noinline__ void task_r2(const DecodeParams &p, unsigned char *smem_raw, int nt, TeamCtx tc) {
    const Dims &dm = p.dm;
    Smem sm;
    smem_layout(dm, nt, &sm, smem_raw);
    const int T = dm.T, N = dm.N, K = dm.K, S = dm.S, n = T * K;
    if (!team_wait_ge(tc, p.sync + SY_R1_DONE, p.n_r1, p)) return;
    for (int i = tc.ttid; i < T * N; i += TEAM) sm.lg[i] = __ldcg(p.logits + i);
    if (tc.ttid < 4) sm.s_cnt[tc.ttid] = 0;
    sm.cnt_hit[tc.ttid] = 0;
    sm.cnt_low[tc.ttid] = 0;
    team_sync(tc.team);
    for (int t = tc.twarp; t < T; t += TW)
        warp_topk_gates(sm.lg + t * N, N, K, p.norm_topk, tc.lane, sm.s_idx + t * K, sm.s_gate + t * K, nullptr);
    team_sync(tc.team);
    // classification (Sec. 4.2 policy) + ordered residual list (set M of Sec. 4.3)
    int base = 0;
    for (int i0 = 0; i0 < n; i0 += TEAM) {
        const int i = i0 + tc.ttid;
        int c = -1, e = 0, sl = -1;
        if (i < n) {
            e = sm.s_idx[i];
            sl = p.w.slot_of_expert[e];
            if (sl >= S) {
                atomicMax(p.tb.status, (int)SPICE_ERR_BAD_TABLE);
                sl = -1;
                c = SPICE_MISS_EXACT;
            } else if (sl >= 0) {
                c = SPICE_HIT;
                atomicAdd(&sm.cnt_hit[sl], 1);
            } else {
                sl = -1;
                const int t = i / K;
                const float cf = p.conf_stride ? p.conf[(size_t)t * p.conf_stride + e] : p.conf[t];
                c = (cf < p.tau) ? SPICE_LOWCONF : SPICE_MISS_EXACT;
                if (c == SPICE_LOWCONF) atomicAdd(&sm.cnt_low[e], 1);
            }
            sm.s_cls[i] = (unsigned char)c;
            sm.s_slot[i] = sl;
            p.idx[i] = e;
            p.gate[i] = sm.s_gate[i];
            p.cls[i] = (uint8_t)c;
            atomicAdd(&sm.s_cnt[c], 1);
        }
        int total;
        const int pos = team_excl_scan(tc, c == SPICE_MISS_EXACT ? 1 : 0, sm.wt, total);
        if (c == SPICE_MISS_EXACT && p.resid_tok) {
            const int o = base + pos;
            p.resid_tok[o] = i / K;
            p.resid_k[o] = i % K;
            p.resid_expert[o] = e;
            p.resid_gate[o] = sm.s_gate[i];
        }
        base += total;
    }
    team_sync(tc.team);
    if (tc.ttid < 3) p.counts[tc.ttid] = sm.s_cnt[tc.ttid];
    // grouping
    const int ch = sm.cnt_hit[tc.ttid], cl = sm.cnt_low[tc.ttid];
    int n_hit, n_low, n_hg, n_lg;
    const int oh = team_excl_scan(tc, ch, sm.wt, n_hit);
    const int ol = team_excl_scan(tc, cl, sm.wt, n_low);
    const int gh = team_excl_scan(tc, ch > 0 ? 1 : 0, sm.wt, n_hg);
    const int gl = team_excl_scan(tc, cl > 0 ? 1 : 0, sm.wt, n_lg);
    sm.off_hit[tc.ttid] = oh;
    sm.off_low[tc.ttid] = ol;
    if (ch > 0) p.tb.groups[1 + gh] = GroupDesc{KIND_HIT, tc.ttid, oh, ch};
    if (cl > 0) p.tb.groups[1 + n_hg + gl] = GroupDesc{KIND_LOW, tc.ttid, ol, cl};
    if (tc.ttid == 0) {
        p.tb.groups[0] = GroupDesc{KIND_SHARED, 0, 0, T};
        p.tb.hdr[HDR_N_GROUPS] = 1 + n_hg + n_lg;
        p.tb.hdr[HDR_N_HIT_GROUPS] = n_hg;
        p.tb.hdr[HDR_N_LOW_GROUPS] = n_lg;
        p.tb.hdr[HDR_N_HIT] = n_hit;
        p.tb.hdr[HDR_N_LOW] = n_low;
    }
    team_sync(tc.team);
    sm.cnt_hit[tc.ttid] = 0;   // now cursors
    sm.cnt_low[tc.ttid] = 0;
    team_sync(tc.team);
    for (int i0 = 0; i0 < n; i0 += TEAM) {
        const int i = i0 + tc.ttid;
        int key = -1;
        if (i < n) {
            const int c = sm.s_cls[i];
            if (c == SPICE_HIT) key = sm.s_slot[i];
            else if (c == SPICE_LOWCONF) key = 1024 + sm.s_idx[i];
        }
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        int pos = -1;
        if (key >= 0) {
            const int leader = __ffs(peers) - 1;
            int basep = 0;
            if (tc.lane == leader)
                basep = (key < 1024) ? atomicAdd(&sm.cnt_hit[key], __popc(peers))
                                     : atomicAdd(&sm.cnt_low[key - 1024], __popc(peers));
            basep = __shfl_sync(peers, basep, leader);
            const int rank = __popc(peers & ((1u << tc.lane) - 1u));
            if (key < 1024) {
                pos = sm.off_hit[key] + basep + rank;
                p.tb.perm_hit[pos] = i;
            } else {
                pos = sm.off_low[key - 1024] + basep + rank;
                p.tb.perm_low[pos] = i;
            }
        }
        if (i < n) p.tb.pos_of_entry[i] = pos;
    }
    for (int t = tc.ttid; t < T; t += TEAM) {
        float c = 1.0f;
        for (int k = 0; k < K; ++k)
            if (sm.s_cls[t * K + k] == SPICE_LOWCONF) c += sm.s_gate[t * K + k];
        p.tb.coef_shared[t] = c;
    }
    team_signal(tc, p.sync + SY_ROUTE_DONE);
}

// fill the per-team token / output-row tables of a group and the per-lane B pointers
template <int NT, bool B_SMEM>
__device__ __forceinline__ void setup_rows(const DecodeParams &p, uint32_t xs_s, int xstride, const TeamCtx &tc,
                                           const GroupDesc &grp, bool orow_is_pos, const unsigned char *b_base,
                                           size_t b_row_bytes, unsigned long long (&bptr)[NT], bool (&bok)[NT]) {
    // tok[n]: token of row n; orow[n]: output row of row n (position in the group's buffer, or entry id)
    if (tc.ttid < 32) {
        int tk = -1, orow = 0;
        if (tc.ttid < grp.m) {
            if (grp.kind == KIND_SHARED) {
                tk = tc.ttid;
                orow = tc.ttid;
            } else {
                const int entry = __ldcg((grp.kind == KIND_HIT ? p.tb.perm_hit : p.tb.perm_low) + grp.off + tc.ttid);
                tk = entry / p.dm.K;
                orow = orow_is_pos ? grp.off + tc.ttid : entry;
            }
        }
        tc.tok[tc.ttid] = tk;
        tc.orow()[tc.ttid] = orow;
    }
    team_sync(tc.team);
    const int g = tc.lane >> 2;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn) {
        const int n = nn * 8 + g;
        bok[nn] = n < grp.m;
        if (B_SMEM) {
            const int tk = bok[nn] ? tc.tok[n] : 0;
            bptr[nn] = (unsigned long long)(xs_s + (uint32_t)(tk * xstride));
        } else {
            bptr[nn] = (unsigned long long)(b_base + (size_t)(bok[nn] ? n : 0) * b_row_bytes);
        }
    }
}

// P1 task: gate/up + SwiGLU rows of the shared expert or of a hit slot, or LoRE A rows
template <int NT>
__device__ __forceinline__ void task_p1(const DecodeParams &p, uint32_t xs_s, int xstride, const TeamCtx &tc, int gi, int tile) {
    const Dims &dm = p.dm;
    const GroupDesc grp = (gi == 0) ? GroupDesc{KIND_SHARED, 0, 0, dm.T} : load_group(p.tb.groups + gi);
    unsigned long long bptr[NT];
    bool bok[NT];
    setup_rows<NT, true>(p, xs_s, xstride, tc, grp, true, nullptr, 0, bptr, bok);
    if (grp.kind == KIND_LOW) {
        const __nv_bfloat16 *A = reinterpret_cast<const __nv_bfloat16 *>(p.w.lore_A) + (size_t)grp.id * dm.r * dm.d;
        team_tile_ksplit<NT, EPI_Z, true>(tc, A, nullptr, tile * 16, dm.r, dm.d, grp.m, bptr, bok, p.z16, nullptr, dm.r);
    } else if (grp.kind == KIND_HIT) {
        const __nv_bfloat16 *W = reinterpret_cast<const __nv_bfloat16 *>(p.w.slot_w_gate_up) + (size_t)grp.id * 2 * dm.I * dm.d;
        team_tile_ksplit<NT, EPI_ACT, true>(tc, W, W + (size_t)dm.I * dm.d, tile * 16, dm.I, dm.d, grp.m, bptr, bok,
                                            p.act_hit16, nullptr, dm.I);
    } else {
        const __nv_bfloat16 *W = reinterpret_cast<const __nv_bfloat16 *>(p.w.shared_w_gate_up);
        team_tile_ksplit<NT, EPI_ACT, true>(tc, W, W + (size_t)dm.Is * dm.d, tile * 16, dm.Is, dm.d, grp.m, bptr, bok,
                                            p.act_shared16, nullptr, dm.Is);
    }
    team_signal(tc, p.sync + SY_GROUP0 + gi);
}

// P2 task: down-projection rows of one group
template <int NT>
__device__ __forceinline__ bool task_p2(const DecodeParams &p, const TeamCtx &tc, int gi, int tile, int need) {
    const Dims &dm = p.dm;
    if (!team_wait_ge(tc, p.sync + SY_GROUP0 + gi, need, p)) return false;
    const GroupDesc grp = (gi == 0) ? GroupDesc{KIND_SHARED, 0, 0, dm.T} : load_group(p.tb.groups + gi);
    unsigned long long bptr[NT];
    bool bok[NT];
    if (grp.kind == KIND_SHARED) {
        setup_rows<NT, false>(p, 0u, 0, tc, grp, false, reinterpret_cast<const unsigned char *>(p.act_shared16), (size_t)dm.Is * 2,
                              bptr, bok);
        team_tile_ksplit<NT, EPI_PART, false>(tc, reinterpret_cast<const __nv_bfloat16 *>(p.w.shared_w_down), nullptr,
                                              tile * 16, dm.d, dm.Is, grp.m, bptr, bok, nullptr, p.tb.part_shared, dm.d);
    } else if (grp.kind == KIND_HIT) {
        setup_rows<NT, false>(p, 0u, 0, tc, grp, false,
                              reinterpret_cast<const unsigned char *>(p.act_hit16 + (size_t)grp.off * dm.I),
                              (size_t)dm.I * 2, bptr, bok);
        const __nv_bfloat16 *W = reinterpret_cast<const __nv_bfloat16 *>(p.w.slot_w_down) + (size_t)grp.id * dm.d * dm.I;
        team_tile_ksplit<NT, EPI_PART, false>(tc, W, nullptr, tile * 16, dm.d, dm.I, grp.m, bptr, bok, nullptr, p.tb.part,
                                              dm.d);
    } else {
        setup_rows<NT, false>(p, 0u, 0, tc, grp, false, reinterpret_cast<const unsigned char *>(p.z16 + (size_t)grp.off * dm.r),
                              (size_t)dm.r * 2, bptr, bok);
        const __nv_bfloat16 *W = reinterpret_cast<const __nv_bfloat16 *>(p.w.lore_B) + (size_t)grp.id * dm.d * dm.r;
        team_block_rows<NT>(tc, W, tile * 128, dm.d, dm.r, grp.m, bptr, bok, p.tb.part, dm.d);
    }
    team_signal(tc, p.sync + SY_P2_DONE);
    return true;
}

// P3 task: 1024 columns of one token
__device__ __noinline__ void task_p3(const DecodeParams &p, int ttid, int t, int blk) {
    const Dims &dm = p.dm;
    const int j = blk * 1024 + ttid * 4;
    if (j >= dm.d) return;
    const int d = dm.d, K = dm.K;
    const float c = __ldcg(p.tb.coef_shared + t);
    float4 s = __ldcg(reinterpret_cast<const float4 *>(p.tb.part_shared + (size_t)t * d + j));
    float4 acc = make_float4(c * s.x, c * s.y, c * s.z, c * s.w);
    for (int k = 0; k < K; ++k) {
        const int i = t * K + k;
        if (__ldcg(p.tb.pos_of_entry + i) < 0) continue;
        const float g = __ldcg(p.gate + i);
        s = __ldcg(reinterpret_cast<const float4 *>(p.tb.part + (size_t)i * d + j));
        acc.x = fmaf(g, s.x, acc.x); acc.y = fmaf(g, s.y, acc.y);
        acc.z = fmaf(g, s.z, acc.z); acc.w = fmaf(g, s.w, acc.w);
    }
    if (p.y_cpu) {
        s = *reinterpret_cast<const float4 *>(p.y_cpu + (size_t)t * d + j);
        acc.x += s.x; acc.y += s.y; acc.z += s.z; acc.w += s.w;
    }
    __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
    *reinterpret_cast<uint2 *>(p.y16 + (size_t)t * d + j) =
        make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
    if (p.x_resid) {
        const uint2 xr = *reinterpret_cast<const uint2 *>(p.x_resid + (size_t)t * d + j);
        lo = __floats2bfloat162_rn(bf_lo(xr.x) + acc.x, bf_hi(xr.x) + acc.y);
        hi = __floats2bfloat162_rn(bf_lo(xr.y) + acc.z, bf_hi(xr.y) + acc.w);
        *reinterpret_cast<uint2 *>(p.x_resid + (size_t)t * d + j) =
            make_uint2(*reinterpret_cast<uint32_t *>(&lo), *reinterpret_cast<uint32_t *>(&hi));
    }
}

template <int NT>
__global__ void __launch_bounds__(DT, 1) decode_layer_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const Dims &dm = p.dm;
    TeamCtx tc;
    tc.team = threadIdx.x >> 8;
    tc.ttid = threadIdx.x & (TEAM - 1);
    tc.twarp = tc.ttid >> 5;
    tc.lane = threadIdx.x & 31;
    {
        Smem sm;
        smem_layout(dm, NT, &sm, smem_raw);
        tc.red = sm.red[tc.team];
        tc.tok = sm.tok[tc.team];
    }
    const int xstride = dm.d * 2 + XPAD;
    const uint32_t xs_s = (uint32_t)__cvta_generic_to_shared(smem_raw);   // the token tile sits first

    // tokens -> shared memory (bf16, padded rows)
    const int vec = dm.d >> 3;
    for (int v = threadIdx.x; v < dm.T * vec; v += DT) {
        const int t = v / vec, cidx = v - t * vec;
        *reinterpret_cast<uint4 *>(smem_raw + (size_t)t * xstride + cidx * 16) =
            *reinterpret_cast<const uint4 *>(p.h + (size_t)t * dm.d + cidx * 8);
    }
    __syncthreads();

    const int n_teams = gridDim.x * 2;
    const int me = blockIdx.x * 2 + tc.team;
    const int tIs = (dm.Is + 15) >> 4, tI = (dm.I + 15) >> 4, tr = (dm.r + 15) >> 4, td = (dm.d + 15) >> 4;
    const int tb128 = (dm.d + 127) >> 7;
    const int nA = p.n_r1 + 1 + tIs;
    int id = me;
    for (; id < nA; id += n_teams) {
        if (id < p.n_r1) task_r1(p, smem_raw, NT, tc, id);
        else if (id == p.n_r1) task_r2(p, smem_raw, NT, tc);
        else task_p1<NT>(p, xs_s, xstride, tc, 0, id - p.n_r1 - 1);
    }
    // every quantity below is uniform across the team (it comes from broadcast wait results)
    bool alive = team_wait_ge(tc, p.sync + SY_ROUTE_DONE, 1, p);
    if (alive) {
        const int n_hg = __ldcg(p.tb.hdr + HDR_N_HIT_GROUPS), n_lg = __ldcg(p.tb.hdr + HDR_N_LOW_GROUPS);
        const int nB_hit = n_hg * tI, nB = nB_hit + n_lg * tr;
        const int nC_sh = td, nC_hit = n_hg * td, nC = nC_sh + nC_hit + n_lg * tb128;
        const int nb = (dm.d + 1023) >> 10;
        const int nD = dm.T * nb;
        const int endB = nA + nB, endC = endB + nC, endD = endC + nD;
        bool p2_ready = false;
        for (; id < endD && alive; id += n_teams) {
            if (id < endB) {
                const int l = id - nA;
                if (l < nB_hit) task_p1<NT>(p, xs_s, xstride, tc, 1 + l / tI, l % tI);
                else task_p1<NT>(p, xs_s, xstride, tc, 1 + n_hg + (l - nB_hit) / tr, (l - nB_hit) % tr);
            } else if (id < endC) {
                const int l = id - endB;
                if (l < nC_sh) alive = task_p2<NT>(p, tc, 0, l, tIs);
                else if (l < nC_sh + nC_hit) alive = task_p2<NT>(p, tc, 1 + (l - nC_sh) / td, (l - nC_sh) % td, tI);
                else {
                    const int q = l - nC_sh - nC_hit;
                    alive = task_p2<NT>(p, tc, 1 + n_hg + q / tb128, q % tb128, tr);
                }
            } else {
                if (!p2_ready) {   // combine needs every down-projected row
                    alive = team_wait_ge(tc, p.sync + SY_P2_DONE, nC, p);
                    if (!alive) break;
                    p2_ready = true;
                }
                const int l = id - endC;
                task_p3(p, tc.ttid, l / nb, l % nb);
            }
        }
    }
    // the last team to finish clears the counters for the next launch
    team_sync(tc.team);
    if (tc.ttid == 0) {
        __threadfence();
        *tc.flag() = atomicAdd(p.sync + SY_TEAMS_DONE, 1);
    }
    team_sync(tc.team);
    if (*tc.flag() == n_teams - 1) {
        __threadfence();
        for (int i = tc.ttid; i < p.sync_words; i += TEAM) p.sync[i] = 0;
    }
}

}  // namespace

size_t decode_smem_bytes(const Dims &dm) {
    const int nt = dm.T <= 8 ? 1 : (dm.T <= 16 ? 2 : 4);
    return smem_layout(dm, nt, nullptr, nullptr);
}

bool decode_supported(const Dims &dm, size_t max_smem) {
    if (dm.T < 1 || dm.T > 8 * NT_MAX) return false;
    if (dm.N > 256 || dm.S > 256) return false;
    return decode_smem_bytes(dm) <= max_smem;
}

// once per process and device: allow the kernels the opt-in shared memory size
int decode_prepare(int max_smem_optin) {
    const void *fns[3] = {reinterpret_cast<const void *>(decode_layer_kernel<1>),
                          reinterpret_cast<const void *>(decode_layer_kernel<2>),
                          reinterpret_cast<const void *>(decode_layer_kernel<4>)};
    for (const void *fn : fns)
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem_optin) != cudaSuccess)
            return -1;
    return 0;
}

int launch_decode(const DecodeParams &p, int n_ctas, cudaStream_t st) {
    const size_t smem = decode_smem_bytes(p.dm);
    const void *fn;
    if (p.dm.T <= 8) fn = reinterpret_cast<const void *>(decode_layer_kernel<1>);
    else if (p.dm.T <= 16) fn = reinterpret_cast<const void *>(decode_layer_kernel<2>);
    else fn = reinterpret_cast<const void *>(decode_layer_kernel<4>);
    void *args[] = {const_cast<DecodeParams *>(&p)};
    if (cudaLaunchCooperativeKernel(fn, dim3(n_ctas), dim3(DT), args, smem, st) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return 1;
}

}  // namespace spice
