// Fused decode kernel on mma.sync: the whole MoE layer (Eq. 1 routing; Sec. 4.2 hit / low-confidence /
// exact-recovery policy; exact resident experts; shared expert + LoRE surrogate; gate-weighted
// aggregation of Sec. 2.1) in ONE persistent cooperative launch for small batches (T <= 16).
// It serves the shapes the tcgen05 / TMA decode kernel (decode_tc.cu) does not take (dimensions that are
// multiples of 8 but not of 64) and can be selected explicitly (SPICE_OPT_PATH = 3).
//
// The layer is HBM-bound at these batch sizes: every weight byte is needed once and reused by at
// most T tokens.  The kernel therefore is a weight streamer.  One CTA per SM holds the tokens in
// shared memory and is split into two independent 8-warp teams.  The work is a flat list of
// tasks, dealt round-robin to the teams; dependencies between tasks are counters in global memory
// (release add by the producer, acquire poll by the consumer, every poll bounded):
//
//   A  R1   router logits of one expert for all tokens         (no dependency)
//      R2   top-k, gates, classification, residual list,
//           grouping of (t,k) entries by slot / expert         (all R1 done)
//      P1s  16 rows of the shared expert's gate/up + SwiGLU    (no dependency)
//   B  P1   16 rows of gate/up of one hit slot, or 16 rows of
//           LoRE A_e of one low-confidence expert              (R2 done)
//   C  P2   16 rows of a down projection (shared / hit slot),
//           or 128 rows of LoRE B_e                            (all P1 rows done)
//   D  P3   combine: y_t = c_t S(h_t) + sum_k g_k part_{t,k}   (all P2 done)
//
// A task streams its weight rows with 128-bit loads straight into mma.sync.m16n8k16 A fragments
// (the reduction index is permuted identically for both operands, so no shuffle is needed); the
// tokens (B fragments, 8 per n-tile) come from shared memory (P1) or L2 (P2).  The 8 warps of a
// team split the reduction dimension and add their partial tiles in shared memory in a fixed
// order, so results are bit-reproducible.  A release costs a fence of about one memory round trip,
// so a warp counts its finished P1 / P2 tiles in a register and publishes the count once, when it
// first has to wait for the next phase (or leaves).
// Tensor cores are used only because they make the per-byte instruction cost negligible; the
// kernel is bandwidth-bound by construction.
#include "route_device.cuh"
#include "spice_internal.cuh"

namespace spice {

namespace {

constexpr int DT = 512;     // threads per CTA
constexpr int TEAM = 256;   // threads per team
constexpr int TW = 8;       // warps per team
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
// team barrier that also ORs a flag over the team (uniform result)
__device__ __forceinline__ bool team_sync_or(int team, bool flag) {
    int out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\tbar.red.or.pred q, %2, %3, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(out)
        : "r"((int)flag), "r"(team + 1), "r"(TEAM)
        : "memory");
    return out != 0;
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

// Optional timeline recorder (compiled in only with -DSPICE_PROF; used while tuning).
#ifdef SPICE_PROF
constexpr int PROF_TEAMS = 296, PROF_EVENTS = 512;
__device__ unsigned long long g_prof[PROF_TEAMS * PROF_EVENTS * 2];
__device__ __forceinline__ unsigned long long prof_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
#define PROF(tc, tag)                                                                        \
    do {                                                                                     \
        if ((tc).ttid == 0 && (tc).gteam < PROF_TEAMS && (tc).nprof < PROF_EVENTS) {         \
            g_prof[((tc).gteam * PROF_EVENTS + (tc).nprof) * 2] = (unsigned long long)(tag); \
            g_prof[((tc).gteam * PROF_EVENTS + (tc).nprof) * 2 + 1] = prof_now();            \
            (tc).nprof++;                                                                    \
        }                                                                                    \
    } while (0)
#else
#define PROF(tc, tag) \
    do {              \
    } while (0)
#endif
#ifdef SPICE_PROF
#define TC_ARG TeamCtx &
#else
#define TC_ARG TeamCtx
#endif

struct TeamCtx {
#ifdef SPICE_PROF
    int gteam, nprof;
#endif
    int team, ttid, twarp, lane;
    int n_p1, n_p2;      // P1 / P2 tiles this team has finished but not yet published
    bool p1_all;         // this team has seen every P1 tile of the layer published
    float *red;          // [TW][2][NT][128] partial tiles of this team
    int *flag;           // [2] broadcast slots
    GroupDesc *gtab;     // [1 + S + N] team-private copy of the group table
    int *perm_h;         // [T*K] copy of perm_hit
    int *perm_l;         // [T*K] copy of perm_low
};

// the team's global stores are done -> publish one unit of progress
__device__ __forceinline__ void team_signal(const TeamCtx &tc, int *ctr) {
    team_sync(tc.team);
    if (tc.ttid == 0) red_release_add(ctr, 1);
}
// Publish the team's finished-tile counts (every warp of a team holds the same counts): one barrier so
// that all stores of the team are issued, then one release by the leader.  Called before the team waits
// for a later phase and when it leaves the task loop.  One atomic per team and phase: thousands of
// atomics on one address would serialise in L2 and delay the phase change by microseconds.
__device__ __forceinline__ void flush_counts(TeamCtx &tc, int *sync) {
    if (tc.n_p1 | tc.n_p2) {   // team-uniform
        team_sync(tc.team);
        if (tc.ttid == 0) {
            if (tc.n_p1) red_release_add(sync + SY_P1_ALL, tc.n_p1);
            if (tc.n_p2) red_release_add(sync + SY_P2_DONE, tc.n_p2);
        }
        tc.n_p1 = 0;
        tc.n_p2 = 0;
    }
}

// Bounded wait (one thread): true when *ctr >= target, false on abort or when the limit expires,
// in which case the sticky status and the abort flag are set.
__device__ __noinline__ bool wait_ge(const int *ctr, int target, int *sync, int *status, int spin_limit) {
    for (int it = 0; it < spin_limit; ++it) {
        if (ld_acquire(ctr) >= target) return true;
        if ((it & 15) == 15 && ld_relaxed(sync + SY_ABORT)) return false;
        if (it > 32) __nanosleep(32);
    }
    atomicMax(status, (int)SPICE_ERR_TIMEOUT);
    atomicExch(sync + SY_ABORT, 1);
    return false;
}

// leader polls, result is broadcast through a slot: team-uniform result
__device__ __forceinline__ bool team_wait_ge(TeamCtx &tc, const int *ctr, int target, const DecodeParams &p) {
    flush_counts(tc, p.sync);
    if (tc.ttid == 0) tc.flag[0] = wait_ge(ctr, target, p.sync, p.tb.status, p.spin_limit) ? 1 : 0;
    team_sync(tc.team);
    const bool ok = tc.flag[0] != 0;
    team_sync(tc.team);
    return ok;
}

__device__ __forceinline__ GroupDesc load_group(const GroupDesc *g) {
    const int4 v = __ldcg(reinterpret_cast<const int4 *>(g));
    return GroupDesc{v.x, v.y, v.z, v.w};
}

// ------------------------------------------------------------------------------------------
// The weight rows of one task as this lane sees them.
struct WRows {
    const __nv_bfloat16 *p0lo, *p0hi;   // rows g and g+8 of the first matrix
    const __nv_bfloat16 *p1lo, *p1hi;   // same rows of the second matrix (gate/up pair) or unused
    int K;                              // reduction length
    int ks0, ks1;                       // this warp's k-steps
    bool ok_lo, ok_hi;                  // rows g / g+8 of the first matrix exist
    bool ok1_lo, ok1_hi;                // same for the second matrix
};

// One warp: C[16 x 8*NT] += W[rows g, g+8][k] * X[token][k] over this warp's k-steps.
// A k-step covers 32 reduction indices; lane (g = lane/4, c = lane%4) owns indices
// ks*32 + c*8 .. +7 of rows g and g+8 (one 128-bit load each) and of token g of every n-tile.
// The U k-steps of a batch are all loaded before the first mma, so their latencies overlap.
// `gate` (P2 only): called once, after the first batch of weight loads is in flight and before the
// first activation load, to wait for the activations to exist.
template <int NT, bool DUAL, bool B_SMEM, int U, typename Gate>
__device__ __forceinline__ void warp_mma_range(const WRows &w, const unsigned long long (&bptr)[NT],
                                               const bool (&bok)[NT], float (&acc0)[NT][4], float (&acc1)[NT][4],
                                               int lane, Gate gate) {
    const int c = lane & 3;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    bool first = true;
    for (int ks = w.ks0; ks < w.ks1 || first; ks += U) {
        uint4 a0lo[U], a0hi[U], a1lo[U], a1hi[U];
        uint4 bg[B_SMEM ? 1 : U][NT];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kb = (ks + u) * 32 + c * 8;
            const bool in = (ks + u < w.ks1) && (kb < w.K);
            a0lo[u] = (in && w.ok_lo) ? ldg_stream(w.p0lo + kb) : zero;
            a0hi[u] = (in && w.ok_hi) ? ldg_stream(w.p0hi + kb) : zero;
            if (DUAL) {
                a1lo[u] = (in && w.ok1_lo) ? ldg_stream(w.p1lo + kb) : zero;
                a1hi[u] = (in && w.ok1_hi) ? ldg_stream(w.p1hi + kb) : zero;
            }
        }
        if (first) {
            gate();
            first = false;
        }
        if (!B_SMEM) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int kb = (ks + u) * 32 + c * 8;
                const bool in = (ks + u < w.ks1) && (kb < w.K);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn)
                    bg[u][nn] = (in && bok[nn])
                                    ? ldcg128(reinterpret_cast<const unsigned char *>(bptr[nn]) + (size_t)kb * 2)
                                    : zero;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int kb = (ks + u) * 32 + c * 8;
            const bool in = (ks + u < w.ks1) && (kb < w.K);
            if (ks + u < w.ks1) {   // warp-uniform
#pragma unroll
                for (int nn = 0; nn < NT; ++nn) {
                    uint4 b;
                    if (B_SMEM) b = (in && bok[nn]) ? lds128((uint32_t)bptr[nn] + kb * 2) : zero;
                    else b = bg[u][nn];
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

enum { EPI_ACT = 0, EPI_Z = 1, EPI_PART = 2, EPI_PART2 = 3 };

// where row n of a group lands: the token (shared expert), the position in the group's buffer
// (P1 of a hit / low group) or the entry id t*K+k (P2 of a hit / low group)
__device__ __forceinline__ int out_row(const TeamCtx &tc, const GroupDesc &grp, bool by_pos, int n) {
    if (grp.kind == KIND_SHARED) return n;
    if (by_pos) return grp.off + n;
    return (grp.kind == KIND_HIT ? tc.perm_h : tc.perm_l)[grp.off + n];
}

// P2 of a LoRE group: part[entry, j] = sum_q B_e[j,q] z[q]; the reduction (r) is short, so each warp
// takes its own 16 rows and nothing is exchanged.
template <int NT, typename Gate>
__device__ __forceinline__ bool team_block_rows(TeamCtx &tc, const GroupDesc &grp, const __nv_bfloat16 *W, int row0,
                                                int n_rows, int K, const unsigned long long (&bptr)[NT],
                                                const bool (&bok)[NT], float *out32, int ld_out, Gate gate) {
    const int g = tc.lane >> 2, c = tc.lane & 3;
    float acc0[NT][4], acc1[NT][4];
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc0[nn][r] = acc1[nn][r] = 0.f;
    const int r0 = row0 + tc.twarp * 16;
    const int rlo = r0 + g, rhi = r0 + g + 8;
    WRows w;
    w.K = K;
    w.ks0 = 0;
    w.ks1 = (K + 31) >> 5;
    w.ok_lo = rlo < n_rows;
    w.ok_hi = rhi < n_rows;
    w.p0lo = W + (size_t)(w.ok_lo ? rlo : 0) * K;
    w.p0hi = W + (size_t)(w.ok_hi ? rhi : 0) * K;
    w.p1lo = w.p1hi = nullptr;
    w.ok1_lo = w.ok1_hi = false;
    bool failed = false;
    warp_mma_range<NT, false, false, 2>(w, bptr, bok, acc0, acc1, tc.lane, [&]() { failed = !gate(); });
    if (team_sync_or(tc.team, failed)) return false;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = (r & 2) ? rhi : rlo;
            const int n = nn * 8 + 2 * c + (r & 1);
            if (n < grp.m && row < n_rows) out32[(size_t)out_row(tc, grp, false, n) * ld_out + row] = acc0[nn][r];
        }
    tc.n_p2++;
    return true;
}

// ------------------------------------------------------------------------------------------
struct Smem {
    unsigned char *xs;   // [T][d*2 + XPAD] tokens, bf16
    int xstride;
    float *red[2];
    int *flag[2];        // per team: 2 broadcast slots
    GroupDesc *gtab[2];  // per team: copy of the group table
    int *perm_h[2], *perm_l[2];
    // R2 scratch
    float *lg;           // [T][N]
    float *s_conf;       // [T][N] or [T]
    int *s_soe;          // [N]
    int *s_idx;          // [T*K]
    float *s_gate;       // [T*K]
    int *s_slot;         // [T*K]
    unsigned char *s_cls;// [T*K]
    int *cnt_hit, *cnt_low, *off_hit, *off_low;   // [256] each
    int *wt;             // [TW+1]
    int *s_cnt;          // [4]
    int *sel_idx;        // [TW][32] top-k scratch
    float *sel_val;      // [TW][32]
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
    size_t o_small = take(2 * 4 * 4);
    const size_t ng = 1 + (size_t)dm.S + dm.N;
    size_t o_gt0 = take(ng * sizeof(GroupDesc)), o_gt1 = take(ng * sizeof(GroupDesc));
    size_t o_ph0 = take((size_t)n * 4), o_ph1 = take((size_t)n * 4), o_pl0 = take((size_t)n * 4), o_pl1 = take((size_t)n * 4);
    size_t o_lg = take((size_t)dm.T * dm.N * 4);
    size_t o_conf = take((size_t)dm.T * dm.N * 4);
    size_t o_soe = take((size_t)dm.N * 4);
    size_t o_idx = take((size_t)n * 4), o_gate = take((size_t)n * 4), o_slot = take((size_t)n * 4), o_cls = take(n);
    size_t o_hist = take(4 * 256 * 4);
    size_t o_wt = take((TW + 1 + 4) * 4);
    size_t o_sel = take(2 * TW * 32 * 4);
    if (s) {
        s->xs = base + o_xs;
        s->xstride = (int)xstride;
        s->red[0] = reinterpret_cast<float *>(base + o_red0);
        s->red[1] = reinterpret_cast<float *>(base + o_red1);
        int *sm = reinterpret_cast<int *>(base + o_small);
        for (int t = 0; t < 2; ++t) s->flag[t] = sm + t * 4;
        s->gtab[0] = reinterpret_cast<GroupDesc *>(base + o_gt0);
        s->gtab[1] = reinterpret_cast<GroupDesc *>(base + o_gt1);
        s->perm_h[0] = reinterpret_cast<int *>(base + o_ph0);
        s->perm_h[1] = reinterpret_cast<int *>(base + o_ph1);
        s->perm_l[0] = reinterpret_cast<int *>(base + o_pl0);
        s->perm_l[1] = reinterpret_cast<int *>(base + o_pl1);
        s->lg = reinterpret_cast<float *>(base + o_lg);
        s->s_conf = reinterpret_cast<float *>(base + o_conf);
        s->s_soe = reinterpret_cast<int *>(base + o_soe);
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
        s->sel_idx = reinterpret_cast<int *>(base + o_sel);
        s->sel_val = reinterpret_cast<float *>(base + o_sel) + TW * 32;
    }
    return align_up(off, 128);
}

// ------------------------------------------------------------------------------------------
// R1: logits of ONE expert for all tokens; the router row sits in registers, the warps share the
// tokens.  Same arithmetic order as lane_dot_bf16 (see route_device.cuh).
__device__ __noinline__ void task_r1(const DecodeParams &p, unsigned char *smem_raw, TC_ARG tc, int e) {
    const Dims &dm = p.dm;
    const int xstride = dm.d * 2 + XPAD;
    const __nv_bfloat16 *row = reinterpret_cast<const __nv_bfloat16 *>(p.w.w_router) + (size_t)e * dm.d;
    PROF(tc, 60);
    for (int t = tc.twarp; t < dm.T; t += TW) {
        const float sdot = lane_dot_bf16(row, reinterpret_cast<const __nv_bfloat16 *>(smem_raw + (size_t)t * xstride), dm.d,
                                         tc.lane);
        const float tot = warp_sum(sdot);
        if (tc.lane == 0) p.logits[(size_t)t * dm.N + e] = tot;
    }
    PROF(tc, 61);
    team_signal(tc, p.sync + SY_R1_DONE);
    PROF(tc, 62);
}

// exclusive scan across the lanes of a warp; returns the prefix of this lane and the warp total
__device__ __forceinline__ int warp_excl_scan(int v, int lane, int &total) {
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    total = __shfl_sync(0xffffffffu, inc, 31);
    return inc - v;
}

// R2: top-k + gates, classification, residual list, grouping (one team).  Everything between the
// arrival of the logits and the published tables works out of shared memory and is spread over the
// 256 threads: this task is the serial section of the layer, every microsecond of it is paid by all SMs.
// The arithmetic of the gates is that of warp_topk_gates (route_device.cuh), so the fused call and the
// stand-alone router agree bit for bit; the winners are found by the same ranking rule.
__device__ __noinline__ void task_r2(const DecodeParams &p, unsigned char *smem_raw, int nt, TC_ARG tc) {
    const Dims &dm = p.dm;
    Smem sm;
    smem_layout(dm, nt, &sm, smem_raw);
    const int T = dm.T, N = dm.N, K = dm.K, S = dm.S, n = T * K;
    // while the logits are being produced: fetch what classification will need
#pragma unroll 1
    for (int i = tc.ttid; i < N; i += TEAM) sm.s_soe[i] = p.w.slot_of_expert[i];
    const int n_conf = p.conf_stride ? T * N : T;
#pragma unroll 1
    for (int i = tc.ttid; i < n_conf; i += TEAM) sm.s_conf[i] = p.conf[i];
    if (tc.ttid < 4) sm.s_cnt[tc.ttid] = 0;
    sm.cnt_hit[tc.ttid] = 0;
    sm.cnt_low[tc.ttid] = 0;
    PROF(tc, 50);
    if (!team_wait_ge(tc, p.sync + SY_R1_DONE, N, p)) return;
    PROF(tc, 51);
#pragma unroll 1
    for (int i = tc.ttid; i < T * N; i += TEAM) {
        float v = __ldcg(p.logits + i);
        sm.lg[i] = (v == v) ? v : -INFINITY;   // NaN never wins
    }
    team_sync(tc.team);
    PROF(tc, 52);
    // winners by ranking, one (token, expert) pair per thread-step: rank = #{j : l_j > l_e or (l_j == l_e and j < e)}
#pragma unroll 1
    for (int i = tc.ttid; i < T * N; i += TEAM) {
        const int t = i / N, e = i - t * N;
        const float *l = sm.lg + t * N;
        const float v = l[e];
        int rank = 0;
#pragma unroll 4
        for (int j = 0; j < N; ++j) {
            const float u = l[j];
            rank += (u > v) || (u == v && j < e);
        }
        if (rank < K) {
            sm.s_idx[t * K + rank] = e;
            sm.s_gate[t * K + rank] = v;   // the logit for now
        }
    }
    team_sync(tc.team);
    // gates: p_k = exp(l_k - l_0); denominator = sum over the winners in k order, or the full softmax sum
#pragma unroll 1
    for (int t = tc.twarp; t < T; t += TW) {
        const float m = sm.s_gate[t * K];
        float denom = 0.f;
        if (!p.norm_topk) {
            float sacc = 0.f;
#pragma unroll 1
            for (int e = tc.lane; e < N; e += 32) sacc += expf(sm.lg[t * N + e] - m);
            denom = warp_sum(sacc);
        }
        const float pk = (tc.lane < K) ? expf(sm.s_gate[t * K + tc.lane] - m) : 0.f;
        if (p.norm_topk) {
            float sacc = 0.f;
#pragma unroll 1
            for (int k = 0; k < K; ++k) sacc += __shfl_sync(0xffffffffu, pk, k);
            denom = sacc;
        }
        __syncwarp();
        if (tc.lane < K) sm.s_gate[t * K + tc.lane] = pk / denom;
    }
    team_sync(tc.team);
    PROF(tc, 53);
    // classification (Sec. 4.2 policy); s_slot holds the grouping key: slot (HIT), 1024 + e (LOWCONF), -1
#pragma unroll 1
    for (int i = tc.ttid; i < n; i += TEAM) {
        const int e = sm.s_idx[i];
        int sl = sm.s_soe[e], c, key = -1;
        if (sl >= S) {
            atomicMax(p.tb.status, (int)SPICE_ERR_BAD_TABLE);
            c = SPICE_MISS_EXACT;
        } else if (sl >= 0) {
            c = SPICE_HIT;
            key = sl;
            atomicAdd(&sm.cnt_hit[sl], 1);
        } else {
            const int t = i / K;
            const float cf = p.conf_stride ? sm.s_conf[t * N + e] : sm.s_conf[t];
            c = (cf < p.tau) ? SPICE_LOWCONF : SPICE_MISS_EXACT;
            if (c == SPICE_LOWCONF) {
                key = 1024 + e;
                atomicAdd(&sm.cnt_low[e], 1);
            }
        }
        sm.s_cls[i] = (unsigned char)c;
        sm.s_slot[i] = key;
        p.idx[i] = e;
        p.gate[i] = sm.s_gate[i];
        p.cls[i] = (uint8_t)c;
        atomicAdd(&sm.s_cnt[c], 1);
    }
    team_sync(tc.team);
    PROF(tc, 54);
    if (tc.twarp == 0) {
        // residual-miss list (set M of Sec. 4.3) in (t,k) order: 32 entries per step, ballot + popc
        int base = 0;
#pragma unroll 1
        for (int i0 = 0; i0 < n; i0 += 32) {
            const int i = i0 + tc.lane;
            const bool miss = i < n && sm.s_cls[i] == SPICE_MISS_EXACT;
            const unsigned m = __ballot_sync(0xffffffffu, miss);
            if (miss && p.resid_tok) {
                const int o = base + __popc(m & ((1u << tc.lane) - 1u));
                p.resid_tok[o] = i / K;
                p.resid_k[o] = i % K;
                p.resid_expert[o] = sm.s_idx[i];
                p.resid_gate[o] = sm.s_gate[i];
            }
            base += __popc(m);
        }
        if (tc.lane < 3) p.counts[tc.lane] = sm.s_cnt[tc.lane];
    } else if (tc.twarp <= 2) {
        // warp 1: hit groups in slot order; warp 2: low-confidence groups in expert order (8 ids per lane).
        // Both need the number of hit groups, so both count them.
        const bool low = tc.twarp == 2;
        const int *cnt = low ? sm.cnt_low : sm.cnt_hit;
        int *off_out = low ? sm.off_low : sm.off_hit;
        int n_here = 0, g_here = 0, gh_here = 0;
#pragma unroll 1
        for (int j = 0; j < 8; ++j) {
            const int cj = cnt[tc.lane * 8 + j];
            n_here += cj;
            g_here += cj > 0;
            gh_here += sm.cnt_hit[tc.lane * 8 + j] > 0;
        }
        int n_tot, n_g, n_hg;
        int off = warp_excl_scan(n_here, tc.lane, n_tot);
        int gi = warp_excl_scan(g_here, tc.lane, n_g);
        warp_excl_scan(gh_here, tc.lane, n_hg);
        const int gbase = low ? 1 + n_hg : 1;
#pragma unroll 1
        for (int j = 0; j < 8; ++j) {
            const int id = tc.lane * 8 + j;
            const int cj = cnt[id];
            off_out[id] = off;
            if (cj > 0) p.tb.groups[gbase + gi++] = GroupDesc{low ? KIND_LOW : KIND_HIT, id, off, cj};
            off += cj;
        }
        if (tc.lane == 0) {
            if (low) {
                p.tb.hdr[HDR_N_LOW_GROUPS] = n_g;
                p.tb.hdr[HDR_N_LOW] = n_tot;
            } else {
                p.tb.groups[0] = GroupDesc{KIND_SHARED, 0, 0, T};
                p.tb.hdr[HDR_N_HIT_GROUPS] = n_g;
                p.tb.hdr[HDR_N_HIT] = n_tot;
            }
        }
    } else {
        // coefficient of the shared expert's output: 1 + sum of LOWCONF gates, in k order
#pragma unroll 1
        for (int t = tc.ttid - 96; t < T; t += TEAM - 96) {
            float c = 1.0f;
#pragma unroll 1
            for (int k = 0; k < K; ++k)
                if (sm.s_cls[t * K + k] == SPICE_LOWCONF) c += sm.s_gate[t * K + k];
            p.tb.coef_shared[t] = c;
        }
    }
    team_sync(tc.team);
    PROF(tc, 55);
    // position of every entry inside its group = offset of the group + number of earlier entries of the group
#pragma unroll 1
    for (int i = tc.ttid; i < n; i += TEAM) {
        const int key = sm.s_slot[i];
        int pos = -1;
        if (key >= 0) {
            int rank = 0;
#pragma unroll 4
            for (int j = 0; j < i; ++j) rank += sm.s_slot[j] == key;
            if (key < 1024) {
                pos = sm.off_hit[key] + rank;
                p.tb.perm_hit[pos] = i;
            } else {
                pos = sm.off_low[key - 1024] + rank;
                p.tb.perm_low[pos] = i;
            }
        }
        p.tb.pos_of_entry[i] = pos;
    }
    team_sync(tc.team);
    PROF(tc, 56);
    if (tc.ttid == 0) {
        p.tb.hdr[HDR_N_GROUPS] = 0;   // (not used by this kernel)
        red_release_add(p.sync + SY_ROUTE_DONE, 1);
    }
    PROF(tc, 57);
}

// ------------------------------------------------------------------------------------------
// Task list.  ids [0, nA) are known at launch; the rest once the router has published the groups.
struct Plan {
    int n_r1, nA;                       // phase A: R1 tasks, R2, shared gate/up tiles
    int tIs, tI, tr, td_sh, td_hit, tb128, nb;   // tiles per matrix
    int rt_sh, rt_hit;                  // 16-row tiles per P2 task (shared / hit groups)
    int n_hg, n_lg, nB_hit, endB;       // phase B: hit gate/up tiles, LoRE A tiles
    int nC_sh, nC_hit, endC, endD;      // phase C: down tiles; phase D: combine blocks
    bool routed;                        // phases B..D resolvable
};
enum { TK_NONE = 0, TK_R1, TK_R2, TK_P1, TK_P2, TK_P3 };
struct TaskRef {
    int kind, gi, tile;
};

__device__ __forceinline__ TaskRef resolve(const Plan &pl, int id) {
    if (id < pl.nA) {
        if (id < pl.n_r1) return TaskRef{TK_R1, 0, id};
        if (id == pl.n_r1) return TaskRef{TK_R2, 0, 0};
        return TaskRef{TK_P1, 0, id - pl.n_r1 - 1};
    }
    if (!pl.routed || id >= pl.endD) return TaskRef{TK_NONE, 0, 0};
    if (id < pl.endB) {
        const int l = id - pl.nA;
        if (l < pl.nB_hit) return TaskRef{TK_P1, 1 + l / pl.tI, l % pl.tI};
        return TaskRef{TK_P1, 1 + pl.n_hg + (l - pl.nB_hit) / pl.tr, (l - pl.nB_hit) % pl.tr};
    }
    if (id < pl.endC) {
        const int l = id - pl.endB;
        if (l < pl.nC_sh) return TaskRef{TK_P2, 0, l};
        if (l < pl.nC_sh + pl.nC_hit) return TaskRef{TK_P2, 1 + (l - pl.nC_sh) / pl.td_hit, (l - pl.nC_sh) % pl.td_hit};
        const int q = l - pl.nC_sh - pl.nC_hit;
        return TaskRef{TK_P2, 1 + pl.n_hg + q / pl.tb128, q % pl.tb128};
    }
    return TaskRef{TK_P3, 0, id - pl.endC};
}

__device__ __forceinline__ GroupDesc group_of(const DecodeParams &p, const TeamCtx &tc, int gi) {
    if (gi == 0) return GroupDesc{KIND_SHARED, 0, 0, p.dm.T};
    return tc.gtab[gi];
}

// per-lane B rows (token g of every n-tile) of a group
template <int NT, bool B_SMEM>
__device__ __forceinline__ void setup_rows(const DecodeParams &p, uint32_t xs_s, int xstride, const TeamCtx &tc,
                                           const GroupDesc &grp, const unsigned char *b_base, size_t b_row_bytes,
                                           unsigned long long (&bptr)[NT], bool (&bok)[NT]) {
    const int g = tc.lane >> 2;
#pragma unroll
    for (int nn = 0; nn < NT; ++nn) {
        const int n = nn * 8 + g;
        bok[nn] = n < grp.m;
        if (B_SMEM) {
            int tk = 0;
            if (bok[nn])
                tk = (grp.kind == KIND_SHARED) ? n : (grp.kind == KIND_HIT ? tc.perm_h : tc.perm_l)[grp.off + n] / p.dm.K;
            bptr[nn] = (unsigned long long)(xs_s + (uint32_t)(tk * xstride));
        } else {
            bptr[nn] = (unsigned long long)(b_base + (size_t)(bok[nn] ? n : 0) * b_row_bytes);
        }
    }
}

// The first P2 tile of a warp publishes the warp's P1 count and waits (after its first weight loads
// are in flight) until every P1 tile of the layer is published; later tiles do not wait.
struct P1DoneGate {
    const DecodeParams &p;
    TeamCtx &tc;
    int p1_total;
    __device__ __forceinline__ bool operator()() const {
        if (tc.p1_all) return true;
        tc.p1_all = team_wait_ge(tc, p.sync + SY_P1_ALL, p1_total, p);
        return tc.p1_all;
    }
};

// What a task runs as.  Consecutive tasks of one team with the same flavour are executed as one
// software-pipelined run (team_run).
enum { FL_NONE = 0, FL_R1, FL_R2, FL_ACT, FL_Z, FL_PART, FL_PART2, FL_LOREB, FL_P3 };

__device__ __forceinline__ int flavour_of(const Plan &pl, const TeamCtx &tc, const TaskRef &t) {
    if (t.kind == TK_NONE) return FL_NONE;
    if (t.kind == TK_R1) return FL_R1;
    if (t.kind == TK_R2) return FL_R2;
    if (t.kind == TK_P3) return FL_P3;
    const int kind = t.gi == 0 ? KIND_SHARED : tc.gtab[t.gi].kind;
    if (t.kind == TK_P1) return kind == KIND_LOW ? FL_Z : FL_ACT;
    if (kind == KIND_LOW) return FL_LOREB;
    return (kind == KIND_HIT ? pl.rt_hit : pl.rt_sh) == 2 ? FL_PART2 : FL_PART;
}

// Everything one tile needs, resolved from its task.
struct TileArgs {
    GroupDesc grp;
    const __nv_bfloat16 *W0, *W1;   // first rows of the matrix (pair)
    int row0, n_rows, K;
    __nv_bfloat16 *out16;
    float *out32;
    int ld_out;
    const unsigned char *b_base;    // P2: first activation row of the group
};

template <int EPI>
__device__ __forceinline__ TileArgs tile_args(const DecodeParams &p, const TeamCtx &tc, const TaskRef &t) {
    const Dims &dm = p.dm;
    TileArgs a;
    a.grp = group_of(p, tc, t.gi);
    const bool hit = a.grp.kind == KIND_HIT;
    a.out16 = nullptr;
    a.out32 = nullptr;
    a.b_base = nullptr;
    a.W1 = nullptr;
    if (EPI == EPI_ACT) {
        a.n_rows = hit ? dm.I : dm.Is;
        a.K = dm.d;
        a.W0 = hit ? reinterpret_cast<const __nv_bfloat16 *>(p.w.slot_w_gate_up) + (size_t)a.grp.id * 2 * dm.I * dm.d
                   : reinterpret_cast<const __nv_bfloat16 *>(p.w.shared_w_gate_up);
        a.W1 = a.W0 + (size_t)a.n_rows * dm.d;
        a.row0 = t.tile * 16;
        a.out16 = hit ? p.act_hit16 : p.act_shared16;
        a.ld_out = a.n_rows;
    } else if (EPI == EPI_Z) {
        a.n_rows = dm.r;
        a.K = dm.d;
        a.W0 = reinterpret_cast<const __nv_bfloat16 *>(p.w.lore_A) + (size_t)a.grp.id * dm.r * dm.d;
        a.row0 = t.tile * 16;
        a.out16 = p.z16;
        a.ld_out = dm.r;
    } else {
        a.n_rows = dm.d;
        a.K = hit ? dm.I : dm.Is;
        a.W0 = hit ? reinterpret_cast<const __nv_bfloat16 *>(p.w.slot_w_down) + (size_t)a.grp.id * dm.d * dm.I
                   : reinterpret_cast<const __nv_bfloat16 *>(p.w.shared_w_down);
        a.row0 = t.tile * (EPI == EPI_PART2 ? 32 : 16);
        a.out32 = hit ? p.tb.part : p.tb.part_shared;
        a.ld_out = dm.d;
        a.b_base = hit ? reinterpret_cast<const unsigned char *>(p.act_hit16 + (size_t)a.grp.off * dm.I)
                       : reinterpret_cast<const unsigned char *>(p.act_shared16);
    }
    return a;
}

// this lane's weight rows and this warp's share of the reduction
template <int EPI>
__device__ __forceinline__ WRows make_rows(const TileArgs &a, const TeamCtx &tc) {
    constexpr bool DUAL = (EPI == EPI_ACT || EPI == EPI_PART2);
    const int g = tc.lane >> 2;
    const int KS = (a.K + 31) >> 5;
    const int base = KS / TW, rem = KS % TW;
    WRows w;
    w.K = a.K;
    w.ks0 = tc.twarp * base + min(tc.twarp, rem);
    w.ks1 = w.ks0 + base + (tc.twarp < rem ? 1 : 0);
    const int rlo = a.row0 + g, rhi = a.row0 + g + 8;
    // second matrix: the up rows of the same indices, or (EPI_PART2) rows +16 of the same matrix
    const int r1lo = (EPI == EPI_PART2) ? rlo + 16 : rlo, r1hi = (EPI == EPI_PART2) ? rhi + 16 : rhi;
    const __nv_bfloat16 *W1 = (EPI == EPI_PART2) ? a.W0 : a.W1;
    w.ok_lo = rlo < a.n_rows;
    w.ok_hi = rhi < a.n_rows;
    w.ok1_lo = DUAL && r1lo < a.n_rows;
    w.ok1_hi = DUAL && r1hi < a.n_rows;
    w.p0lo = a.W0 + (size_t)(w.ok_lo ? rlo : 0) * a.K;
    w.p0hi = a.W0 + (size_t)(w.ok_hi ? rhi : 0) * a.K;
    w.p1lo = DUAL ? W1 + (size_t)(w.ok1_lo ? r1lo : 0) * a.K : nullptr;
    w.p1hi = DUAL ? W1 + (size_t)(w.ok1_hi ? r1hi : 0) * a.K : nullptr;
    return w;
}

// issue the 128-bit loads of U k-steps starting at ks (rows / k-steps that do not exist give zeros)
template <bool DUAL, int U>
__device__ __forceinline__ void load_batch(const WRows &w, int ks, uint4 (&a0lo)[U], uint4 (&a0hi)[U], uint4 (&a1lo)[U],
                                           uint4 (&a1hi)[U], int c) {
    const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const int kb = (ks + u) * 32 + c * 8;
        const bool in = (ks + u < w.ks1) && (kb < w.K);
        a0lo[u] = (in && w.ok_lo) ? ldg_stream(w.p0lo + kb) : zero;
        a0hi[u] = (in && w.ok_hi) ? ldg_stream(w.p0hi + kb) : zero;
        if (DUAL) {
            a1lo[u] = (in && w.ok1_lo) ? ldg_stream(w.p1lo + kb) : zero;
            a1hi[u] = (in && w.ok1_hi) ? ldg_stream(w.p1hi + kb) : zero;
        }
    }
}

// A run of consecutive tiles of one flavour for one team, reduction split over the 8 warps.
//   EPI_ACT  : W0 = gate rows, W1 = up rows; act[orow][row] = silu(g)*u            (P1 shared / hit)
//   EPI_Z    : z[orow][row] = sum                                                 (P1 LoRE A)
//   EPI_PART : part[orow][row] = sum                                              (P2 down, 16 rows)
//   EPI_PART2: the same for 32 rows: rows +16 share the activation loads          (P2 down, short K)
// The weight loads of a tile's next batch -- or of the NEXT tile's first batch -- are issued before
// the partial sums are exchanged, so the memory pipe stays busy through barriers and epilogue.
// Returns the id of the first task not executed; *alive = 0 (team-uniform) when a wait failed.
template <int NT, int EPI, int UD>
__device__ __forceinline__ int team_run(const DecodeParams &p, const Plan &pl, TeamCtx &tc, uint32_t xs_s, int xstride, int id,
                                     int n_teams, int p1_total, int *alive) {
    constexpr bool DUAL = (EPI == EPI_ACT || EPI == EPI_PART2);
    constexpr bool B_SMEM = (EPI == EPI_ACT || EPI == EPI_Z);
    constexpr int MATS = DUAL ? 2 : 1;
    // k-steps in flight per warp.  More than the bandwidth-delay product only deepens the memory queues
    // (every dependent access on the router's critical path then waits behind them): measured optimum.
    constexpr int U = DUAL ? UD : 2 * UD;
    constexpr int MYFL = EPI == EPI_ACT ? FL_ACT : (EPI == EPI_Z ? FL_Z : (EPI == EPI_PART ? FL_PART : FL_PART2));
    const int c = tc.lane & 3;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    uint4 a0lo[U], a0hi[U], a1lo[U], a1hi[U];
    TileArgs a = tile_args<EPI>(p, tc, resolve(pl, id));
    WRows w = make_rows<EPI>(a, tc);
    load_batch<DUAL, U>(w, w.ks0, a0lo, a0hi, a1lo, a1hi, c);
    bool failed = false;
    if (!B_SMEM && !tc.p1_all) {   // first P2 tile of this team: every P1 tile must be published
        tc.p1_all = team_wait_ge(tc, p.sync + SY_P1_ALL, p1_total, p);   // (publishes the team's own count first)
        failed = !tc.p1_all;
    }
    *alive = 1;
    for (;;) {
        PROF(tc, 100 + (B_SMEM ? TK_P1 : TK_P2));
        const int nid = id + n_teams;
        const TaskRef nt = resolve(pl, nid);
        const bool same = flavour_of(pl, tc, nt) == MYFL;
        unsigned long long bptr[NT];
        bool bok[NT];
        setup_rows<NT, B_SMEM>(p, xs_s, xstride, tc, a.grp, a.b_base, (size_t)a.K * 2, bptr, bok);
        float acc0[NT][4], acc1[NT][4];
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int r = 0; r < 4; ++r) acc0[nn][r] = acc1[nn][r] = 0.f;
        uint4 bg[B_SMEM ? 1 : U][NT];   // activations (P2): fetched one batch ahead, like the weights
        auto load_acts = [&](int ks) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int kb = (ks + u) * 32 + c * 8;
                const bool in = (ks + u < w.ks1) && (kb < w.K);
#pragma unroll
                for (int nn = 0; nn < NT; ++nn)
                    bg[B_SMEM ? 0 : u][nn] =
                        (in && bok[nn]) ? ldcg128(reinterpret_cast<const unsigned char *>(bptr[nn]) + (size_t)kb * 2) : zero;
            }
        };
        if (!B_SMEM) load_acts(w.ks0);
        for (int ks = w.ks0;; ks += U) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int kb = (ks + u) * 32 + c * 8;
                const bool in = (ks + u < w.ks1) && (kb < w.K);
                if (ks + u < w.ks1) {   // warp-uniform
#pragma unroll
                    for (int nn = 0; nn < NT; ++nn) {
                        uint4 b;
                        if (B_SMEM) b = (in && bok[nn]) ? lds128((uint32_t)bptr[nn] + kb * 2) : zero;
                        else b = bg[B_SMEM ? 0 : u][nn];
                        mma_bf16(acc0[nn], a0lo[u].x, a0hi[u].x, a0lo[u].y, a0hi[u].y, b.x, b.y);
                        mma_bf16(acc0[nn], a0lo[u].z, a0hi[u].z, a0lo[u].w, a0hi[u].w, b.z, b.w);
                        if (DUAL) {
                            mma_bf16(acc1[nn], a1lo[u].x, a1hi[u].x, a1lo[u].y, a1hi[u].y, b.x, b.y);
                            mma_bf16(acc1[nn], a1lo[u].z, a1hi[u].z, a1lo[u].w, a1hi[u].w, b.z, b.w);
                        }
                    }
                }
            }
            if (ks + U < w.ks1) {
                load_batch<DUAL, U>(w, ks + U, a0lo, a0hi, a1lo, a1hi, c);
                if (!B_SMEM) load_acts(ks + U);
            } else {
                if (same) {   // first batch of the next tile rides through this tile's exchange and epilogue
                    const TileArgs an = tile_args<EPI>(p, tc, nt);
                    const WRows wn = make_rows<EPI>(an, tc);
                    load_batch<DUAL, U>(wn, wn.ks0, a0lo, a0hi, a1lo, a1hi, c);
                }
                break;
            }
        }
        PROF(tc, 20);
        // every warp is past the previous tile's epilogue once it arrives here
        if (team_sync_or(tc.team, failed)) {
            *alive = 0;
            return nid;
        }
        float *red = tc.red;
#pragma unroll
        for (int nn = 0; nn < NT; ++nn)
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                red[((tc.twarp * MATS + 0) * NT + nn) * 128 + r * 32 + tc.lane] = acc0[nn][r];
                if (DUAL) red[((tc.twarp * MATS + 1) * NT + nn) * 128 + r * 32 + tc.lane] = acc1[nn][r];
            }
        team_sync(tc.team);
        PROF(tc, 21);
        for (int e = tc.ttid; e < NT * 128; e += TEAM) {
            const int nn = e >> 7, r = (e >> 5) & 3, ln = e & 31;
            const int row = a.row0 + (ln >> 2) + ((r & 2) ? 8 : 0);
            const int n = nn * 8 + 2 * (ln & 3) + (r & 1);
            float s0 = 0.f, s1 = 0.f;
#pragma unroll
            for (int wi = 0; wi < TW; ++wi) {
                s0 += red[((wi * MATS + 0) * NT + nn) * 128 + r * 32 + ln];
                if (DUAL) s1 += red[((wi * MATS + 1) * NT + nn) * 128 + r * 32 + ln];
            }
            if (n < a.grp.m && row < a.n_rows) {
                const size_t o = (size_t)out_row(tc, a.grp, B_SMEM, n) * a.ld_out + row;
                if (EPI == EPI_ACT) a.out16[o] = __float2bfloat16(silu_f(s0) * s1);
                else if (EPI == EPI_Z) a.out16[o] = __float2bfloat16(s0);
                else a.out32[o] = s0;
                if (EPI == EPI_PART2 && row + 16 < a.n_rows) a.out32[o + 16] = s1;
            }
        }
        PROF(tc, 22);
        if (B_SMEM) tc.n_p1++;
        else tc.n_p2++;
        id = nid;
        if (!same) break;
        a = tile_args<EPI>(p, tc, nt);
        w = make_rows<EPI>(a, tc);
    }
    return id;
}

// P2 of a LoRE group (short reduction, 128 rows per task); not pipelined, the tasks are tiny
template <int NT>
__device__ __noinline__ bool task_lore_b(const DecodeParams &p, TeamCtx &tc, int gi, int tile, int p1_total) {
    const Dims &dm = p.dm;
    const GroupDesc grp = group_of(p, tc, gi);
    unsigned long long bptr[NT];
    bool bok[NT];
    setup_rows<NT, false>(p, 0u, 0, tc, grp, reinterpret_cast<const unsigned char *>(p.z16 + (size_t)grp.off * dm.r),
                          (size_t)dm.r * 2, bptr, bok);
    const __nv_bfloat16 *W = reinterpret_cast<const __nv_bfloat16 *>(p.w.lore_B) + (size_t)grp.id * dm.d * dm.r;
    return team_block_rows<NT>(tc, grp, W, tile * 128, dm.d, dm.r, bptr, bok, p.tb.part, dm.d, P1DoneGate{p, tc, p1_total});
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

template <int NT, int UD>
__global__ void __launch_bounds__(DT, 1) decode_layer_kernel(const __grid_constant__ DecodeParams p) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const Dims &dm = p.dm;
    TeamCtx tc;
    tc.team = threadIdx.x >> 8;
    tc.ttid = threadIdx.x & (TEAM - 1);
    tc.twarp = tc.ttid >> 5;
    tc.lane = threadIdx.x & 31;
    tc.n_p1 = tc.n_p2 = 0;
    tc.p1_all = false;
#ifdef SPICE_PROF
    tc.gteam = blockIdx.x * 2 + tc.team;
    tc.nprof = 0;
#endif
    PROF(tc, 1);
    {
        Smem sm;
        smem_layout(dm, NT, &sm, smem_raw);
        tc.red = sm.red[tc.team];
        tc.flag = sm.flag[tc.team];
        tc.gtab = sm.gtab[tc.team];
        tc.perm_h = sm.perm_h[tc.team];
        tc.perm_l = sm.perm_l[tc.team];
    }
    const int xstride = dm.d * 2 + XPAD;
    const uint32_t xs_s = (uint32_t)__cvta_generic_to_shared(smem_raw);   // the token tile sits first

    Plan pl;
    pl.n_r1 = p.n_r1;
    pl.tIs = (dm.Is + 15) >> 4;
    pl.tI = (dm.I + 15) >> 4;
    pl.tr = (dm.r + 15) >> 4;
    pl.rt_sh = pl.rt_hit = 1;   // decided once the number of hit groups is known
    pl.td_sh = pl.td_hit = (dm.d + 15) >> 4;
    pl.tb128 = (dm.d + 127) >> 7;
    pl.nb = (dm.d + 1023) >> 10;
    pl.nA = p.n_r1 + 1 + pl.tIs;
    pl.routed = false;
    pl.n_hg = pl.n_lg = pl.nB_hit = pl.endB = pl.nC_sh = pl.nC_hit = pl.endC = pl.endD = 0;

    const int n_teams = gridDim.x * 2;
    int id = blockIdx.x * 2 + tc.team;

    // tokens -> shared memory (bf16, padded rows); 8 loads in flight per thread
    {
        const int vec = dm.d >> 3, total = dm.T * vec;
        for (int v0 = threadIdx.x; v0 < total; v0 += DT * 8) {
            uint4 tmp[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = v0 + i * DT;
                if (v < total) {
                    const int t = v / vec, cidx = v - t * vec;
                    tmp[i] = __ldg(reinterpret_cast<const uint4 *>(p.h + (size_t)t * dm.d + cidx * 8));
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v = v0 + i * DT;
                if (v < total) {
                    const int t = v / vec, cidx = v - t * vec;
                    *reinterpret_cast<uint4 *>(smem_raw + (size_t)t * xstride + cidx * 16) = tmp[i];
                }
            }
        }
    }
    __syncthreads();
    PROF(tc, 2);

    // One dispatch loop: a single call site per tile flavour keeps the code small.  Everything that
    // steers it is uniform across the team (ids, and results of team-wide reductions).
    int alive = 1, p1_total = 0, nC = 0;
    bool p2_ready = false;
    int end = pl.nA;
    while (alive) {
        if (id >= end) {
            if (pl.routed) break;
            // first task beyond phase A: the router's tables are needed from here on
            PROF(tc, 30);
            alive = team_wait_ge(tc, p.sync + SY_ROUTE_DONE, 1, p) ? 1 : 0;
            PROF(tc, 31);
            if (!alive) break;
            // team-private copy of the group table and the permutations: task set-up never goes to L2 again
            // (everything is requested at once, at its maximum size, so this costs one memory round trip)
            pl.n_hg = __ldcg(p.tb.hdr + HDR_N_HIT_GROUPS);
            pl.n_lg = __ldcg(p.tb.hdr + HDR_N_LOW_GROUPS);
            {
                const int ng_max = 1 + min(dm.S, dm.T * dm.K) + min(dm.N, dm.T * dm.K), ne = dm.T * dm.K;
                for (int i = tc.ttid; i < ng_max; i += TEAM) tc.gtab[i] = load_group(p.tb.groups + i);
                for (int i = tc.ttid; i < ne; i += TEAM) {
                    tc.perm_h[i] = __ldcg(p.tb.perm_hit + i);
                    tc.perm_l[i] = __ldcg(p.tb.perm_low + i);
                }
            }
            pl.nB_hit = pl.n_hg * pl.tI;
            pl.endB = pl.nA + pl.nB_hit + pl.n_lg * pl.tr;
            // 32-row down tiles halve the activation reads and the tile-closing overhead per byte, but only pay
            // when every team still gets several of them; with few tiles 16 rows keep more teams busy
            if ((1 + pl.n_hg) * pl.td_sh >= 6 * n_teams) {
                pl.rt_sh = dm.Is <= 4096 ? 2 : 1;
                pl.rt_hit = dm.I <= 4096 ? 2 : 1;
                pl.td_sh = (dm.d + 16 * pl.rt_sh - 1) / (16 * pl.rt_sh);
                pl.td_hit = (dm.d + 16 * pl.rt_hit - 1) / (16 * pl.rt_hit);
            }
            pl.nC_sh = pl.td_sh;
            pl.nC_hit = pl.n_hg * pl.td_hit;
            nC = pl.nC_sh + pl.nC_hit + pl.n_lg * pl.tb128;
            pl.endC = pl.endB + nC;
            pl.endD = pl.endC + dm.T * pl.nb;
            pl.routed = true;
            p1_total = pl.tIs + pl.nB_hit + pl.n_lg * pl.tr;
            end = pl.endD;
            team_sync(tc.team);
            continue;
        }
        const TaskRef t = resolve(pl, id);
        const int fl = flavour_of(pl, tc, t);
        if (fl == FL_ACT) id = team_run<NT, EPI_ACT, UD>(p, pl, tc, xs_s, xstride, id, n_teams, p1_total, &alive);
        else if (fl == FL_Z) id = team_run<NT, EPI_Z, UD>(p, pl, tc, xs_s, xstride, id, n_teams, p1_total, &alive);
        else if (fl == FL_PART2) id = team_run<(NT <= 2 ? NT : 1), EPI_PART2, UD>(p, pl, tc, xs_s, xstride, id, n_teams, p1_total, &alive);
        else if (fl == FL_PART) id = team_run<NT, EPI_PART, UD>(p, pl, tc, xs_s, xstride, id, n_teams, p1_total, &alive);
        else {
            if (fl == FL_R1) {
                PROF(tc, 100 + TK_R1);
                task_r1(p, smem_raw, tc, id);
            } else if (fl == FL_R2) {
                PROF(tc, 100 + TK_R2);
                task_r2(p, smem_raw, NT, tc);
            } else if (fl == FL_LOREB) {
                alive = task_lore_b<NT>(p, tc, t.gi, t.tile, p1_total) ? 1 : 0;
            } else {
                if (!p2_ready) {   // combine needs every down-projected row (counted per warp)
                    alive = team_wait_ge(tc, p.sync + SY_P2_DONE, nC, p) ? 1 : 0;
                    if (!alive) break;
                    p2_ready = true;
                }
                task_p3(p, tc.ttid, t.tile / pl.nb, t.tile % pl.nb);
            }
            id += n_teams;
        }
    }
    // the last team to finish clears the counters for the next launch
    PROF(tc, 40);
    flush_counts(tc, p.sync);
    team_sync(tc.team);
    if (tc.ttid == 0) {
        __threadfence();
        tc.flag[1] = atomicAdd(p.sync + SY_TEAMS_DONE, 1);
    }
    team_sync(tc.team);
    if (tc.flag[1] == n_teams - 1) {
        __threadfence();
        for (int i = tc.ttid; i < p.sync_words; i += TEAM) p.sync[i] = 0;
    }
}

}  // namespace

size_t decode_smem_bytes(const Dims &dm) {
    const int nt = dm.T <= 8 ? 1 : 2;
    return smem_layout(dm, nt, nullptr, nullptr);
}

bool decode_supported(const Dims &dm, size_t max_smem) {
    // beyond 16 tokens the tensor-core path is faster (mma.sync work per weight byte grows with the n-tiles)
    if (dm.T < 1 || dm.T > 16) return false;
    if (dm.N > 256 || dm.S > 256) return false;
    return decode_smem_bytes(dm) <= max_smem;
}

namespace {
// (n-tiles, k-steps in flight per warp).  More in flight than the bandwidth-delay product only deepens the
// memory queues, and every dependent access of the router's critical path then waits behind them; the
// settings are the measured optimum on B200 for both layer shapes.
const void *decode_variant(const Dims &dm) {
    if (dm.T <= 8) return reinterpret_cast<const void *>(decode_layer_kernel<1, 2>);
    return reinterpret_cast<const void *>(decode_layer_kernel<2, 1>);
}
}  // namespace

// once per process and device: allow the kernels the opt-in shared memory size
int decode_prepare(int max_smem_optin) {
    const void *fns[2] = {reinterpret_cast<const void *>(decode_layer_kernel<1, 2>),
                          reinterpret_cast<const void *>(decode_layer_kernel<2, 1>)};
    for (const void *fn : fns)
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem_optin) != cudaSuccess)
            return -1;
    return 0;
}

int launch_decode(const DecodeParams &p, int n_ctas, cudaStream_t st) {
    const size_t smem = decode_smem_bytes(p.dm);
    const void *fn = decode_variant(p.dm);
    void *args[] = {const_cast<DecodeParams *>(&p)};
    if (cudaLaunchCooperativeKernel(fn, dim3(n_ctas), dim3(DT), args, smem, st) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return 1;
}

#ifdef SPICE_PROF
extern "C" int spice_debug_prof_read(unsigned long long *host, size_t n_words) {
    size_t total = sizeof(unsigned long long) * (size_t)PROF_TEAMS * PROF_EVENTS * 2;
    if (n_words * 8 < total) return -1;
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(host, g_prof, total) == cudaSuccess ? 0 : -2;
}
extern "C" int spice_debug_prof_clear(void) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_prof) != cudaSuccess) return -1;
    return cudaMemset(ptr, 0, sizeof(unsigned long long) * (size_t)PROF_TEAMS * PROF_EVENTS * 2) == cudaSuccess ? 0 : -2;
}
#endif

}  // namespace spice
