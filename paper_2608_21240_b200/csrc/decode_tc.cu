// Fused decode kernel on the Blackwell tensor-core pipeline: the whole MoE layer (Eq. 1 routing;
// Sec. 4.2 hit / low-confidence / exact-recovery policy; exact resident experts; shared expert +
// LoRE surrogate; gate-weighted aggregation of Sec. 2.1) in ONE persistent cooperative launch for
// small batches (T <= 64).
//
// At these batch sizes the layer is HBM-bound: every weight byte is needed once.  The kernel is a
// weight streamer built like a GEMM with the operands swapped: the WEIGHT rows are the M side of
// the MMA (128 rows per tile), the tokens are the N side (16, 32 or 64 columns), so one
// tcgen05.mma consumes 128 x 16 weight elements per token column and the per-byte instruction
// cost vanishes.  Every group (shared expert, resident slot, low-confidence expert) is computed
// for ALL tokens of the batch -- the tensor core is idle anyway -- and the epilogue keeps only the
// columns of tokens routed to the group; nothing is gathered.
//
// One CTA per SM, 14 warps:
//   warp 0      TMA producer: walks the task list, waits (bounded) for a task's dependency counter,
//               queues the task for the other roles and streams its operands k-chunk by k-chunk
//               (128 weight rows x 128 k + NB token rows x 128 k, as 64-k boxes with 128-byte swizzle) into a
//               shared-memory ring of up to 5 stages of 128 k each; mbarrier complete_tx
//   warp 1      issues tcgen05.mma (M = 128, N = NB, K = 16, bf16 -> fp32 in TMEM); accumulators are
//               double-buffered; tcgen05.commit frees ring stages and publishes accumulators
//   warps 2-5   epilogue: tcgen05.ld, SwiGLU (gate rows in TMEM lanes 0-63, up rows in lanes 64-127,
//               paired through shared memory) or plain; stores; release of the task's counter
//   warps 6-13  auxiliary team: router logits (its share), then the routing decisions computed
//               REDUNDANTLY by every CTA from the logits (top-k, gates, classification, grouping):
//               the tables land in shared memory without a second grid-wide hop (batches of more than
//               32 tokens: each token is routed by one warp of the grid and every CTA collects the
//               entries after one more counter); finally the combine
//
// Tasks (a CTA starts with the id of its index and draws every further id from a global counter; a task
// depends only on tasks with smaller ids, and every CTA issues its tasks in increasing order):
//   A  gate/up tile of the shared expert: 64 gate + 64 up rows, K = d              (no dependency)
//      down tile of the shared expert: 128 rows, one K range                       (the A gate/up tiles)
//      gate/up tiles of the first n_spec slots, streamed before the routing is known when a slot is
//      unlikely to go unused (see launch_decode_tc); such a slot is a group even without a token
//   B  gate/up tile of a resident slot; A_e tile of a low-confidence expert        (routing)
//   C  down tile, 128 rows, of a slot; B_e tile                                    (that group's B tiles)
//   D  combine y_t = c_t S(h_t) + sum_k g_k part_{t,k}  (auxiliary teams)          (all C tiles)
// Dependencies are counters in global memory: red.release by the finishing warp, bounded
// ld.acquire polls by the waiting one.  Data written by plain stores and later fetched by TMA is
// ordered by a fence.proxy.async between the reader's acquire and its TMA copies.  Every wait in the kernel is bounded; on expiry
// the CTA records SPICE_ERR_TIMEOUT, raises the abort flag, drains its copies in flight, frees
// its TMEM and returns.  No load uses cluster multicast.
//
// Second weight precision (decode_tc_kernel<NB, true>): the routed and shared expert weights are E4M3 bytes with one
// fp32 scale per output row (half the bytes of bf16 on the path that is bound by them).  The MMA then runs as
// kind::f8f6f4 with the weights as E4M3 on the M side; the bf16 activations on the N side are written as the exact sum
// of three E5M2 terms (a bf16 has 8 significant bits, an E5M2 three: hi = rn(x), mid = rn(x - hi), lo = rn(x - hi - mid)
// reproduces every bf16 of magnitude 2^-7 .. 57344 exactly and smaller ones to 2^-17 absolute), each term in its own
// group of N columns, so the token side grows from NB to 3 NB columns -- an MMA still takes the same time -- and the
// epilogue adds the three accumulators and applies the row scale.  Nothing is converted per weight element.  The LoRE
// factors and the router stay bf16 (kind::f16 tasks of the same kernel).  A ring stage holds 256 reduction elements of
// such a task (the same 32 KB of weights as 128 bf16 elements).
#include <cuda.h>
#include <cuda_fp8.h>
#include <cmath>

#include "route_device.cuh"
#include "spice_internal.cuh"
#include "tc_device.cuh"

namespace spice {

namespace {

using namespace tcdev;

constexpr int DTC_THREADS = 448;
constexpr int AUX_T0 = 192, AUX_T = 256, AUX_W = 8;
constexpr int MAX_STAGES = 5, TQ = 4;   // deeper rings only lengthen the memory queues (every fence waits behind them)
constexpr int KSTAGE = 128;                 // reduction elements per ring stage: two 64-element sub-chunks
constexpr int KSTAGE8 = 256;                // the same for 8-bit weights: two 128-element sub-chunks
constexpr int SUB_A = 128 * 64 * 2;         // weight bytes of one sub-chunk
constexpr int A_BYTES = 2 * SUB_A;
constexpr int MAX_SPLIT = 16, CHUNKS_PER_SPLIT = 16;

enum { TASK_EXIT = 0, TASK_ACT = 1, TASK_Z = 2, TASK_DOWN = 3 };
enum { MAP_H = 0, MAP_SLOT_GU, MAP_SH_GU, MAP_LORE_A, MAP_SLOT_D, MAP_SH_D, MAP_LORE_B, MAP_ACT_HIT, MAP_ACT_SH, MAP_Z, MAP_X8, N_MAPS };

struct TaskDesc {
    int32_t kind, gi, tile, split, nk;
    int32_t f8;     // 8-bit weights: kind::f8f6f4, three token column groups, 256-element stages
    int32_t pad1, pad2;
};

struct DtcParams {
    DecodeParams p;
    float *part_split;   // [nsplit_sh][T][d] partial sums of the shared expert's down projection
    int32_t stages;      // ring depth
    int32_t nsplit_sh;   // K ranges of the shared down projection
    int32_t cps_sh;      // k-chunks per range
    int32_t r1_sub;      // token subsets per expert in the router-logit units
    int32_t n_spec;      // slots 0 .. n_spec-1 are groups 1 .. n_spec whether or not a token is routed to them: their gate/up
                         // tiles are known at launch and stream while the routing is being computed
    // 8-bit weight precision (decode_tc_kernel<NB, true>): row scales, and the activations as three E5M2 planes
    const float *s_slot_gu, *s_slot_d, *s_sh_gu, *s_sh_d;   // [S,2I], [S,d], [2Is], [d]
    uint8_t *act8_hit;   // [group][3][T][I]
    uint8_t *act8_sh;    // [3][T][Is]
    uint8_t *x8_h;       // [3][T][d]: the input activations, written by the auxiliary teams at the start of the kernel
};
struct DtcMaps {
    CUtensorMap m[N_MAPS];
};

struct Ctl {
    alignas(8) unsigned long long full[MAX_STAGES], empty[MAX_STAGES];
    unsigned long long tmem_full[2], tmem_empty[2];
    unsigned long long tq_full[TQ], tq_empty[TQ];
    unsigned long long xch_full[2], xch_empty[2];
    unsigned long long plan_ready, mma_drain, logits_done;
    TaskDesc tq[TQ];
    uint32_t tmem_base;
    int abort_flag;
    int n_hg, n_lg;
    int aux_flag;
    int last_flag;
    int no_more;   // the producer has issued its last task
    int wsum[2][AUX_W];
};

// auxiliary team's shared memory (routing scratch and the tables every role reads)
struct AuxSmem {
    float *conf, *gate, *coef, *xch;
    int *soe, *idx, *pos, *perm_h, *perm_l, *off_hit, *off_low;
    uint32_t *mask_hit, *mask_low;   // [S][2], [N][2] members of a slot's / an expert's group as a bit mask over the tokens
    int *ready;   // [1 + S + N] group g's gate/up (or A_e) tiles are all published (set by the watcher warp)
    unsigned char *cls;
    GroupDesc *gtab;
};

__host__ __device__ inline size_t up16(size_t v) { return (v + 15) & ~size_t(15); }

// Shared memory is what bounds the depth of the weight ring, so the auxiliary team's part is kept small: confidences are
// staged in shared memory only while they are few (else classification reads them from L2) and the routing tables are
// sized by the slot and expert counts, and the exchange area of the SwiGLU epilogue covers 32 token columns at a time.
// (32 token columns then have 5 ring stages instead of 4, 64 columns 4 instead of 3.)
__host__ __device__ inline bool conf_staged(const Dims &dm, int conf_stride) {
    return (conf_stride ? (size_t)dm.T * dm.N : (size_t)dm.T) <= 1024;
}
// the SwiGLU epilogue's exchange area: two buffers of min(nb, 32) token columns x 64 rows (one buffer would serialise the
// epilogue's two halves: measured slower)
__host__ __device__ inline size_t xch_floats(int nb) { return (size_t)2 * (nb > 32 ? 32 : nb) * 64; }

__host__ __device__ inline size_t aux_layout(const Dims &dm, int conf_stride, int nb, AuxSmem *s, unsigned char *base) {
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += up16(bytes);
        return o;
    };
    const size_t n = (size_t)dm.T * dm.K, TN = (size_t)dm.T * dm.N;
    const size_t o_conf = take(conf_staged(dm, conf_stride) ? (conf_stride ? TN : (size_t)dm.T) * 4 : 0), o_gate = take(n * 4);
    const size_t o_coef = take((size_t)dm.T * 4), o_xch = take(xch_floats(nb) * 4);
    const size_t o_soe = take((size_t)dm.N * 4), o_idx = take(n * 4), o_pos = take(n * 4);
    const size_t o_ph = take(n * 4), o_pl = take(n * 4), o_hist = take((size_t)3 * (dm.S + dm.N) * 4);
    const size_t o_cls = take(n), o_gt = take((1 + (size_t)dm.S + dm.N) * sizeof(GroupDesc));
    const size_t o_rdy = take((1 + (size_t)dm.S + dm.N) * 4);
    if (s) {
        s->conf = reinterpret_cast<float *>(base + o_conf);
        s->gate = reinterpret_cast<float *>(base + o_gate);
        s->coef = reinterpret_cast<float *>(base + o_coef);
        s->xch = reinterpret_cast<float *>(base + o_xch);
        s->soe = reinterpret_cast<int *>(base + o_soe);
        s->idx = reinterpret_cast<int *>(base + o_idx);
        s->pos = reinterpret_cast<int *>(base + o_pos);
        s->perm_h = reinterpret_cast<int *>(base + o_ph);
        s->perm_l = reinterpret_cast<int *>(base + o_pl);
        int *hist = reinterpret_cast<int *>(base + o_hist);
        s->off_hit = hist;                                                    // [S]
        s->off_low = hist + dm.S;                                             // [N]
        s->mask_hit = reinterpret_cast<uint32_t *>(hist + dm.S + dm.N);       // [2 S]
        s->mask_low = reinterpret_cast<uint32_t *>(hist + 3 * dm.S + dm.N);   // [2 N]
        s->cls = base + o_cls;
        s->gtab = reinterpret_cast<GroupDesc *>(base + o_gt);
        s->ready = reinterpret_cast<int *>(base + o_rdy);
    }
    return off;
}

__host__ __device__ inline int nb_of(int T) { return T <= 16 ? 16 : (T <= 32 ? 32 : 64); }
__host__ __device__ inline int stage_bytes_of(int nb, bool f8 = false) { return A_BYTES + (f8 ? 6 : 2) * nb * 128; }

// ------------------------------------------------------------------------------------------
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
__device__ __forceinline__ int ld_acquire_cta(const int *p) {
    int v;
    asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"((uint32_t)__cvta_generic_to_shared(p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_cta(int *p, int v) {
    asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"((uint32_t)__cvta_generic_to_shared(p)), "r"(v) : "memory");
}
__device__ __forceinline__ void cp_async4(uint32_t dst, const void *src) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void aux_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Bounded wait of ONE thread on a dependency counter: true when *ctr >= target; false on abort or when
// the limit expires, in which case the sticky status and both abort flags are set.
__device__ __noinline__ bool wait_ge(const int *ctr, int target, int *sync, int *status, int spin_limit, volatile int *cta_abort) {
    for (int it = 0; it < spin_limit; ++it) {
        if (ld_acquire(ctr) >= target) return true;
        if ((it & 15) == 15 && (ld_relaxed(sync + SY_ABORT) || *cta_abort)) {
            *cta_abort = 1;
            return false;
        }
        if (it > 32) __nanosleep(32);
    }
    atomicMax(status, (int)SPICE_ERR_TIMEOUT);
    atomicExch(sync + SY_ABORT, 1);
    *cta_abort = 1;
    return false;
}

__device__ __forceinline__ unsigned long long now_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Optional timeline recorder (compiled in only with -DSPICE_PROF; used while tuning).
#ifdef SPICE_PROF
constexpr int PR_CTAS = 148, PR_ROLES = 4, PR_EVENTS = 512;
__device__ unsigned long long g_dtc_prof[PR_CTAS * PR_ROLES * PR_EVENTS * 2];
__device__ unsigned long long g_dtc_cal[PR_CTAS * 4];   // (global ns, cycle counter) at the start and end of each CTA
#define DPROF(role, cnt, tag)                                                                 \
    do {                                                                                      \
        if (blockIdx.x < PR_CTAS && (cnt) < PR_EVENTS) {                                      \
            const size_t o_ = (((size_t)blockIdx.x * PR_ROLES + (role)) * PR_EVENTS + (cnt)) * 2; \
            g_dtc_prof[o_] = (unsigned long long)(tag);                                       \
            g_dtc_prof[o_ + 1] = (unsigned long long)clock64();                               \
            ++(cnt);                                                                          \
        }                                                                                     \
    } while (0)
#else
#define DPROF(role, cnt, tag) \
    do {                      \
    } while (0)
#endif
#define APROF(a, tag)                                \
    do {                                             \
        if ((a).atid == 0) DPROF(2, (a).npf, tag);   \
    } while (0)

// limits in SM clock cycles (clock64 is a cheap local counter; the global timer costs about a microsecond to read)
constexpr long long ROLE_WAIT_CYCLES = 2000000000ll;   // a role gives up after about a second without progress
constexpr long long DRAIN_WAIT_CYCLES = 400000000ll;

// mbarrier wait bounded by elapsed cycles (a try_wait may itself suspend the thread for a while, so polls are
// not a measure); false when the limit expired or another role already gave up
__device__ __forceinline__ bool mb_wait(uint32_t a, uint32_t parity, volatile int *abort_flag) {
    if (mbar_try(a, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try(a, parity)) return true;
        if (i > 16u) __nanosleep(20);   // leave the issue slots to the warps that have work
        if ((i & 31u) == 0u) {
            if (*abort_flag) return false;
            if (clock64() - t0 > ROLE_WAIT_CYCLES) break;
        }
    }
    *abort_flag = 1;
    return false;
}
// the same without the abort check, for waits that must outlast an abort (copies / MMAs in flight)
__device__ __forceinline__ void mb_drain(uint32_t a, uint32_t parity) {
    const long long t0 = clock64();
    for (uint32_t i = 1;; ++i) {
        if (mbar_try(a, parity)) return;
        if ((i & 31u) == 0u && clock64() - t0 > DRAIN_WAIT_CYCLES) return;
    }
}

// whole warp: lane 0 polls (bounded), the outcome is warp-uniform; every lane then observes the completed phase itself
__device__ __forceinline__ bool warp_mb_wait(uint32_t a, uint32_t parity, volatile int *abort_flag, int lane) {
    bool ok = true;
    if (lane == 0) ok = mb_wait(a, parity, abort_flag);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) (void)mbar_try(a, parity);
    return ok;
}

// v[nn] for a register array and an index known only at run time (the same in every lane): a tree of selects on the bits of nn
template <int N>
__device__ __forceinline__ uint32_t pick_column(const uint32_t (&v)[N], int nn) {
    uint32_t s[N / 2];
#pragma unroll
    for (int i = 0; i < N / 2; ++i) s[i] = (nn & 1) ? v[2 * i + 1] : v[2 * i];
#pragma unroll
    for (int w = N / 4, bit = 2; w >= 1; w >>= 1, bit <<= 1) {
#pragma unroll
        for (int i = 0; i < w; ++i) s[i] = (nn & bit) ? s[2 * i + 1] : s[2 * i];
    }
    return s[0];
}

// ------------------------------------------------------------------------------------------
// Task list.  ids [0, nA) are known at launch; the rest once the routing tables exist.
struct Plan {
    int tIs, tI, tz, td;            // tiles per matrix
    int kcd, kcI, kcr, kcdz;        // ring stages of d, I (expert matrices), r and d (LoRE factors)
    int nsplit, cps, kcIs;          // shared down projection: K ranges, chunks per range, chunks in all
    int nA, nSp, n_spec, nBh, endB, nCs, nCh, endC;
    int n_hg, n_lg;
    int sh_early;                   // the shared down tiles are part of phase A (else they follow phase B)
};

__device__ __forceinline__ void plan_static(Plan &pl, const DtcParams &q, int kst = KSTAGE) {
    const Dims &dm = q.p.dm;
    pl.tIs = (dm.Is + 63) >> 6;
    pl.tI = (dm.I + 63) >> 6;
    pl.tz = (dm.r + 127) >> 7;
    pl.td = (dm.d + 127) >> 7;
    pl.kcd = (dm.d + kst - 1) / kst;           // stages of the expert matrices (kst = 256 for 8-bit weights)
    pl.kcI = (dm.I + kst - 1) / kst;
    pl.kcr = (dm.r + KSTAGE - 1) / KSTAGE;     // the LoRE factors are bf16 in either precision
    pl.kcdz = (dm.d + KSTAGE - 1) / KSTAGE;
    pl.kcIs = (dm.Is + kst - 1) / kst;
    pl.nsplit = q.nsplit_sh;
    pl.cps = q.cps_sh;
    pl.nCs = pl.td * pl.nsplit;
    // Before the routing is known only the shared expert can be worked on.  Its down tiles wait for ALL its
    // gate/up tiles, so they go first only when the CTAs that take them would have nothing else to do.
    pl.sh_early = (pl.tIs + pl.nCs <= (int)gridDim.x) ? 1 : 0;
    // Known at launch, in this order: the shared expert's gate/up tiles, its early down tiles, the gate/up tiles of the
    // slots that are groups regardless of the routing (the leading hit groups, in slot order).
    pl.n_spec = q.n_spec;
    pl.nSp = q.n_spec * pl.tI;
    pl.nA = pl.tIs + (pl.sh_early ? pl.nCs : 0) + pl.nSp;
    pl.n_hg = q.n_spec;
    pl.n_lg = pl.nBh = pl.nCh = 0;
    pl.endB = pl.endC = pl.nA;
}
__device__ __forceinline__ void plan_routed(Plan &pl, int n_hg, int n_lg) {
    pl.n_hg = n_hg;
    pl.n_lg = n_lg;
    pl.nBh = (n_hg - pl.n_spec) * pl.tI;   // (the first n_spec groups' tiles are part of nA)
    pl.endB = pl.nA + pl.nBh + n_lg * pl.tz;
    pl.nCh = n_hg * pl.td;
    pl.endC = pl.endB + (pl.sh_early ? 0 : pl.nCs) + pl.nCh + n_lg * pl.td;
}

// ------------------------------------------------------------------------------------------
// Auxiliary team
struct AuxCtx {
    int atid, lane, aw;
    int npf;   // timeline events recorded (tuning builds only)
};

// leader polls, result broadcast through shared memory: team-uniform
__device__ __forceinline__ bool aux_wait_ge(const DtcParams &q, Ctl *sh, const AuxCtx &a, const int *ctr, int target) {
    if (a.atid == 0)
        sh->aux_flag = wait_ge(ctr, target, q.p.sync, q.p.tb.status, q.p.spin_limit, &sh->abort_flag) ? 1 : 0;
    aux_sync();
    const bool ok = sh->aux_flag != 0;
    aux_sync();
    return ok;
}

// G router logits of one expert row: tokens t, t + step, ... (those past the batch are computed on the last token's row and
// dropped).  Per dot: slices k = lane*8 + 256 i reduced by slice_dot and added in increasing i, then the xor-shuffle tree.
template <int G>
__device__ __forceinline__ void logits_group(const DecodeParams &p, const __nv_bfloat16 *__restrict__ row, int t, int step, int e,
                                             int lane) {
    const Dims &dm = p.dm;
    const __nv_bfloat16 *x[G];
    float acc[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const int tg = min(t + g * step, dm.T - 1);
        x[g] = p.h + (size_t)tg * dm.d;
        acc[g] = 0.f;
    }
#pragma unroll 4
    for (int k = lane * 8; k < dm.d; k += 256) {
        const uint4 u = *reinterpret_cast<const uint4 *>(row + k);
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] += slice_dot(u, *reinterpret_cast<const uint4 *>(x[g] + k));
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float tot = warp_sum(acc[g]);
        if (lane == 0 && t + g * step < dm.T) p.logits[(size_t)(t + g * step) * dm.N + e] = tot;
    }
}

// router logits: unit u = (expert e, token subset s); each warp takes the tokens s*8 + warp (+ 8*r1_sub ...).
// Same arithmetic order as the stand-alone router (route_device.cuh): logits agree bit for bit.
__device__ __forceinline__ void aux_logits(const DtcParams &q, const AuxCtx &a) {
    const DecodeParams &p = q.p;
    const Dims &dm = p.dm;
    const int n_units = dm.N * q.r1_sub;
    int done = 0;
    // (units are dealt from the last CTA down: the first CTAs start with the shared expert's tiles, and a load issued
    // behind an SM's own weight stream waits for the bytes already queued)
    for (int u = gridDim.x - 1 - blockIdx.x; u < n_units; u += gridDim.x, ++done) {
        const int e = u % dm.N, s = u / dm.N;
        const __nv_bfloat16 *row = reinterpret_cast<const __nv_bfloat16 *>(p.w.w_router) + (size_t)e * dm.d;
        // the warp's tokens four (or two) at a time: the router row is loaded once for them and their loads are all in
        // flight together; each dot keeps the summation order of lane_dot_bf16
        const int step = AUX_W * q.r1_sub;
        int t = s * AUX_W + a.aw;
        for (; t + 2 * step < dm.T; t += 4 * step) logits_group<4>(p, row, t, step, e, a.lane);
        for (; t + step < dm.T; t += 2 * step) logits_group<2>(p, row, t, step, e, a.lane);
        for (; t < dm.T; t += step) logits_group<1>(p, row, t, step, e, a.lane);
    }
    if (done) {   // CTA-uniform
        aux_sync();
        if (a.atid == 0) red_release_add(p.sync + SY_R1_DONE, done);
    }
}

// three E5M2 terms whose sum is the bf16 value x (exactly for 2^-7 <= |x| <= 57344): bytes hi | mid << 8 | lo << 16
__device__ __forceinline__ uint32_t split_e5m2x3(float x) {
    uint32_t out = 0;
#pragma unroll
    for (int j = 0; j < 3; ++j) {
        const __nv_fp8_storage_t b = __nv_cvt_float_to_fp8(x, __NV_SATFINITE, __NV_E5M2);
        out |= (uint32_t)b << (8 * j);
        x -= __half2float(__half(__nv_cvt_fp8_to_halfraw(b, __NV_E5M2)));   // exact: both have few significant bits
    }
    return out;
}

// 8-bit weights: number of CTAs that write the three-term copy of h (= the target of SY_H8_DONE)
__device__ __forceinline__ int h8_ctas(const DtcParams &q) {
    const int n_units = q.p.dm.N * q.r1_sub, free_ctas = (int)gridDim.x - n_units;
    return free_ctas >= 8 ? free_ctas : (int)gridDim.x;
}
__device__ __forceinline__ void aux_split_h(const DtcParams &q, const AuxCtx &a, int n, int part, int parts) {
#pragma unroll 1
    for (int i = part * AUX_T + a.atid; i < n; i += parts * AUX_T) {
        const uint32_t b3 = split_e5m2x3(__bfloat162float(q.p.h[i]));
        q.x8_h[i] = (uint8_t)b3;
        q.x8_h[(size_t)n + i] = (uint8_t)(b3 >> 8);
        q.x8_h[2 * (size_t)n + i] = (uint8_t)(b3 >> 16);
    }
}

// Routing decisions from the logits, entirely in shared memory.  Every CTA computes the same tables
// (the code is deterministic: counts by atomics, positions by ranking); CTA 0 also writes the outputs.
// The arithmetic of the gates is that of warp_topk_gates (route_device.cuh).
// DIST: the batch is spread over the grid instead (CTA c takes tokens 8c .. 8c+7, a warp one token), the warp writes its
// token's entries to the context's exchange arrays and every CTA collects all of them afterwards (aux_route): per
// CTA the work no longer grows with the batch.  The token's confidences then travel with its logits (same indexing, one
// coalesced load) and the winner's value is handed to lane k by a shuffle, so classification waits for no load of its own.
template <int NPL, bool DIST>
__device__ __forceinline__ void aux_route_tokens(const DtcParams &q, Ctl *sh, const AuxSmem &ax, AuxCtx &a) {
    const DecodeParams &p = q.p;
    const Dims &dm = p.dm;
    const int T = dm.T, N = dm.N, K = dm.K, S = dm.S;
    // One warp per token (two tokens at a time, interleaved, so that the reductions of one hide the latency
    // of the other), no barrier inside: the logits go from L2 straight into registers (element e = lane + 32 m),
    // the K winners are found by K rounds of two warp reductions on order-preserving integer keys (largest key, then
    // smallest index among its holders: equal logits go to the smaller expert index), then gates and classes of
    // the token's K entries follow in lanes 0..K-1.  A group's members are kept as a bit mask over the tokens.
    // NPL = elements per lane (N <= 32 NPL).
    constexpr int TT = DIST ? 1 : 2;
    const int t_first = DIST ? (int)blockIdx.x * AUX_W + a.aw : a.aw, t_pass = DIST ? (int)gridDim.x * AUX_W : AUX_W * TT;
#pragma unroll 1
    for (int t0 = t_first; t0 < T; t0 += t_pass) {
        float val[TT][NPL], cf[TT][NPL];
        uint32_t key[TT][NPL];
#pragma unroll
        for (int u = 0; u < TT; ++u) {
            const int t = t0 + u * AUX_W;
#pragma unroll
            for (int m = 0; m < NPL; ++m) {
                const int e = a.lane + 32 * m;
                val[u][m] = (e < N && t < T) ? __ldcg(p.logits + (size_t)t * N + e) : 0.f;
                if (DIST) cf[u][m] = (e < N && t < T && !p.roll_depth) ? __ldg(p.conf + (p.conf_stride ? (size_t)t * N + e : (size_t)t)) : 0.f;
            }
        }
#pragma unroll
        for (int u = 0; u < TT; ++u)
#pragma unroll
            for (int m = 0; m < NPL; ++m) {
                const int e = a.lane + 32 * m;
                float v = val[u][m];
                v = (v == v) ? v + 0.0f : -INFINITY;   // NaN never wins; -0 and +0 are one value
                val[u][m] = v;
                const uint32_t bts = __float_as_uint(v);
                key[u][m] = e < N ? ((bts & 0x80000000u) ? ~bts : (bts | 0x80000000u)) : 0u;   // 0 is below every real key
            }
        int my_idx[TT];
        float my_val[TT], my_cf[TT];
#pragma unroll
        for (int u = 0; u < TT; ++u) {
            my_idx[u] = 0;
            my_val[u] = 0.f;
            my_cf[u] = 0.f;
        }
        if (key[0][0] != 1u) APROF(a, 75);
#pragma unroll 1
        for (int k = 0; k < K; ++k) {
            uint32_t bk[TT], wmax[TT];
            int bi[TT], widx[TT];
#pragma unroll
            for (int u = 0; u < TT; ++u) {
                bk[u] = 0u;
                bi[u] = 0x7fffffff;
#pragma unroll
                for (int m = 0; m < NPL; ++m)
                    if (key[u][m] > bk[u]) {
                        bk[u] = key[u][m];
                        bi[u] = a.lane + 32 * m;
                    }
            }
#pragma unroll
            for (int u = 0; u < TT; ++u) wmax[u] = __reduce_max_sync(0xffffffffu, bk[u]);
#pragma unroll
            for (int u = 0; u < TT; ++u)
                widx[u] = (int)__reduce_min_sync(0xffffffffu, (unsigned)(bk[u] == wmax[u] ? bi[u] : 0x7fffffff));
#pragma unroll
            for (int u = 0; u < TT; ++u) {
                float wc = 0.f;   // DIST: the winner's confidence, from the lane that holds it
#pragma unroll
                for (int m = 0; m < NPL; ++m) {
                    if (a.lane + 32 * m == widx[u]) key[u][m] = 0u;   // taken
                    if (DIST && (widx[u] >> 5) == m) wc = cf[u][m];
                }
                if (DIST) wc = __shfl_sync(0xffffffffu, wc, widx[u] & 31);
                if (a.lane == k) {
                    my_idx[u] = widx[u];
                    my_val[u] = __uint_as_float((wmax[u] & 0x80000000u) ? (wmax[u] ^ 0x80000000u) : ~wmax[u]);
                    if (DIST) my_cf[u] = wc;
                }
            }
        }
        APROF(a, 76);
#pragma unroll
        for (int u = 0; u < TT; ++u) {
            const int t = t0 + u * AUX_W;
            if (t >= T) continue;   // warp-uniform
            // gates: p_k = exp(l_k - l_0); denominator = sum over the winners in k order, or the full softmax sum
            const float mx = __shfl_sync(0xffffffffu, my_val[u], 0);
            float denom = 0.f;
            if (!p.norm_topk) {
                float sacc = 0.f;
#pragma unroll
                for (int m = 0; m < NPL; ++m)
                    if (a.lane + 32 * m < N) sacc += expf(val[u][m] - mx);
                denom = warp_sum(sacc);
            }
            const float pk = (a.lane < K) ? expf(my_val[u] - mx) : 0.f;
            if (p.norm_topk) {
                float sacc = 0.f;
#pragma unroll 1
                for (int k = 0; k < K; ++k) sacc += __shfl_sync(0xffffffffu, pk, k);
                denom = sacc;
            }
            // rollout mode (Algorithm 1): C = sum of the gates in k order; halting rule; outputs of this depth by CTA 0
            bool roll_cont = false;
            if (p.roll_depth) {
                const float g = pk / denom;
                float cs = 0.f;
#pragma unroll 1
                for (int k = 0; k < K; ++k) cs += __shfl_sync(0xffffffffu, g, k);
                const bool on = p.roll_depth == 1 ? true : p.roll_active_in[t] != 0;
                const bool stop = p.roll_depth >= p.roll_l_min && cs < p.roll_tau;
                roll_cont = on && !stop;
                if (blockIdx.x == 0) {
                    if (a.lane < K) p.roll_idx_out[t * K + a.lane] = on ? my_idx[u] : -1;
                    if (a.lane == 0) {
                        p.roll_conf_out[t] = on ? cs : 0.f;
                        p.roll_active_out[t] = roll_cont ? 1 : 0;
                        if (on) p.roll_depth_out[t] = p.roll_depth;
                        else if (p.roll_depth == 1) p.roll_depth_out[t] = 0;
                    }
                }
            }
            // classification (Sec. 4.2 policy)
            if (a.lane < K) {
                const int i = t * K + a.lane, e = my_idx[u];
                const int sl = p.roll_depth ? -1 : ax.soe[e];
                int c;
                if (sl >= S) {
                    atomicMax(p.tb.status, (int)SPICE_ERR_BAD_TABLE);
                    c = SPICE_MISS_EXACT;
                } else if (sl >= 0) {
                    c = SPICE_HIT;
                    if (!DIST) atomicOr(&ax.mask_hit[2 * sl + (t >> 5)], 1u << (t & 31));
                } else {
                    bool low;
                    if (p.roll_depth) {
                        low = roll_cont;
                    } else {
                        const int ci = p.conf_stride ? t * N + e : t;
                        const float cfv = DIST ? my_cf[u] : (conf_staged(dm, p.conf_stride) ? ax.conf[ci] : __ldg(p.conf + ci));
                        low = cfv < p.tau;
                    }
                    c = low ? SPICE_LOWCONF : SPICE_MISS_EXACT;
                    if (low && !DIST) atomicOr(&ax.mask_low[2 * e + (t >> 5)], 1u << (t & 31));
                }
                if (DIST) {
                    p.x_idx[i] = e;
                    p.x_gate[i] = pk / denom;
                    p.x_cls[i] = (unsigned char)c;
                } else {
                    ax.idx[i] = e;
                    ax.gate[i] = pk / denom;
                    ax.cls[i] = (unsigned char)c;
                }
            }
        }
    }
}

// the routing of a batch is spread over the grid once a CTA would need more than two passes of its 8 warps (the extra
// grid-wide hop costs about as much as one pass)
__device__ __forceinline__ bool route_dist(const DecodeParams &p) { return p.dm.T > 4 * AUX_W && !p.roll_depth; }

__device__ __forceinline__ bool aux_route(const DtcParams &q, Ctl *sh, const AuxSmem &ax, AuxCtx &a) {
    const DecodeParams &p = q.p;
    const Dims &dm = p.dm;
    const int T = dm.T, N = dm.N, K = dm.K, S = dm.S, n = T * K;
    if (route_dist(p)) {
        if (N <= 64) aux_route_tokens<2, true>(q, sh, ax, a);
        else if (N <= 128) aux_route_tokens<4, true>(q, sh, ax, a);
        else aux_route_tokens<8, true>(q, sh, ax, a);
        aux_sync();
        if (a.atid == 0) {
            int mine = 0;
            for (int t = (int)blockIdx.x * AUX_W; t < T; t += (int)gridDim.x * AUX_W) mine += min(AUX_W, T - t);
            if (mine) red_release_add(p.sync + SY_ROUTE_DONE, mine);
        }
        if (!aux_wait_ge(q, sh, a, p.sync + SY_ROUTE_DONE, T)) return false;
        // every CTA collects all entries and rebuilds the groups' member masks
#pragma unroll 1
        for (int i = a.atid; i < n; i += AUX_T) {
            const int e = __ldcg(p.x_idx + i), t = i / K;
            const int c = __ldcg(p.x_cls + i);
            ax.idx[i] = e;
            ax.gate[i] = __ldcg(p.x_gate + i);
            ax.cls[i] = (unsigned char)c;
            if (c == SPICE_HIT) atomicOr(&ax.mask_hit[2 * ax.soe[e] + (t >> 5)], 1u << (t & 31));
            else if (c == SPICE_LOWCONF) atomicOr(&ax.mask_low[2 * e + (t >> 5)], 1u << (t & 31));
        }
    } else {
        if (N <= 64) aux_route_tokens<2, false>(q, sh, ax, a);
        else if (N <= 128) aux_route_tokens<4, false>(q, sh, ax, a);
        else aux_route_tokens<8, false>(q, sh, ax, a);
    }
    aux_sync();
    APROF(a, 73);
    // groups: thread i owns slot i and expert i; packed scan of (entries, non-empty flag << 16)
    {
        const int ch = a.atid < S ? __popc(ax.mask_hit[2 * a.atid]) + __popc(ax.mask_hit[2 * a.atid + 1]) : 0;
        const int cl = a.atid < N ? __popc(ax.mask_low[2 * a.atid]) + __popc(ax.mask_low[2 * a.atid + 1]) : 0;
        const bool fh = ch > 0 || a.atid < q.n_spec;   // a group (possibly without members)
        const int va = ch | (fh << 16), vb = cl | ((cl > 0) << 16);
        int ia = va, ib = vb;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int na = __shfl_up_sync(0xffffffffu, ia, o), nbv = __shfl_up_sync(0xffffffffu, ib, o);
            if (a.lane >= o) {
                ia += na;
                ib += nbv;
            }
        }
        if (a.lane == 31) {
            sh->wsum[0][a.aw] = ia;
            sh->wsum[1][a.aw] = ib;
        }
        aux_sync();
        int ba = 0, bb = 0, ta = 0;
#pragma unroll
        for (int w = 0; w < AUX_W; ++w) {
            const int sa = sh->wsum[0][w], sb = sh->wsum[1][w];
            if (w < a.aw) {
                ba += sa;
                bb += sb;
            }
            ta += sa;
        }
        const int ea = ba + ia - va, eb = bb + ib - vb;   // exclusive
        const int n_hg = ta >> 16;
        if (a.atid < S) ax.off_hit[a.atid] = ea & 0xffff;
        if (a.atid < N) ax.off_low[a.atid] = eb & 0xffff;
        if (fh) ax.gtab[1 + (ea >> 16)] = GroupDesc{KIND_HIT, a.atid, ea & 0xffff, ch};
        if (cl > 0) ax.gtab[1 + n_hg + (eb >> 16)] = GroupDesc{KIND_LOW, a.atid, eb & 0xffff, cl};
        if (a.atid == AUX_T - 1) {   // this thread's inclusive sums are the totals
            sh->n_hg = n_hg;
            sh->n_lg = (bb + ib) >> 16;
            ax.gtab[0] = GroupDesc{KIND_SHARED, 0, 0, T};
        }
    }
    // coefficient of the shared expert's output: 1 + sum of LOWCONF gates, in k order (rollout: the sum alone)
#pragma unroll 1
    for (int t = a.atid; t < T; t += AUX_T) {
        float c = p.roll_depth ? 0.0f : 1.0f;
#pragma unroll 1
        for (int k = 0; k < K; ++k)
            if (ax.cls[t * K + k] == SPICE_LOWCONF) c += ax.gate[t * K + k];
        ax.coef[t] = c;
    }
    aux_sync();
    APROF(a, 74);
    // position of every entry inside its group = offset of the group + number of members with a smaller token index
    // (an expert occurs at most once among a token's K choices, so the members of a group are distinct tokens)
#pragma unroll 1
    for (int i = a.atid; i < n; i += AUX_T) {
        // grouping key of the entry: its slot (HIT), 1024 + its expert (LOWCONF), -1 (listed for exact recovery)
        const int e_i = ax.idx[i], c_i = ax.cls[i];
        const int key = c_i == SPICE_HIT ? ax.soe[e_i] : (c_i == SPICE_LOWCONF ? 1024 + e_i : -1), t = i / K;
        int pos = -1;
        if (key >= 0) {
            const uint32_t *mk = key < 1024 ? ax.mask_hit + 2 * key : ax.mask_low + 2 * (key - 1024);
            const uint32_t below = (1u << (t & 31)) - 1u;
            const int rank = t < 32 ? __popc(mk[0] & below) : __popc(mk[0]) + __popc(mk[1] & below);
            if (key < 1024) {
                pos = ax.off_hit[key] + rank;
                ax.perm_h[pos] = i;
            } else {
                pos = ax.off_low[key - 1024] + rank;
                ax.perm_l[pos] = i;
            }
        }
        ax.pos[i] = pos;
    }
    aux_sync();
    return true;
}

// CTA 0: routing results for the caller (top-k, gates, classes, counts, residual-miss list in (t,k) order)
__device__ __forceinline__ void aux_write_outputs(const DtcParams &q, Ctl *sh, const AuxSmem &ax, const AuxCtx &a) {
    const DecodeParams &p = q.p;
    const int K = p.dm.K, n = p.dm.T * K;
    // (a spread routing was exchanged through the context's arrays: an output that IS such an array is written already,
    // and other CTAs may still be reading it)
    const bool dist = route_dist(p);
    const bool w_idx = !dist || p.idx != p.x_idx, w_gate = !dist || p.gate != p.x_gate, w_cls = !dist || p.cls != p.x_cls;
#pragma unroll 1
    for (int i = a.atid; i < n; i += AUX_T) {
        if (w_idx) p.idx[i] = ax.idx[i];
        if (w_gate) p.gate[i] = ax.gate[i];
        if (w_cls) p.cls[i] = ax.cls[i];
    }
    if (a.aw == 0) {
        int base = 0, n_hit = 0, n_low = 0;
#pragma unroll 1
        for (int i0 = 0; i0 < n; i0 += 32) {
            const int i = i0 + a.lane;
            const bool miss = i < n && ax.cls[i] == SPICE_MISS_EXACT;
            const unsigned m = __ballot_sync(0xffffffffu, miss);
            n_hit += __popc(__ballot_sync(0xffffffffu, i < n && ax.cls[i] == SPICE_HIT));
            n_low += __popc(__ballot_sync(0xffffffffu, i < n && ax.cls[i] == SPICE_LOWCONF));
            if (miss && p.resid_tok) {
                const int o = base + __popc(m & ((1u << a.lane) - 1u));
                p.resid_tok[o] = i / K;
                p.resid_k[o] = i % K;
                p.resid_expert[o] = ax.idx[i];
                p.resid_gate[o] = ax.gate[i];
            }
            base += __popc(m);
        }
        if (a.lane < 3) p.counts[a.lane] = a.lane == SPICE_HIT ? n_hit : (a.lane == SPICE_MISS_EXACT ? base : n_low);
    }
}

// combine: 256 columns of one token per 64-thread unit; the reads of up to 8 entries are in flight together
__device__ __forceinline__ void aux_combine(const DtcParams &q, const AuxSmem &ax, int t, int j) {
    const DecodeParams &p = q.p;
    const Dims &dm = p.dm;
    if (j >= dm.d) return;
    const int d = dm.d, K = dm.K;
    float4 sh4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int s0 = 0; s0 < q.nsplit_sh; s0 += 4) {
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (s0 + u < q.nsplit_sh)
                v[u] = __ldcg(reinterpret_cast<const float4 *>(q.part_split + ((size_t)(s0 + u) * dm.T + t) * d + j));
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (s0 + u < q.nsplit_sh) {
                sh4.x += v[u].x; sh4.y += v[u].y; sh4.z += v[u].z; sh4.w += v[u].w;
            }
    }
    const float c = ax.coef[t];
    float4 acc = make_float4(c * sh4.x, c * sh4.y, c * sh4.z, c * sh4.w);
#pragma unroll 1
    for (int k0 = 0; k0 < K; k0 += 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = t * K + k0 + u;
            if (k0 + u < K && ax.pos[i] >= 0) v[u] = __ldcg(reinterpret_cast<const float4 *>(p.tb.part + (size_t)i * d + j));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int i = t * K + k0 + u;
            if (k0 + u < K && ax.pos[i] >= 0) {
                const float g = ax.gate[i];
                acc.x = fmaf(g, v[u].x, acc.x); acc.y = fmaf(g, v[u].y, acc.y);
                acc.z = fmaf(g, v[u].z, acc.z); acc.w = fmaf(g, v[u].w, acc.w);
            }
        }
    }
    if (p.y_cpu) {
        const float4 s = *reinterpret_cast<const float4 *>(p.y_cpu + (size_t)t * d + j);
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

// ------------------------------------------------------------------------------------------
template <int NB, bool F8 = false>
__global__ void __launch_bounds__(DTC_THREADS, 1) decode_tc_kernel(const __grid_constant__ DtcParams q,
                                                                   const __grid_constant__ DtcMaps maps) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    constexpr int STAGE_BYTES = A_BYTES + (F8 ? 6 : 2) * NB * 128;   // (stage pitch; a bf16 task of the 8-bit kernel fills less)
    constexpr int ACC = F8 ? 4 * NB : NB;                              // TMEM columns between the two accumulator buffers (8-bit: 3 NB used)
    constexpr int TMEM_COLS = 2 * ACC <= 32 ? 32 : (2 * ACC <= 64 ? 64 : (2 * ACC <= 128 ? 128 : (2 * ACC <= 256 ? 256 : 512)));
    constexpr int KST = F8 ? KSTAGE8 : KSTAGE;
    const DecodeParams &p = q.p;
    const Dims &dm = p.dm;
    unsigned char *ring = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Ctl *sh = reinterpret_cast<Ctl *>(ring + (size_t)q.stages * STAGE_BYTES);
    AuxSmem ax;
    aux_layout(dm, p.conf_stride, NB, &ax, reinterpret_cast<unsigned char *>(sh) + ((sizeof(Ctl) + 15) & ~size_t(15)));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = &sh->abort_flag;
    const int stages = q.stages;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1);
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sh->tmem_full[b]), 1);
            mbar_init(smem_u32(&sh->tmem_empty[b]), 4);
            mbar_init(smem_u32(&sh->xch_full[b]), 2);
            mbar_init(smem_u32(&sh->xch_empty[b]), 2);
        }
        for (int s = 0; s < TQ; ++s) {
            mbar_init(smem_u32(&sh->tq_full[s]), 1);
            mbar_init(smem_u32(&sh->tq_empty[s]), 5);
        }
        mbar_init(smem_u32(&sh->plan_ready), 1);
        mbar_init(smem_u32(&sh->logits_done), 1);
        mbar_init(smem_u32(&sh->mma_drain), 1);
        sh->abort_flag = 0;
        sh->aux_flag = 0;
        sh->last_flag = 0;
        sh->no_more = 0;
        sh->n_hg = sh->n_lg = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = threadIdx.x; i < 1 + dm.S + dm.N; i += DTC_THREADS) ax.ready[i] = 0;
    {   // the router matrix is needed first and by few warps: every thread of the grid asks for one of its lines now
        const size_t n_lines = ((size_t)dm.N * dm.d * 2 + 127) >> 7;
        const size_t g = (size_t)blockIdx.x * DTC_THREADS + threadIdx.x, n_thr = (size_t)gridDim.x * DTC_THREADS;
        for (size_t l = g; l < n_lines; l += n_thr)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.w.w_router) + (l << 7)));
        // so are the confidences where classification reads them from global memory
        const size_t c_lines = (!p.roll_depth && (route_dist(p) || !conf_staged(dm, p.conf_stride)))
                                   ? ((p.conf_stride ? (size_t)dm.T * dm.N : (size_t)dm.T) * 4 + 127) >> 7 : 0;
        for (size_t l = n_thr - 1 - g; l < c_lines; l += n_thr)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char *>(p.conf) + (l << 7)));
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh->tmem_base)), "r"(TMEM_COLS));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;
#ifdef SPICE_PROF
    if (threadIdx.x == 0 && blockIdx.x < PR_CTAS) {
        g_dtc_cal[blockIdx.x * 4 + 0] = now_ns();
        g_dtc_cal[blockIdx.x * 4 + 1] = (unsigned long long)clock64();
    }
#endif

    if (warp == 0) {
        // ---------------- TMA producer: lane 0 drives, lanes 0-3 each issue one of a stage's copies.  A stage holds
        // two 64-element sub-chunks.  The SM accepts a TMA instruction only every 150 cycles or so, whatever its size
        // and whichever thread issues it, so the copies are made as large as the tensor maps allow: for the big
        // matrices ONE box covers both sub-chunks (and both the gate and the up rows) of a stage -- the maps view a
        // row as [k-block][64] with the k-block as an outer dimension, so the box lands as [k-block][row][64] -- and
        // one more box brings the token rows.  Operands whose reduction length is the LoRE rank use plain maps, one
        // box per sub-chunk (lanes 2 and 3).
        constexpr unsigned PM = 0xFu;
        if (lane < 4) {
            Plan pl;
            plan_static(pl, q, KST);
            bool routed = false;
            int npf = 0;
            if (lane == 0) DPROF(0, npf, 1);
            uint32_t it = 0, tcount = 0;
            int s = 0;
            uint32_t ring_phase = 0;   // parity of the current pass over the ring
            int end = pl.nA;   // (what is known at launch: the shared expert's tiles and the gate/up tiles of the first n_spec slots)
            bool ok = true;
            // ids: the first one is the CTA's index, every later one is drawn from a global counter.  The draw is
            // issued before the task's copies and used after them, so its latency hides behind the copies.
            int id = blockIdx.x;
            bool logits_seen = false;   // this CTA's router-logit units are done (only asked before the routing is known)
            bool h8_ok = false;   // (8-bit weights) the three-term copy of h is complete
            const uint64_t w_policy = l2_policy_evict_first();
            auto lead_wait = [&](uint32_t bar, uint32_t parity) {   // lane 0 waits, the outcome is uniform
                int r = 1;
                if (lane == 0) r = mb_wait(bar, parity, abort_flag) ? 1 : 0;
                return __shfl_sync(PM, r, 0) != 0;
            };
            while (ok) {
                if (id >= end) {
                    if (routed) break;
                    if (lane == 0) DPROF(0, npf, 30);
                    if (!lead_wait(smem_u32(&sh->plan_ready), 0)) { ok = false; break; }
                    if (lane == 0) DPROF(0, npf, 31);
                    routed = true;
                    plan_routed(pl, sh->n_hg, sh->n_lg);
                    end = pl.endC;
                    if (id >= end) break;
                }
                // resolve the task: operands, k range, dependency
                TaskDesc t{};
                const CUtensorMap *ma, *mb;
                int a_row0, a_z = 0, b_z = 0, k0 = 0, dep = -1, dep_target = 0;
                bool plain = false;   // operands with reduction length r: plain maps, one box per sub-chunk
                const int c0 = pl.endB + (pl.sh_early ? 0 : pl.nCs);   // first down tile of a slot
                const int sp0 = pl.tIs + (pl.sh_early ? pl.nCs : 0);   // first gate/up tile of the slots that are groups regardless
                const bool sh_down = pl.sh_early ? (id >= pl.tIs && id < sp0) : (id >= pl.endB && id < c0);
                if (id < pl.tIs) {                       // gate/up tile of the shared expert
                    t.kind = TASK_ACT;
                    t.tile = id;
                    t.nk = pl.kcd;
                    t.f8 = F8;
                    ma = &maps.m[MAP_SH_GU];
                    mb = &maps.m[F8 ? MAP_X8 : MAP_H];
                    a_row0 = t.tile * 64;
                } else if (sh_down) {                    // down tile of the shared expert, one K range
                    const int l = id - (pl.sh_early ? pl.tIs : pl.endB);
                    t.kind = TASK_DOWN;
                    t.tile = l % pl.td;
                    t.split = l / pl.td;
                    k0 = t.split * pl.cps;
                    t.nk = min(pl.cps, pl.kcIs - k0);
                    t.f8 = F8;
                    ma = &maps.m[MAP_SH_D];
                    mb = &maps.m[MAP_ACT_SH];
                    a_row0 = t.tile * 128;
                    dep = SY_GROUP0;
                    dep_target = 2 * pl.tIs;
                } else if (id < pl.nA + pl.nBh) {        // gate/up tile of a resident slot (the others of the launch-time range are taken above)
                    const int l = id < pl.nA ? id - sp0 : pl.nSp + id - pl.nA;
                    t.kind = TASK_ACT;
                    t.gi = 1 + l / pl.tI;
                    t.tile = l % pl.tI;
                    t.nk = pl.kcd;
                    t.f8 = F8;
                    ma = &maps.m[MAP_SLOT_GU];
                    mb = &maps.m[F8 ? MAP_X8 : MAP_H];
                    a_row0 = t.tile * 64;
                    a_z = t.gi <= q.n_spec ? t.gi - 1 : ax.gtab[t.gi].id;   // (the group table may not exist yet)
                } else if (id < pl.endB) {               // A_e tile of a low-confidence expert
                    const int l = id - pl.nA - pl.nBh;
                    t.kind = TASK_Z;
                    t.gi = 1 + pl.n_hg + l / pl.tz;
                    t.tile = l % pl.tz;
                    t.nk = pl.kcdz;
                    ma = &maps.m[MAP_LORE_A];
                    mb = &maps.m[MAP_H];
                    a_row0 = t.tile * 128;
                    a_z = ax.gtab[t.gi].id;
                } else if (id < c0 + pl.nCh) {           // down tile of a resident slot
                    const int l = id - c0;
                    t.kind = TASK_DOWN;
                    t.gi = 1 + l / pl.td;
                    t.tile = l % pl.td;
                    t.nk = pl.kcI;
                    t.f8 = F8;
                    ma = &maps.m[MAP_SLOT_D];
                    mb = &maps.m[MAP_ACT_HIT];
                    a_row0 = t.tile * 128;
                    a_z = ax.gtab[t.gi].id;
                    b_z = t.gi - 1;
                    dep = SY_GROUP0 + t.gi;
                    dep_target = 2 * pl.tI;
                    if (ax.gtab[t.gi].m == 0) {   // a slot that is a group without a token: nothing to multiply, the roles only count the tile
                        t.nk = 0;
                        dep = -1;
                    }
                } else {                                 // B_e tile of a low-confidence expert
                    const int l = id - c0 - pl.nCh;
                    t.kind = TASK_DOWN;
                    t.gi = 1 + pl.n_hg + l / pl.td;
                    t.tile = l % pl.td;
                    t.nk = pl.kcr;
                    ma = &maps.m[MAP_LORE_B];
                    mb = &maps.m[MAP_Z];
                    plain = true;
                    a_row0 = t.tile * 128;
                    a_z = ax.gtab[t.gi].id;
                    b_z = t.gi - 1 - pl.n_hg;
                    dep = SY_GROUP0 + t.gi;
                    dep_target = 4 * pl.tz;
                }
                // A gate/up tile streamed ahead of the routing must not delay the routing itself: the loads of the CTA's
                // router-logit units would queue behind the tile's copies, so the tile waits for them.
                if (!routed && t.kind == TASK_ACT && t.gi > 0 && (int)gridDim.x - 1 - (int)blockIdx.x < p.dm.N * q.r1_sub && !logits_seen) {
                    if (!lead_wait(smem_u32(&sh->logits_done), 0)) { ok = false; break; }
                    logits_seen = true;
                }
                if (lane == 0) DPROF(0, npf, 10 + t.kind);
                // this lane's copy of every stage: lane 0 the weights, lane 1 the tokens (sub-chunk 0 only when the
                // maps are plain); lanes 2, 3 the same for sub-chunk 1 of plain maps
                const int sub = lane >> 1, is_b = lane & 1;
                const CUtensorMap *my_map = is_b ? mb : ma;
                const uint32_t my_off = is_b ? (uint32_t)(A_BYTES + sub * NB * 128) : (uint32_t)(sub * SUB_A);
                const int my_y = is_b ? 0 : a_row0;
                const int my_z = is_b ? b_z : a_z;
                const bool my_on = sub == 0 || plain;
                // bytes a stage of this task receives (a bf16 task of the 8-bit kernel leaves part of the token area unused)
                const uint32_t tx_bytes = (F8 && !t.f8) ? (uint32_t)(A_BYTES + 2 * NB * 128) : (uint32_t)STAGE_BYTES;
                auto copy = [&](int kb, int stage) {   // this lane's box of k-stage kb into ring stage `stage`
                    const uint32_t full = smem_u32(&sh->full[stage]);
                    const uint32_t dst = smem_u32(ring + (size_t)stage * STAGE_BYTES);
                    // (weights are read once per call: evict-first, so that they do not displace the kernel's code, the
                    // router matrix and the activations from L2; the token operands keep the default policy)
                    if (plain) {
                        if (is_b) tma_load_5d(dst + my_off, my_map, (k0 + kb) * KSTAGE + sub * 64, my_y, 0, 0, my_z, full);
                        else tma_load_5d_hint(dst + my_off, my_map, (k0 + kb) * KSTAGE + sub * 64, my_y, 0, 0, my_z, full, w_policy);
                    } else {
                        if (is_b) tma_load_5d(dst + my_off, my_map, 0, my_y, 0, (k0 + kb) * 2, my_z, full);
                        else tma_load_5d_hint(dst + my_off, my_map, 0, my_y, 0, (k0 + kb) * 2, my_z, full, w_policy);
                    }
                };
                // 8-bit weights: the first gate/up task of the CTA waits for the three-term copy of h, which the auxiliary
                // teams of all CTAs write at the start of the kernel (its weights are copied meanwhile, like a down tile's)
                bool pending = false;
                if (F8 && t.kind == TASK_ACT && !h8_ok) {
                    dep = SY_H8_DONE;
                    dep_target = h8_ctas(q);
                    pending = true;
                } else
                // has the watcher warp already seen the group complete?
                if (dep >= 0) {
                    int seen = 0;
                    if (lane == 0) {
                        seen = ld_acquire_cta(ax.ready + t.gi);
                        DPROF(0, npf, 24 + (seen ? 1 : 0));
                    }
                    pending = __shfl_sync(PM, seen, 0) == 0;
                }
                {   // hand the task to the MMA and epilogue roles
                    const int slot = tcount % TQ;
                    if (!lead_wait(smem_u32(&sh->tq_empty[slot]), ((tcount / TQ) & 1) ^ 1)) { ok = false; break; }
                    if (lane == 0) {
                        sh->tq[slot] = t;
                        mbar_arrive(smem_u32(&sh->tq_full[slot]));
                    }
                    ++tcount;
                }
                if (lane == 0) DPROF(0, npf, 21);
                int kb0 = 0;
                if (pending) {
                    // The activations are not there yet, but the weights do not depend on them: arm the first stages
                    // and start their weight copies, wait, then add the token copies to the same stages.
                    const int pre = min(t.nk, stages);
                    const int s0 = s;
                    for (int kb = 0; kb < pre && ok; ++kb, ++it) {
                        if (!lead_wait(smem_u32(&sh->empty[s]), ring_phase ^ 1)) { ok = false; break; }
                        if (lane == 0) mbar_expect_tx(smem_u32(&sh->full[s]), tx_bytes);
                        __syncwarp(PM);
                        if (my_on && !is_b) copy(kb, s);
                        if (++s == stages) {
                            s = 0;
                            ring_phase ^= 1;
                        }
                    }
                    if (!ok) break;
                    int r = 1;
                    if (lane == 0) r = wait_ge(p.sync + dep, dep_target, p.sync, p.tb.status, p.spin_limit, abort_flag) ? 1 : 0;
                    __syncwarp(PM);
                    if (__shfl_sync(PM, r, 0) == 0) { ok = false; break; }
                    if (lane == 0) DPROF(0, npf, 22);
                    if (F8 && dep == SY_H8_DONE) h8_ok = true;
                    fence_proxy_async();
                    for (int kb = 0, ss = s0; kb < pre; ++kb) {
                        if (my_on && is_b) copy(kb, ss);
                        if (++ss == stages) ss = 0;
                    }
                    kb0 = pre;
                } else if (dep >= 0) {
                    fence_proxy_async();
                }
                // (drawn only now: an acquire or a fence issued while the atomic is in flight would wait for it)
                int drawn = 0;
                if (lane == 0) drawn = (int)gridDim.x + atomicAdd(p.sync + SY_NEXT_TASK, 1);
                for (int kb = kb0; kb < t.nk; ++kb, ++it) {
                    if (!lead_wait(smem_u32(&sh->empty[s]), ring_phase ^ 1)) { ok = false; break; }
                    if (lane == 0) mbar_expect_tx(smem_u32(&sh->full[s]), tx_bytes);
                    __syncwarp(PM);
                    if (my_on) copy(kb, s);
#ifdef SPICE_PROF_STAGES
                    if (lane == 0 && it < 64) DPROF(0, npf, 90);
#endif
                    if (++s == stages) {
                        s = 0;
                        ring_phase ^= 1;
                    }
                }
                id = __shfl_sync(PM, drawn, 0);
                // nothing will follow this task: let the epilogue publish its down tiles as it finishes them
                if (routed && id >= end && lane == 0) st_release_cta(&sh->no_more, 1);
            }
            if (lane == 0) DPROF(0, npf, 40);
            if (ok && lane == 0) {   // tell the other roles that the list is exhausted
                const int slot = tcount % TQ;
                if (mb_wait(smem_u32(&sh->tq_empty[slot]), ((tcount / TQ) & 1) ^ 1, abort_flag)) {
                    sh->tq[slot].kind = TASK_EXIT;
                    mbar_arrive(smem_u32(&sh->tq_full[slot]));
                }
            }
            // drain: every stage that was armed must have landed before the CTA may end
            if (lane == 0) {
                const uint32_t n_back = it < (uint32_t)stages ? it : (uint32_t)stages;
                int ds = s;
                uint32_t dph = ring_phase;
                for (uint32_t j = 0; j < n_back; ++j) {
                    if (--ds < 0) {
                        ds = stages - 1;
                        dph ^= 1;
                    }
                    mb_drain(smem_u32(&sh->full[ds]), dph);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (one lane)
        if (lane == 0) {
            constexpr uint32_t IDESC = make_idesc(128, NB);
            constexpr uint32_t IDESC8 = make_idesc_e4m3_e5m2(128, 3 * NB);
#ifdef SPICE_PROF_STAGES
            int npf_m = 0;
#endif
            int s = 0;
            uint32_t ring_phase = 0;
            for (uint32_t tcount = 0;; ++tcount) {
                const int slot = tcount % TQ;
                if (!mb_wait(smem_u32(&sh->tq_full[slot]), (tcount / TQ) & 1, abort_flag)) break;
                const int kind = sh->tq[slot].kind, nk = sh->tq[slot].nk;
                const bool f8 = F8 && sh->tq[slot].f8 != 0;
                if (kind == TASK_EXIT) break;
                const int buf = tcount & 1;
                if (!mb_wait(smem_u32(&sh->tmem_empty[buf]), ((tcount >> 1) & 1) ^ 1, abort_flag)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * ACC;
                bool ok = true;
                for (int kb = 0; kb < nk; ++kb) {
                    if (!mb_wait(smem_u32(&sh->full[s]), ring_phase, abort_flag)) { ok = false; break; }
#ifdef SPICE_PROF_STAGES
                    if (npf_m < 48) DPROF(3, npf_m, 91);
#endif
                    tc_fence_after();
                    const uint32_t a0 = smem_u32(ring + (size_t)s * STAGE_BYTES), b0 = a0 + A_BYTES;
                    if (f8) {   // 32 one-byte elements per instruction: the same 32-byte steps through a 128-byte row
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            const uint64_t da = make_desc(a0 + c * SUB_A), db = make_desc(b0 + c * 3 * NB * 128);
#pragma unroll
                            for (int k = 0; k < 4; ++k) tc_mma_f8(d_tmem, da + 2 * k, db + 2 * k, IDESC8, (kb | c | k) ? 1u : 0u);
                        }
                    } else {
#pragma unroll
                        for (int c = 0; c < 2; ++c) {
                            const uint64_t da = make_desc(a0 + c * SUB_A), db = make_desc(b0 + c * NB * 128);
#pragma unroll
                            for (int k = 0; k < 4; ++k) tc_mma(d_tmem, da + 2 * k, db + 2 * k, IDESC, (kb | c | k) ? 1u : 0u);
                        }
                    }
                    tc_commit(smem_u32(&sh->empty[s]));
                    if (++s == stages) {
                        s = 0;
                        ring_phase ^= 1;
                    }
                }
                if (!ok) break;
                tc_commit(smem_u32(&sh->tmem_full[buf]));
                mbar_arrive(smem_u32(&sh->tq_empty[slot]));
            }
            // every MMA issued by this thread must have completed before the TMEM columns are given back
            tc_commit(smem_u32(&sh->mma_drain));
            mb_drain(smem_u32(&sh->mma_drain), 0);
        }
    } else if (warp < 6) {
        // ---------------- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 = weight rows of the tile
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        uint32_t xc = 0;   // gate/up tiles seen (exchange buffer use count)
        int n_down = 0;    // down tiles finished by this warp, published once: only the combine waits for them
        const int T = dm.T;
        int npf = 0;
        for (uint32_t tcount = 0;; ++tcount) {
            const int slot = tcount % TQ;
            if (!warp_mb_wait(smem_u32(&sh->tq_full[slot]), (tcount / TQ) & 1, abort_flag, lane)) break;
            const TaskDesc t = sh->tq[slot];
            if (t.kind == TASK_EXIT) break;
            const int buf = tcount & 1;
            if (warp == 2 && lane == 0) DPROF(1, npf, 50 + t.kind);
            if (!warp_mb_wait(smem_u32(&sh->tmem_full[buf]), (tcount >> 1) & 1, abort_flag, lane)) break;
            if (warp == 2 && lane == 0) DPROF(1, npf, 54);
            tc_fence_after();
            uint32_t v[NB];
            const uint32_t t0 = tmem_base + buf * ACC + ((uint32_t)(qd * 32) << 16);
            if (F8 && t.f8) {   // (warp-uniform) three accumulators per token: hi, mid and lo term of the activations
#pragma unroll
                for (int c = 0; c < NB; c += 16) {
                    uint32_t m1[16], m2[16];
                    tc_ld16(t0 + c, &v[c]);
                    tc_ld16(t0 + NB + c, m1);
                    tc_ld16(t0 + 2 * NB + c, m2);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        v[c + j] = __float_as_uint((__uint_as_float(v[c + j]) + __uint_as_float(m1[j])) + __uint_as_float(m2[j]));
                }
            } else {
#pragma unroll
                for (int c = 0; c < NB; c += 16) tc_ld16(t0 + c, &v[c]);
            }
            tc_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty[buf]));   // accumulator is in registers now
            if (warp == 2 && lane == 0) DPROF(1, npf, 56);
            // (a gate/up tile of one of the first n_spec slots may be finished before the group table exists)
            const GroupDesc grp = t.gi == 0 ? GroupDesc{KIND_SHARED, 0, 0, T}
                                            : (t.kind == TASK_ACT && t.gi <= q.n_spec ? GroupDesc{KIND_HIT, t.gi - 1, 0, 0} : ax.gtab[t.gi]);
            int *ctr = p.sync + SY_GROUP0 + t.gi;
            if (t.kind == TASK_ACT) {
                const bool hit = grp.kind == KIND_HIT;
                const int n_cols = hit ? dm.I : dm.Is;
                __nv_bfloat16 *out = hit ? p.act_hit16 + (size_t)(t.gi - 1) * T * dm.I : p.act_shared16;
                // The up rows reach the warps that hold the gate rows through a double-buffered exchange area of
                // XW token columns; a tile of 64 columns goes through it in two rounds (the buffers alternate, so the
                // rounds pipeline like consecutive tiles do), which keeps the area small enough for a deeper weight ring.
                constexpr int XW = NB > 32 ? 32 : NB, XR = NB / XW;
                // 8-bit weights: scale of this thread's weight row (gate rows first, then the up rows)
                float rs = 1.0f;
                if (F8) {
                    const int col = t.tile * 64 + (L & 63);
                    const float *sc = hit ? q.s_slot_gu + (size_t)grp.id * 2 * dm.I : q.s_sh_gu;
                    rs = col < n_cols ? sc[(qd >= 2 ? n_cols : 0) + col] : 0.0f;
                }
                bool dead = false;
#pragma unroll
                for (int xr = 0; xr < XR; ++xr, ++xc) {
                    const int xb = xc & 1;
                    const uint32_t xuse = xc >> 1;   // uses of this buffer so far
                    float *xch = ax.xch + xb * XW * 64;
                    if (qd >= 2) {   // up rows: park them for the warps that hold the gate rows
                        if (!warp_mb_wait(smem_u32(&sh->xch_empty[xb]), (xuse & 1) ^ 1, abort_flag, lane)) { dead = true; break; }
#pragma unroll
                        for (int nn = 0; nn < XW; ++nn)
                            xch[nn * 64 + (L - 64)] = F8 ? __uint_as_float(v[xr * XW + nn]) * rs : __uint_as_float(v[xr * XW + nn]);
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&sh->xch_full[xb]));
                    } else {
                        if (!warp_mb_wait(smem_u32(&sh->xch_full[xb]), xuse & 1, abort_flag, lane)) { dead = true; break; }
                        const int col = t.tile * 64 + L;
                        if (F8) {
                            // the activation, rounded to bf16 as in the 16-bit kernel, stored as its three E5M2 terms
                            uint8_t *out8 = hit ? q.act8_hit + (size_t)(t.gi - 1) * 3 * T * dm.I : q.act8_sh;
                            const size_t plane = (size_t)T * n_cols;
#pragma unroll
                            for (int nn = 0; nn < XW; ++nn) {
                                const int tk = xr * XW + nn;
                                if (tk < T && col < n_cols) {
                                    const float u = xch[nn * 64 + L];
                                    const float a = __bfloat162float(__float2bfloat16(silu_f(__uint_as_float(v[tk]) * rs) * u));
                                    const uint32_t b3 = split_e5m2x3(a);
                                    uint8_t *o = out8 + (size_t)tk * n_cols + col;
                                    o[0] = (uint8_t)b3;
                                    o[plane] = (uint8_t)(b3 >> 8);
                                    o[2 * plane] = (uint8_t)(b3 >> 16);
                                }
                            }
                        } else {
#pragma unroll
                            for (int nn = 0; nn < XW; ++nn) {
                                const int tk = xr * XW + nn;
                                if (tk < T && col < n_cols) {
                                    const float u = xch[nn * 64 + L];
                                    out[(size_t)tk * n_cols + col] = __float2bfloat16(silu_f(__uint_as_float(v[tk])) * u);
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&sh->xch_empty[xb]));
                    }
                }
                if (dead) break;
            } else if (t.kind == TASK_Z) {
                const int row = t.tile * 128 + L;
                __nv_bfloat16 *out = p.z16 + (size_t)(t.gi - 1 - sh->n_hg) * T * dm.r;
#pragma unroll
                for (int nn = 0; nn < NB; ++nn)
                    if (nn < T && row < dm.r) out[(size_t)nn * dm.r + row] = __float2bfloat16(__uint_as_float(v[nn]));
            } else {
                // down tile: token column n belongs to the group's entry of token n, if it has one.  The members are a bit
                // mask over the tokens (warp-uniform tests with constant shifts, no table in shared memory), and the entry of
                // member n is the rank(n)-th of the group's list, which is ordered by token.
                uint32_t m0, m1 = 0u;
                const int *perm = ax.perm_h;
                if (grp.kind == KIND_SHARED) {
                    m0 = T >= 32 ? 0xffffffffu : (1u << T) - 1u;
                    if (NB > 32) m1 = T >= 64 ? 0xffffffffu : (T > 32 ? (1u << (T - 32)) - 1u : 0u);
                } else {
                    const uint32_t *mk = grp.kind == KIND_HIT ? ax.mask_hit + 2 * grp.id : ax.mask_low + 2 * grp.id;
                    m0 = mk[0];
                    if (NB > 32) m1 = mk[1];
                    if (grp.kind != KIND_HIT) perm = ax.perm_l;
                }
                const int row = t.tile * 128 + L;
                float *out = grp.kind == KIND_SHARED ? q.part_split + (size_t)t.split * T * dm.d : p.tb.part;
                float rs = 1.0f;
                if (F8 && t.f8 && row < dm.d) rs = grp.kind == KIND_SHARED ? q.s_sh_d[row] : q.s_slot_d[(size_t)grp.id * dm.d + row];
                if (grp.kind == KIND_SHARED) {
#pragma unroll
                    for (int nn = 0; nn < NB; ++nn)
                        if (nn < T && row < dm.d) out[(size_t)nn * dm.d + row] = F8 ? __uint_as_float(v[nn]) * rs : __uint_as_float(v[nn]);
                } else {
                    // Few columns are members: a short loop over the set bits of the mask, the column's value picked out
                    // of the accumulator registers by a tree of selects on the bits of its index.  (Sixty-four unrolled
                    // tests with their stores were straight-line code of some 20 KB that every tile had to fetch again: 2 us
                    // per tile, which bounded the tiny B_e tiles at the end of the list.)
                    perm += grp.off;
                    unsigned long long mm = (unsigned long long)m0 | ((unsigned long long)m1 << 32);
                    int j = 0;
#pragma unroll 1
                    while (mm) {
                        const int nn = __ffsll((long long)mm) - 1;
                        mm &= mm - 1ull;
                        const int e = perm[j++];
                        const float val = __uint_as_float(pick_column<NB>(v, nn));
                        if (row < dm.d) out[(size_t)e * dm.d + row] = F8 ? val * rs : val;
                    }
                }
            }
            if (warp == 2 && lane == 0) DPROF(1, npf, 57);
            if (t.kind == TASK_DOWN) {
                ++n_down;
                if (ld_acquire_cta(&sh->no_more)) {   // (warp-uniform: one shared word)
                    __syncwarp();
                    if (lane == 0) red_release_add(p.sync + SY_P2_DONE, n_down);
                    n_down = 0;
                }
                if (lane == 0) mbar_arrive(smem_u32(&sh->tq_empty[slot]));
            } else {
                // Publish: only warps that stored rows signal (gate/up tiles: the two gate-row warps).  The release is
                // one loaded memory round trip; the proxy fence that the TMA reads of these rows need lies on the
                // reader's side of the release / acquire pair (in the producer), which keeps it off this path.
                __syncwarp();
                if (lane == 0) {
                    if (t.kind != TASK_ACT || qd < 2) red_release_add(ctr, 1);
                    mbar_arrive(smem_u32(&sh->tq_empty[slot]));
                }
            }
            if (warp == 2 && lane == 0) DPROF(1, npf, 55);
        }
        __syncwarp();
        if (lane == 0 && n_down) red_release_add(p.sync + SY_P2_DONE, n_down);
    } else {
        // ---------------- auxiliary team
        AuxCtx a;
        a.atid = threadIdx.x - AUX_T0;
        a.lane = lane;
        a.aw = a.atid >> 5;
        a.npf = 0;
        APROF(a, 60);
        const int T = dm.T, N = dm.N;
        // what classification will need is copied asynchronously (global -> shared) while the logits are produced
        const int n_conf = p.conf_stride ? T * N : T;
        if (!p.roll_depth) {   // (the rollout decides the classes by its halting rule)
#pragma unroll 1
            for (int i = a.atid; i < N; i += AUX_T) cp_async4(smem_u32(ax.soe + i), p.w.slot_of_expert + i);
            if (conf_staged(dm, p.conf_stride)) {
#pragma unroll 1
                for (int i = a.atid; i < n_conf; i += AUX_T) cp_async4(smem_u32(ax.conf + i), p.conf + i);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        if (a.atid < dm.S) ax.mask_hit[2 * a.atid] = ax.mask_hit[2 * a.atid + 1] = 0u;
        if (a.atid < N) ax.mask_low[2 * a.atid] = ax.mask_low[2 * a.atid + 1] = 0u;
        APROF(a, 61);
        if (F8) {
            // h as the sum of three E5M2 terms, written before anything else by the CTAs that hold no router-logit unit
            // (the first h8_ctas ones; all CTAs when fewer than 8 are free, then after their logits), a slice each;
            // published with one counter that the producers poll
            const int n = T * dm.d, nc = h8_ctas(q);
            if (nc < (int)gridDim.x) {
                if ((int)blockIdx.x < nc) {   // (CTA-uniform)
                    aux_split_h(q, a, n, blockIdx.x, nc);
                    aux_sync();
                    if (a.atid == 0) red_release_add(p.sync + SY_H8_DONE, 1);
                }
                aux_logits(q, a);
            } else {
                aux_logits(q, a);
                aux_split_h(q, a, n, blockIdx.x, nc);
                aux_sync();
                if (a.atid == 0) red_release_add(p.sync + SY_H8_DONE, 1);
            }
        } else {
            aux_logits(q, a);
        }
        if (a.atid == 0) mbar_arrive(smem_u32(&sh->logits_done));   // (after the barrier inside aux_logits, if it had units)
        APROF(a, 62);
        asm volatile("cp.async.wait_group 0;" ::: "memory");   // (made visible to the team by the barriers of the wait below)
        bool ok = aux_wait_ge(q, sh, a, p.sync + SY_R1_DONE, N * q.r1_sub);
        APROF(a, 63);
        if (ok) ok = aux_route(q, sh, ax, a);
        if (ok) {
            if (a.atid == 0) mbar_arrive(smem_u32(&sh->plan_ready));
            APROF(a, 64);
            if (blockIdx.x == 0) aux_write_outputs(q, sh, ax, a);
            Plan pl;
            plan_static(pl, q, KST);
            plan_routed(pl, sh->n_hg, sh->n_lg);
            // Warp 1 of the auxiliary team (warp 7 of the CTA) watches the per-group counters while the weights stream, so that the producer finds a flag in
            // shared memory instead of paying a round trip to L2 when it reaches a down tile.  It ends when every
            // group is complete (or on abort / after its time limit); the producer never depends on it.
            if (a.aw == 1) {
                const int n_groups = 1 + pl.n_hg + pl.n_lg;
                const long long w0 = clock64();
                bool all = false;
#pragma unroll 1
                for (int round = 0; !all; ++round) {
                    bool mine = true;
#pragma unroll 1
                    for (int g = a.lane; g < n_groups; g += 32) {
                        if (ax.ready[g]) continue;
                        const int target = g == 0 ? 2 * pl.tIs : (g <= pl.n_hg ? 2 * pl.tI : 4 * pl.tz);
                        if (ld_acquire(p.sync + SY_GROUP0 + g) >= target) st_release_cta(ax.ready + g, 1);
                        else mine = false;
                    }
                    all = __all_sync(0xffffffffu, mine);
                    if (!all) {
                        if (*abort_flag || ld_relaxed(p.sync + SY_ABORT) || clock64() - w0 > ROLE_WAIT_CYCLES) break;
                        __nanosleep(400);
                    }
                }
            }
            // combine units: 64 threads take 256 columns of one token
            const int nb = (dm.d + 255) >> 8, n_tasks = T * nb;
            if ((int)blockIdx.x * 4 < n_tasks) {   // CTA-uniform
                APROF(a, 65);
                ok = aux_wait_ge(q, sh, a, p.sync + SY_P2_DONE, 4 * ((pl.sh_early ? pl.nCs : 0) + pl.endC - pl.endB));
                APROF(a, 66);
                if (ok)
                    for (int task = blockIdx.x * 4 + (a.atid >> 6); task < n_tasks; task += gridDim.x * 4)
                        aux_combine(q, ax, task / nb, (task % nb) * 256 + (a.atid & 63) * 4);
                APROF(a, 67);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS));
    }
#ifdef SPICE_PROF
    if (threadIdx.x == 0 && blockIdx.x < PR_CTAS) {
        g_dtc_cal[blockIdx.x * 4 + 2] = now_ns();
        g_dtc_cal[blockIdx.x * 4 + 3] = (unsigned long long)clock64();
    }
#endif
    // The last CTA to finish clears the counters for the next launch.  Every other CTA has passed this point, aborted
    // or not, so the counters (the abort word among them) are nobody's any more: the next call on this ctx starts
    // clean even when this one gave up, and the sticky status word keeps the record of that.
    if (threadIdx.x == 0) {
        if (sh->abort_flag) atomicMax(p.tb.status, (int)SPICE_ERR_TIMEOUT);
        __threadfence();
        sh->last_flag = atomicAdd(p.sync + SY_TEAMS_DONE, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (sh->last_flag) {
        __threadfence();
        for (int i = threadIdx.x; i < p.sync_words; i += DTC_THREADS) p.sync[i] = 0;
    }
}

// ------------------------------------------------------------------------------------------
// host side
size_t dtc_smem_bytes(const Dims &dm, int conf_stride, int stages, bool f8) {
    const int nb = nb_of(dm.T);
    return 1024 + (size_t)stages * stage_bytes_of(nb, f8) + ((sizeof(Ctl) + 15) & ~size_t(15)) + aux_layout(dm, conf_stride, nb, nullptr, nullptr);
}

int dtc_stages(const Dims &dm, int conf_stride, size_t max_smem, bool f8) {
    for (int s = MAX_STAGES; s >= 3; --s)
        if (dtc_smem_bytes(dm, conf_stride, s, f8) <= max_smem) return s;
    return 0;
}

}  // namespace

bool decode_tc_supported(const Dims &dm, int conf_stride, size_t max_smem, bool f8) {
    if (dm.T < 1 || dm.T > (f8 ? 32 : 64)) return false;
    // 8-bit weights are viewed as [row][k-block][128 bytes]
    if (f8 && (dm.d % 128 || dm.I % 128 || dm.Is % 128)) return false;
    if (dm.N > 256 || dm.S > 256) return false;
    if ((size_t)dm.T * dm.K > 1024 || (size_t)dm.T * dm.N > 8192) return false;
    // the big operands are viewed as [row][k-block][64]: their reduction lengths must be whole k-blocks
    if (dm.d % 64 || dm.I % 64 || dm.Is % 64 || dm.r % 8) return false;
    if (decode_tc_nsplit(dm, f8) > MAX_SPLIT) return false;
    return dtc_stages(dm, conf_stride, max_smem, f8) >= 3;
}

int decode_tc_nsplit(const Dims &dm, bool f8) {
    const int kst = f8 ? KSTAGE8 : KSTAGE;
    const int kcIs = (dm.Is + kst - 1) / kst;
    return (kcIs + CHUNKS_PER_SPLIT - 1) / CHUNKS_PER_SPLIT;
}

int decode_tc_prepare(int max_smem_optin) {
    const void *fns[5] = {reinterpret_cast<const void *>(decode_tc_kernel<16>), reinterpret_cast<const void *>(decode_tc_kernel<32>),
                          reinterpret_cast<const void *>(decode_tc_kernel<64>), reinterpret_cast<const void *>(decode_tc_kernel<16, true>),
                          reinterpret_cast<const void *>(decode_tc_kernel<32, true>)};
    for (const void *fn : fns)
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem_optin) != cudaSuccess) return -1;
    return 0;
}

int launch_decode_tc(const DecodeParams &p, float *part_split, int n_ctas, int max_smem_optin, cudaStream_t st, const Fp8Layer *f8) {
    const Dims &dm = p.dm;
    DtcParams q{};
    q.p = p;
    q.part_split = part_split;
    q.stages = dtc_stages(dm, p.conf_stride, (size_t)max_smem_optin, f8 != nullptr);
    if (q.stages < 3) return -1;
    const int kst = f8 ? KSTAGE8 : KSTAGE;
    const int kcIs = (dm.Is + kst - 1) / kst;
    q.nsplit_sh = decode_tc_nsplit(dm, f8 != nullptr);
    q.cps_sh = (kcIs + q.nsplit_sh - 1) / q.nsplit_sh;
    int launches = 1;
    if (f8) {
        q.s_slot_gu = f8->s_slot_gu;
        q.s_slot_d = f8->s_slot_d;
        q.s_sh_gu = f8->s_sh_gu;
        q.s_sh_d = f8->s_sh_d;
        q.act8_hit = f8->act8_hit;
        q.act8_sh = f8->act8_sh;
        q.x8_h = f8->x8_h;
    }
    {
        const int per = (dm.T + AUX_W - 1) / AUX_W, fit = n_ctas / dm.N;
        q.r1_sub = per < 1 ? 1 : per;
        if (q.r1_sub > fit) q.r1_sub = fit < 1 ? 1 : fit;
    }
    {
        // Slots whose gate/up tiles stream before the routing is known (Sec. 4.2 leaves the order of the expert work open).
        // The routing tables exist 8 to 20 us into the kernel; until then only the shared expert's tiles are known, which
        // for a small shared expert leaves most SMs without work.  The first n_spec slots are therefore made groups
        // unconditionally and their gate/up tiles join the launch-time part of the list.  Their number: what fills about
        // 20 us of the stream beside the shared expert, scaled down by how likely a slot is to go unused.  Measured per
        // slot (DeepSeek-V2-Lite shape, 16 tokens, uniform and Zipf-skewed routers): a slot that is used shortens the call
        // by 0.56 us, one that is not lengthens it by 0.91 us (its gate/up bytes, part of them in time that was idle), so
        // streaming ahead pays while a slot goes unused with probability below 0.38.  Under uniform routing that
        // probability is (1 - K/N)^T; real routers are more skewed, so the count shrinks linearly from the full window at
        // probability 0 to nothing at 0.38 (16 tokens, 6 of 64 experts: 0.21, 4 of 8 slots; 32 tokens: 0.04, 7 slots).
        q.n_spec = 0;
        const double wb = f8 ? 1.0 : 2.0;
        const double shared_bytes = 3.0 * dm.Is * dm.d * wb, slot_gu_bytes = 2.0 * dm.I * dm.d * wb;
        const double window_bytes = f8 ? 72e6 : 128e6;   // (the 8-bit kernel streams fewer bytes per microsecond)
        const double p_unused = pow(1.0 - (double)dm.K / dm.N, (double)dm.T), p_even = 0.38;
        if (!p.roll_depth && p_unused < p_even && (long long)dm.T * dm.K >= dm.S && window_bytes > shared_bytes) {
            const int ns = (int)((window_bytes - shared_bytes) / slot_gu_bytes * (1.0 - p_unused / p_even) + 0.5);
            q.n_spec = ns > dm.S ? dm.S : ns;
        }
    }
    const int nb = nb_of(dm.T);
    const uint64_t T = dm.T, d = dm.d, I = dm.I, Is = dm.Is, r = dm.r;
    const uint64_t n = T * dm.K, g_hit = (uint64_t)dm.S < n ? dm.S : n, g_low = (uint64_t)dm.N < n ? dm.N : n;
    DtcMaps maps;
    bool ok = true;
    // big operands: (64 elements, rows, halves, k-blocks of 64, matrices); the box takes two k-blocks
    auto big = [&](int which, const void *base, uint64_t rows, uint64_t K, uint64_t halves, uint64_t mats, uint64_t mat_elems,
                   uint32_t box_rows) {
        const uint64_t dims[5] = {64, rows, halves, K / 64, mats};
        const uint64_t strides[4] = {K * 2, rows * K * 2, 128, mat_elems * 2};
        const uint32_t box[5] = {64, box_rows, (uint32_t)halves, 2, 1};
        ok = ok && tc_encode_map5(&maps.m[which], base, dims, strides, box);
    };
    // operands reduced over the LoRE rank: (k, rows, 1, 1, matrices), one 64-element box per sub-chunk
    auto plain = [&](int which, const void *base, uint64_t rows, uint64_t K, uint64_t mats, uint32_t box_rows) {
        const uint64_t dims[5] = {K, rows, 1, 1, mats};
        const uint64_t strides[4] = {K * 2, rows * K * 2, rows * K * 2, rows * K * 2};
        const uint32_t box[5] = {64, box_rows, 1, 1, 1};
        ok = ok && tc_encode_map5(&maps.m[which], base, dims, strides, box);
    };
    // 8-bit weights: (128 bytes, rows, halves, k-blocks of 128, matrices); the box takes two k-blocks
    auto big8 = [&](int which, const void *base, uint64_t rows, uint64_t K, uint64_t halves, uint64_t mats, uint64_t mat_bytes,
                    uint32_t box_rows) {
        const uint64_t dims[5] = {128, rows, halves, K / 128, mats};
        const uint64_t strides[4] = {K, rows * K, 128, mat_bytes};
        const uint32_t box[5] = {128, box_rows, (uint32_t)halves, 2, 1};
        ok = ok && tc_encode_map5(&maps.m[which], base, dims, strides, box, 1);
    };
    // activations as three E5M2 planes [group][3][T][K]: (128 bytes, tokens, terms, k-blocks, groups); the box takes all
    // three terms of nb tokens and two k-blocks and lands as [k-block][term][token][128]
    auto x8 = [&](int which, const void *base, uint64_t K, uint64_t groups) {
        const uint64_t dims[5] = {128, T, 3, K / 128, groups};
        const uint64_t strides[4] = {K, T * K, 128, 3 * T * K};
        const uint32_t box[5] = {128, (uint32_t)nb, 3, 2, 1};
        ok = ok && tc_encode_map5(&maps.m[which], base, dims, strides, box, 1);
    };
    big(MAP_H, p.h, T, d, 1, 1, T * d, nb);
    big(MAP_LORE_A, p.w.lore_A, r, d, 1, dm.N, r * d, 128);
    plain(MAP_LORE_B, p.w.lore_B, d, r, dm.N, 128);
    plain(MAP_Z, p.z16, T, r, g_low, nb);
    if (f8) {
        big8(MAP_SLOT_GU, f8->q_slot_gu, I, d, 2, dm.S, 2 * I * d, 64);
        big8(MAP_SH_GU, f8->q_sh_gu, Is, d, 2, 1, 2 * Is * d, 64);
        big8(MAP_SLOT_D, f8->q_slot_d, d, I, 1, dm.S, d * I, 128);
        big8(MAP_SH_D, f8->q_sh_d, d, Is, 1, 1, d * Is, 128);
        x8(MAP_X8, f8->x8_h, d, 1);
        x8(MAP_ACT_HIT, f8->act8_hit, I, g_hit);
        x8(MAP_ACT_SH, f8->act8_sh, Is, 1);
    } else {
        big(MAP_SLOT_GU, p.w.slot_w_gate_up, I, d, 2, dm.S, 2 * I * d, 64);
        big(MAP_SH_GU, p.w.shared_w_gate_up, Is, d, 2, 1, 2 * Is * d, 64);
        big(MAP_SLOT_D, p.w.slot_w_down, d, I, 1, dm.S, d * I, 128);
        big(MAP_SH_D, p.w.shared_w_down, d, Is, 1, 1, d * Is, 128);
        big(MAP_ACT_HIT, p.act_hit16, T, I, 1, g_hit, T * I, nb);
        big(MAP_ACT_SH, p.act_shared16, T, Is, 1, 1, T * Is, nb);
        maps.m[MAP_X8] = maps.m[MAP_H];   // (never used)
    }
    if (!ok) return -1;
    const size_t smem = dtc_smem_bytes(dm, p.conf_stride, q.stages, f8 != nullptr);
    const void *fn;
    if (f8)
        fn = nb == 16 ? reinterpret_cast<const void *>(decode_tc_kernel<16, true>) : reinterpret_cast<const void *>(decode_tc_kernel<32, true>);
    else
        fn = nb == 16 ? reinterpret_cast<const void *>(decode_tc_kernel<16>)
                      : (nb == 32 ? reinterpret_cast<const void *>(decode_tc_kernel<32>) : reinterpret_cast<const void *>(decode_tc_kernel<64>));
    void *args[] = {&q, &maps};
    if (cudaLaunchCooperativeKernel(fn, dim3(n_ctas), dim3(DTC_THREADS), args, smem, st) != cudaSuccess) {
        cudaGetLastError();
        return -1;
    }
    return launches;
}

#ifdef SPICE_PROF
extern "C" int spice_debug_dtc_prof_read(unsigned long long *host, size_t n_words) {
    const size_t total = sizeof(unsigned long long) * (size_t)PR_CTAS * PR_ROLES * PR_EVENTS * 2;
    if (n_words * 8 < total) return -1;
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(host, g_dtc_prof, total) == cudaSuccess ? 0 : -2;
}
extern "C" int spice_debug_dtc_cal_read(unsigned long long *host) {
    cudaDeviceSynchronize();
    return cudaMemcpyFromSymbol(host, g_dtc_cal, sizeof(unsigned long long) * PR_CTAS * 4) == cudaSuccess ? 0 : -2;
}
extern "C" int spice_debug_dtc_prof_clear(void) {
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_dtc_prof) != cudaSuccess) return -1;
    return cudaMemset(ptr, 0, sizeof(unsigned long long) * (size_t)PR_CTAS * PR_ROLES * PR_EVENTS * 2) == cudaSuccess ? 0 : -2;
}
#endif

}  // namespace spice
