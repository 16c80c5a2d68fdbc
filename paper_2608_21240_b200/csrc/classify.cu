// Hit / miss / low-confidence classification (runtime policy of Sec. 4.2 of the paper), the
// residual-miss list (set M of Sec. 4.3) and the token-to-expert grouping that the expert kernels
// consume.  For decode batches both run as ONE CTA: the tables are a few thousand entries at most and
// every step is a histogram, a scan or an ordered compaction.  Large batches (tens of thousands of
// entries) use multi-CTA variants of the same steps: element-wise passes over the entries with
// warp-aggregated global atomics, and one small scan in between.
#include "spice_internal.cuh"

namespace spice {

constexpr int CT = 1024;  // threads of the single CTA

// exclusive scan of one value per thread across the CTA; returns the exclusive prefix and the total
__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_tot /* [33] smem */, int &total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
    }
    __syncthreads();   // protect warp_tot from the previous use
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int n = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += n;
        }
        warp_tot[lane] = winc - w;
        if (lane == 31) warp_tot[32] = winc;
    }
    __syncthreads();
    total = warp_tot[32];
    return warp_tot[warp] + inc - v;
}

// (cls and slot carry no __restrict__: the fused kernel below reads them back after a barrier)
__device__ __forceinline__ void classify_body(int T, int N, int K, int S, int conf_stride, float tau,
                                              const int32_t *__restrict__ idx, const float *__restrict__ gate,
                                              const int32_t *__restrict__ slot_of_expert, const float *__restrict__ conf,
                                              uint8_t *cls, int32_t *slot, int32_t *__restrict__ counts,
                                              int32_t *__restrict__ resid_tok, int32_t *__restrict__ resid_k,
                                              int32_t *__restrict__ resid_expert, float *__restrict__ resid_gate,
                                              int32_t *__restrict__ status) {
    __shared__ int warp_tot[33];
    __shared__ int s_cnt[3];
    if (threadIdx.x < 3) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    const int n = T * K;
    int base = 0;   // residual entries emitted by earlier chunks
    for (int i0 = 0; i0 < n; i0 += CT) {
        const int i = i0 + threadIdx.x;
        int c = -1, e = 0, sl = -1;
        if (i < n) {
            e = idx[i];
            if (e < 0 || e >= N) {                 // cannot happen after spice_route_topk
                atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
                c = SPICE_MISS_EXACT;
            } else {
                sl = slot_of_expert[e];
                if (sl >= S) {                     // corrupt table entry: do not touch the pool
                    atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
                    sl = -1;
                    c = SPICE_MISS_EXACT;
                } else if (sl >= 0) {
                    c = SPICE_HIT;
                } else {
                    sl = -1;
                    const int t = i / K;
                    const float cf = conf_stride ? conf[(size_t)t * conf_stride + e] : conf[t];
                    c = (cf < tau) ? SPICE_LOWCONF : SPICE_MISS_EXACT;
                }
            }
            cls[i] = (uint8_t)c;
            slot[i] = sl;
            atomicAdd(&s_cnt[c], 1);
        }
        int total;
        const int pos = block_exclusive_scan(c == SPICE_MISS_EXACT ? 1 : 0, warp_tot, total);
        if (c == SPICE_MISS_EXACT && resid_tok) {
            const int o = base + pos;
            resid_tok[o] = i / K;
            resid_k[o] = i % K;
            resid_expert[o] = e;
            resid_gate[o] = gate[i];
        }
        base += total;
    }
    __syncthreads();
    if (threadIdx.x < 3) counts[threadIdx.x] = s_cnt[threadIdx.x];
}

__global__ void __launch_bounds__(CT) classify_kernel(int T, int N, int K, int S, int conf_stride, float tau,
                                                      const int32_t *__restrict__ idx, const float *__restrict__ gate,
                                                      const int32_t *__restrict__ slot_of_expert,
                                                      const float *__restrict__ conf, uint8_t *__restrict__ cls,
                                                      int32_t *__restrict__ slot, int32_t *__restrict__ counts,
                                                      int32_t *__restrict__ resid_tok, int32_t *__restrict__ resid_k,
                                                      int32_t *__restrict__ resid_expert,
                                                      float *__restrict__ resid_gate, int32_t *__restrict__ status) {
    classify_body(T, N, K, S, conf_stride, tau, idx, gate, slot_of_expert, conf, cls, slot, counts, resid_tok, resid_k,
                  resid_expert, resid_gate, status);
}

// Builds, from cls / slot / idx / gate:
//   groups[0] = shared expert (m = T); then one group per slot with >= 1 HIT entry (slot order);
//   then one group per expert with >= 1 LOWCONF entry (expert order);
//   perm_hit / perm_low: entry ids grouped accordingly; pos_of_entry; coef_shared[t] = 1 + sum of
//   LOWCONF gates in k order.
// Positions inside a group are handed out by warp-aggregated shared-memory atomics; the order of
// entries inside a group is therefore not fixed, which no result depends on (every entry's row is
// computed independently and the combine step gathers by entry id).
__device__ __forceinline__ void group_body(int T, int N, int K, int S, const int32_t *__restrict__ idx,
                                           const float *__restrict__ gate, const uint8_t *cls, const int32_t *slot, Tables tb) {
    __shared__ int warp_tot[33];
    __shared__ int cnt_hit[1024], cnt_low[1024];   // later reused as cursors
    __shared__ int off_hit[1024], off_low[1024];
    const int tid = threadIdx.x, lane = tid & 31;
    const int n = T * K;
    cnt_hit[tid] = 0;
    cnt_low[tid] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += CT) {
        const int c = cls[i];
        if (c == SPICE_HIT) {
            if (!slot) continue;   // caller only wants the shared / low-confidence groups
            const int s = slot[i];
            if (s >= 0 && s < S) atomicAdd(&cnt_hit[s], 1);
            else atomicMax(tb.status, (int)SPICE_ERR_BAD_TABLE);
        } else if (c == SPICE_LOWCONF) {
            const int e = idx[i];
            if (e >= 0 && e < N) atomicAdd(&cnt_low[e], 1);
            else atomicMax(tb.status, (int)SPICE_ERR_BAD_TABLE);
        }
    }
    __syncthreads();
    const int ch = cnt_hit[tid], cl = cnt_low[tid];
    int n_hit, n_low, n_hg, n_lg;
    const int oh = block_exclusive_scan(ch, warp_tot, n_hit);
    const int ol = block_exclusive_scan(cl, warp_tot, n_low);
    const int gh = block_exclusive_scan(ch > 0 ? 1 : 0, warp_tot, n_hg);
    const int gl = block_exclusive_scan(cl > 0 ? 1 : 0, warp_tot, n_lg);
    off_hit[tid] = oh;
    off_low[tid] = ol;
    if (ch > 0) tb.groups[1 + gh] = GroupDesc{KIND_HIT, tid, oh, ch};
    if (cl > 0) tb.groups[1 + n_hg + gl] = GroupDesc{KIND_LOW, tid, ol, cl};
    if (tid == 0) {
        tb.groups[0] = GroupDesc{KIND_SHARED, 0, 0, T};
        tb.hdr[HDR_N_GROUPS] = 1 + n_hg + n_lg;
        tb.hdr[HDR_N_HIT_GROUPS] = n_hg;
        tb.hdr[HDR_N_LOW_GROUPS] = n_lg;
        tb.hdr[HDR_N_HIT] = n_hit;
        tb.hdr[HDR_N_LOW] = n_low;
    }
    __syncthreads();
    cnt_hit[tid] = 0;   // cursors
    cnt_low[tid] = 0;
    __syncthreads();
    for (int i0 = 0; i0 < n; i0 += CT) {   // warp-uniform trip count
        const int i = i0 + tid;
        int key = -1;                        // 0..1023 hit slot, 1024..2047 low expert
        if (i < n) {
            const int c = cls[i];
            if (c == SPICE_HIT) {
                const int s = slot ? slot[i] : -1;
                if (s >= 0 && s < S) key = s;
            } else if (c == SPICE_LOWCONF) {
                const int e = idx[i];
                if (e >= 0 && e < N) key = 1024 + e;
            }
        }
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        int pos = -1;
        if (key >= 0) {
            const int leader = __ffs(peers) - 1;
            int basep = 0;
            if (lane == leader)
                basep = (key < 1024) ? atomicAdd(&cnt_hit[key], __popc(peers))
                                     : atomicAdd(&cnt_low[key - 1024], __popc(peers));
            basep = __shfl_sync(peers, basep, leader);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            if (key < 1024) {
                pos = off_hit[key] + basep + rank;
                tb.perm_hit[pos] = i;
            } else {
                pos = off_low[key - 1024] + basep + rank;
                tb.perm_low[pos] = i;
            }
        }
        if (i < n) tb.pos_of_entry[i] = pos;
    }
    for (int t = tid; t < T; t += CT) {
        float c = 1.0f;
        for (int k = 0; k < K; ++k)
            if (cls[t * K + k] == SPICE_LOWCONF) c += gate[t * K + k];
        tb.coef_shared[t] = c;
    }
}

__global__ void __launch_bounds__(CT) group_kernel(int T, int N, int K, int S, const int32_t *__restrict__ idx,
                                                   const float *__restrict__ gate, const uint8_t *__restrict__ cls,
                                                   const int32_t *__restrict__ slot, Tables tb) {
    group_body(T, N, K, S, idx, gate, cls, slot, tb);
}

// Both steps in one launch for batches whose tables one CTA builds: classification, a barrier (the classes and slots
// it wrote are read back by the same CTA), grouping.
__global__ void __launch_bounds__(CT) classify_group_kernel(int T, int N, int K, int S, int conf_stride, float tau,
                                                            const int32_t *__restrict__ idx, const float *__restrict__ gate,
                                                            const int32_t *__restrict__ slot_of_expert,
                                                            const float *__restrict__ conf, uint8_t *cls, int32_t *slot,
                                                            int32_t *__restrict__ counts, int32_t *__restrict__ resid_tok,
                                                            int32_t *__restrict__ resid_k, int32_t *__restrict__ resid_expert,
                                                            float *__restrict__ resid_gate, int32_t *__restrict__ status, Tables tb) {
    classify_body(T, N, K, S, conf_stride, tau, idx, gate, slot_of_expert, conf, cls, slot, counts, resid_tok, resid_k,
                  resid_expert, resid_gate, status);
    __syncthreads();
    group_body(T, N, K, S, idx, gate, cls, slot, tb);
}

// ---------------------------------------------------------------------------------------------
// Multi-CTA variants for large batches.

// classification of 1024 entries per CTA; counts by atomics; blk_miss[b] = exact-recovery misses of chunk b
__global__ void __launch_bounds__(CT) classify_mc_kernel(int T, int N, int K, int S, int conf_stride, float tau,
                                                         const int32_t *__restrict__ idx, const int32_t *__restrict__ slot_of_expert,
                                                         const float *__restrict__ conf, uint8_t *__restrict__ cls,
                                                         int32_t *__restrict__ slot, int32_t *__restrict__ counts,
                                                         int32_t *__restrict__ blk_miss, int32_t *__restrict__ status) {
    __shared__ int s_cnt[3];
    if (threadIdx.x < 3) s_cnt[threadIdx.x] = 0;
    __syncthreads();
    const int n = T * K;
    const int i = blockIdx.x * CT + threadIdx.x;
    if (i < n) {
        int c, sl = -1;
        const int e = idx[i];
        if (e < 0 || e >= N) {
            atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
            c = SPICE_MISS_EXACT;
        } else {
            sl = slot_of_expert[e];
            if (sl >= S) {
                atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
                sl = -1;
                c = SPICE_MISS_EXACT;
            } else if (sl >= 0) {
                c = SPICE_HIT;
            } else {
                sl = -1;
                const int t = i / K;
                const float cf = conf_stride ? conf[(size_t)t * conf_stride + e] : conf[t];
                c = (cf < tau) ? SPICE_LOWCONF : SPICE_MISS_EXACT;
            }
        }
        cls[i] = (uint8_t)c;
        slot[i] = sl;
        atomicAdd(&s_cnt[c], 1);
    }
    __syncthreads();
    if (threadIdx.x < 3 && s_cnt[threadIdx.x]) atomicAdd(&counts[threadIdx.x], s_cnt[threadIdx.x]);
    if (threadIdx.x == 0) blk_miss[blockIdx.x] = s_cnt[SPICE_MISS_EXACT];
}

// residual-miss list in (t,k) order: chunk b starts at the sum of the earlier chunks' miss counts
__global__ void __launch_bounds__(CT) resid_scatter_kernel(int T, int K, const int32_t *__restrict__ idx, const float *__restrict__ gate,
                                                           const uint8_t *__restrict__ cls, const int32_t *__restrict__ blk_miss,
                                                           int32_t *__restrict__ resid_tok, int32_t *__restrict__ resid_k,
                                                           int32_t *__restrict__ resid_expert, float *__restrict__ resid_gate) {
    __shared__ int warp_tot[33];
    __shared__ int s_base;
    int part = 0;
    for (int b = threadIdx.x; b < (int)blockIdx.x; b += CT) part += blk_miss[b];
    int total;
    block_exclusive_scan(part, warp_tot, total);
    if (threadIdx.x == 0) s_base = total;
    __syncthreads();
    const int base = s_base;
    const int n = T * K, i = blockIdx.x * CT + threadIdx.x;
    const bool miss = i < n && cls[i] == SPICE_MISS_EXACT;
    const int pos = block_exclusive_scan(miss ? 1 : 0, warp_tot, total);
    if (miss) {
        const int o = base + pos;
        resid_tok[o] = i / K;
        resid_k[o] = i % K;
        resid_expert[o] = idx[i];
        resid_gate[o] = gate[i];
    }
}

__device__ __forceinline__ int group_key(int i, int N, int S, const int32_t *idx, const uint8_t *cls, const int32_t *slot,
                                         int32_t *status) {
    const int c = cls[i];
    if (c == SPICE_HIT) {
        if (!slot) return -1;
        const int s = slot[i];
        if (s >= 0 && s < S) return s;
        atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
    } else if (c == SPICE_LOWCONF) {
        const int e = idx[i];
        if (e >= 0 && e < N) return 1024 + e;
        atomicMax(status, (int)SPICE_ERR_BAD_TABLE);
    }
    return -1;
}

// entries per slot / per expert, warp-aggregated; cnt[0..1023] slots, cnt[1024..2047] experts
__global__ void __launch_bounds__(256) group_hist_kernel(int n, int N, int S, const int32_t *__restrict__ idx,
                                                         const uint8_t *__restrict__ cls, const int32_t *__restrict__ slot,
                                                         int32_t *cnt, int32_t *status) {
    const int lane = threadIdx.x & 31;
    for (int i0 = blockIdx.x * 256; i0 < n; i0 += gridDim.x * 256) {   // warp-uniform trip count
        const int i = i0 + threadIdx.x;
        const int key = i < n ? group_key(i, N, S, idx, cls, slot, status) : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        if (key >= 0 && lane == __ffs(peers) - 1) atomicAdd(&cnt[key], __popc(peers));
    }
}

// group table, offsets and header from the counts (one CTA, thread i owns slot i and expert i)
__global__ void __launch_bounds__(CT) group_scan_kernel(int T, const int32_t *__restrict__ cnt, int32_t *__restrict__ off, Tables tb) {
    __shared__ int warp_tot[33];
    const int tid = threadIdx.x;
    const int ch = cnt[tid], cl = cnt[1024 + tid];
    int n_hit, n_low, n_hg, n_lg;
    const int oh = block_exclusive_scan(ch, warp_tot, n_hit);
    const int ol = block_exclusive_scan(cl, warp_tot, n_low);
    const int gh = block_exclusive_scan(ch > 0 ? 1 : 0, warp_tot, n_hg);
    const int gl = block_exclusive_scan(cl > 0 ? 1 : 0, warp_tot, n_lg);
    off[tid] = oh;
    off[1024 + tid] = ol;
    if (ch > 0) tb.groups[1 + gh] = GroupDesc{KIND_HIT, tid, oh, ch};
    if (cl > 0) tb.groups[1 + n_hg + gl] = GroupDesc{KIND_LOW, tid, ol, cl};
    if (tid == 0) {
        tb.groups[0] = GroupDesc{KIND_SHARED, 0, 0, T};
        tb.hdr[HDR_N_GROUPS] = 1 + n_hg + n_lg;
        tb.hdr[HDR_N_HIT_GROUPS] = n_hg;
        tb.hdr[HDR_N_LOW_GROUPS] = n_lg;
        tb.hdr[HDR_N_HIT] = n_hit;
        tb.hdr[HDR_N_LOW] = n_low;
    }
}

// positions inside the groups (order inside a group is not fixed, as in the single-CTA kernel) and the shared coefficient
__global__ void __launch_bounds__(256) group_scatter_kernel(int T, int N, int K, int S, const int32_t *__restrict__ idx,
                                                            const float *__restrict__ gate, const uint8_t *__restrict__ cls,
                                                            const int32_t *__restrict__ slot, const int32_t *__restrict__ off,
                                                            int32_t *cursor, Tables tb) {
    const int lane = threadIdx.x & 31, n = T * K;
    for (int i0 = blockIdx.x * 256; i0 < n; i0 += gridDim.x * 256) {   // warp-uniform trip count
        const int i = i0 + threadIdx.x;
        const int key = i < n ? group_key(i, N, S, idx, cls, slot, tb.status) : -1;
        const unsigned peers = __match_any_sync(0xffffffffu, key);
        int pos = -1;
        if (key >= 0) {
            const int leader = __ffs(peers) - 1;
            int basep = 0;
            if (lane == leader) basep = atomicAdd(&cursor[key], __popc(peers));
            basep = __shfl_sync(peers, basep, leader);
            pos = off[key] + basep + __popc(peers & ((1u << lane) - 1u));
            if (key < 1024) tb.perm_hit[pos] = i;
            else tb.perm_low[pos] = i;
        }
        if (i < n) tb.pos_of_entry[i] = pos;
    }
    for (int t = blockIdx.x * 256 + threadIdx.x; t < T; t += gridDim.x * 256) {
        float c = 1.0f;
        for (int k = 0; k < K; ++k)
            if (cls[t * K + k] == SPICE_LOWCONF) c += gate[t * K + k];
        tb.coef_shared[t] = c;
    }
}

constexpr int MC_ENTRIES = 4096;   // batches with more (token, expert) entries than this use the multi-CTA kernels

int launch_classify(const Dims &dm, int conf_stride, float tau, const int32_t *idx, const float *gate,
                    const int32_t *slot_of_expert, const float *conf, uint8_t *cls, int32_t *slot,
                    int32_t *counts, int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                    float *resid_gate, int32_t *status, cudaStream_t st, const GroupScratch *scratch) {
    const int n = dm.T * dm.K;
    if (scratch && scratch->blk_miss && n > MC_ENTRIES) {
        const int blocks = (n + CT - 1) / CT;
        if (cudaMemsetAsync(counts, 0, 3 * sizeof(int32_t), st) != cudaSuccess) return -1;
        classify_mc_kernel<<<blocks, CT, 0, st>>>(dm.T, dm.N, dm.K, dm.S, conf_stride, tau, idx, slot_of_expert, conf, cls, slot,
                                                  counts, scratch->blk_miss, status);
        if (cudaGetLastError() != cudaSuccess) return -1;
        if (!resid_tok) return 1;
        resid_scatter_kernel<<<blocks, CT, 0, st>>>(dm.T, dm.K, idx, gate, cls, scratch->blk_miss, resid_tok, resid_k, resid_expert,
                                                    resid_gate);
        return cudaGetLastError() == cudaSuccess ? 2 : -1;
    }
    classify_kernel<<<1, CT, 0, st>>>(dm.T, dm.N, dm.K, dm.S, conf_stride, tau, idx, gate, slot_of_expert, conf, cls,
                                      slot, counts, resid_tok, resid_k, resid_expert, resid_gate, status);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_classify_group(const Dims &dm, int conf_stride, float tau, const int32_t *idx, const float *gate,
                          const int32_t *slot_of_expert, const float *conf, uint8_t *cls, int32_t *slot, int32_t *counts,
                          int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert, float *resid_gate, const Tables &tb,
                          cudaStream_t st, const GroupScratch *scratch) {
    if (dm.T * dm.K > MC_ENTRIES) {
        const int a = launch_classify(dm, conf_stride, tau, idx, gate, slot_of_expert, conf, cls, slot, counts, resid_tok, resid_k,
                                      resid_expert, resid_gate, tb.status, st, scratch);
        if (a < 0) return -1;
        const int b = launch_group(dm, idx, gate, cls, slot, tb, st, scratch);
        return b < 0 ? -1 : a + b;
    }
    classify_group_kernel<<<1, CT, 0, st>>>(dm.T, dm.N, dm.K, dm.S, conf_stride, tau, idx, gate, slot_of_expert, conf, cls, slot,
                                            counts, resid_tok, resid_k, resid_expert, resid_gate, tb.status, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_group(const Dims &dm, const int32_t *idx, const float *gate, const uint8_t *cls, const int32_t *slot,
                 const Tables &tb, cudaStream_t st, const GroupScratch *scratch) {
    const int n = dm.T * dm.K;
    if (scratch && scratch->cnt && n > MC_ENTRIES) {
        // cnt and cursor are adjacent: one clear
        if (cudaMemsetAsync(scratch->cnt, 0, 2 * 2048 * sizeof(int32_t), st) != cudaSuccess) return -1;
        const int blocks = min((n + 255) / 256, 592);
        group_hist_kernel<<<blocks, 256, 0, st>>>(n, dm.N, dm.S, idx, cls, slot, scratch->cnt, tb.status);
        group_scan_kernel<<<1, CT, 0, st>>>(dm.T, scratch->cnt, scratch->off, tb);
        group_scatter_kernel<<<blocks, 256, 0, st>>>(dm.T, dm.N, dm.K, dm.S, idx, gate, cls, slot, scratch->off,
                                                     scratch->cnt + 2048, tb);
        return cudaGetLastError() == cudaSuccess ? 3 : -1;
    }
    group_kernel<<<1, CT, 0, st>>>(dm.T, dm.N, dm.K, dm.S, idx, gate, cls, slot, tb);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace spice
