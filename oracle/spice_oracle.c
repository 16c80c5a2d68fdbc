/*
 * spice_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, obviously-correct CPU statement of the GPU part of one offloaded-MoE
 * decode layer as the SPICE paper defines it.  It exists only so that tests, the smoke
 * check and the benchmark's CPU-baseline leg have something independent to compare the
 * CUDA library with.  It shares no code, header, table or helper with the CUDA path and
 * nothing in the product may call it.
 *
 * Precision: inputs are fp32 values (the same bf16-representable numbers the GPU gets),
 * every sum and every transcendental is carried in fp64, outputs are fp64.  There is no
 * blocking, fusion or reordering: each function is the formula of the cited passage
 * written as loops.  OpenMP only distributes independent output elements over threads.
 *
 * The layer (all citations are to the paper):
 *   routing            S_t = TopK(Router(h_t), K)                        Eq. 1, Sec. 2.2
 *   aggregation        shared experts always on; routed outputs weighted  Sec. 2.1
 *   hit                resident/prefetched expert -> executed exactly     Sec. 4.2 (runtime policy)
 *   low-conf. miss     y~_e = S(h) + B_e A_e h  (LoRE surrogate)          Sec. 4.2, Eqs. for y~_e, Delta_e
 *   remaining misses   exact recovery elsewhere (set M of Sec. 4.3); here they are only listed
 *
 * Readings taken where the paper is silent (kept identical in the CUDA library):
 *   - Router is a bias-free linear map followed by softmax; TopK picks the K largest
 *     logits, equal logits resolved towards the smaller expert index.
 *   - Gates are the softmax restricted to the K winners (norm_topk=1, they sum to 1) or
 *     the un-renormalised full-softmax probabilities (norm_topk=0).
 *   - A miss's "routing confidence" is the draft model's probability for that expert,
 *     conf[t,e] (or one scalar per token when conf_stride==0); LOWCONF iff conf < tau,
 *     strictly; NaN compares false and therefore means exact recovery.
 *   - The surrogate replaces the routed expert inside the gate-weighted sum, so the
 *     shared output enters with coefficient 1 + sum of LOWCONF gates.
 *   - Gates are not renormalised after exact-recovery misses are left out.
 *   - Expert FFN is SwiGLU: E(x) = W_d ( silu(W_g x) * (W_u x) ), silu(v) = v / (1 + exp(-v)).
 *
 * Pins (tests/test_oracle_pins.py): brute-force dense evaluation through an independent
 * numpy path, gate invariants, all-hit reduction to the standard MoE layer, rank-sufficient
 * LoRE reproducing the exact expert, closed forms for all-miss cases, threshold edges, a
 * hand-computed example (tests/golden/swiglu_hand_example.txt).  No function is unpinned.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>

#define ORACLE_HIT 0
#define ORACLE_MISS_EXACT 1
#define ORACLE_LOWCONF 2

typedef struct {
    int32_t d;            /* hidden width */
    int32_t n_experts;    /* N */
    int32_t top_k;        /* K */
    int32_t inter;        /* I   routed intermediate width */
    int32_t inter_shared; /* I_s shared intermediate width */
    int32_t lore_rank;    /* r */
    int32_t norm_topk;    /* 1: gates renormalised over the K winners */
    int32_t conf_stride;  /* N: conf[t*N+e]; 0: conf[t] */
    float tau;            /* confidence threshold */
} oracle_cfg;

static double dot_fd(const float *w, const float *x, int n) {
    double acc = 0.0;
    for (int j = 0; j < n; ++j) acc += (double)w[j] * (double)x[j];
    return acc;
}

static double dot_fdd(const float *w, const double *x, int n) {
    double acc = 0.0;
    for (int j = 0; j < n; ++j) acc += (double)w[j] * x[j];
    return acc;
}

/* Eq. 1: Router(h_t) as a linear map.  logits[t,e] = sum_j W_r[e,j] h[t,j]. */
void oracle_router_logits(int T, int d, int N, const float *h, const float *w_router, double *logits) {
#pragma omp parallel for collapse(2) schedule(static)
    for (int t = 0; t < T; ++t)
        for (int e = 0; e < N; ++e)
            logits[(size_t)t * N + e] = dot_fd(w_router + (size_t)e * d, h + (size_t)t * d, d);
}

/* Eq. 1 TopK and the gate scores that the runtime policy of Sec. 4.2 takes as its input.
 * K rounds of arg-max over the experts not yet taken; ties go to the smaller index.
 * idx[t,0..K-1] is in order of decreasing logit. */
void oracle_topk_gates(int T, int N, int K, int norm_topk, const double *logits, int32_t *idx, double *gate) {
    for (int t = 0; t < T; ++t) {
        const double *l = logits + (size_t)t * N;
        int32_t *ix = idx + (size_t)t * K;
        double *g = gate + (size_t)t * K;
        for (int k = 0; k < K; ++k) {
            int best = -1;
            for (int e = 0; e < N; ++e) {
                int taken = 0;
                for (int q = 0; q < k; ++q)
                    if (ix[q] == e) taken = 1;
                if (taken) continue;
                if (best < 0 || l[e] > l[best]) best = e;
            }
            ix[k] = best;
        }
        double m = l[ix[0]];
        double denom = 0.0;
        if (norm_topk) {
            for (int k = 0; k < K; ++k) denom += exp(l[ix[k]] - m);
        } else {
            for (int e = 0; e < N; ++e) denom += exp(l[e] - m);
        }
        for (int k = 0; k < K; ++k) g[k] = exp(l[ix[k]] - m) / denom;
    }
}

/* Draft-router confidence of Sec. 4.1: pi_hat = softmax(draft logits) over all N experts,
 * S_hat = TopK(pi_hat, K) (Eq. 2), C(pi_hat) = sum_{i in S_hat} pi_hat_i (Eq. 5).
 * Written out from the definitions: the full distribution first, then K rounds of arg-max over the
 * probabilities not yet taken (ties to the smaller index), then the sum in order of selection. */
void oracle_draft_confidence(int T, int N, int K, const double *logits, int32_t *idx_hat, double *pi_hat, double *conf) {
    for (int t = 0; t < T; ++t) {
        const double *l = logits + (size_t)t * N;
        double *p = pi_hat + (size_t)t * N;
        int32_t *ix = idx_hat + (size_t)t * K;
        double m = l[0];
        for (int e = 1; e < N; ++e)
            if (l[e] > m) m = l[e];
        double denom = 0.0;
        for (int e = 0; e < N; ++e) denom += exp(l[e] - m);
        for (int e = 0; e < N; ++e) p[e] = exp(l[e] - m) / denom;
        double c = 0.0;
        for (int k = 0; k < K; ++k) {
            int best = -1;
            for (int e = 0; e < N; ++e) {
                int taken = 0;
                for (int q = 0; q < k; ++q)
                    if (ix[q] == e) taken = 1;
                if (taken) continue;
                /* compare the logits: exp is monotone but may round two different logits to one probability */
                if (best < 0 || l[e] > l[best]) best = e;
            }
            ix[k] = best;
            c += p[best];
        }
        conf[t] = c;
    }
}

/* Sec. 4.2 runtime policy: resident -> exact (HIT); missing and low confidence -> surrogate
 * (LOWCONF); any other miss -> exact recovery (MISS_EXACT).  counts[c] = entries of class c. */
void oracle_classify(int T, int N, int K, const int32_t *idx, const uint8_t *resident, const float *conf,
                     int conf_stride, float tau, uint8_t *cls, int32_t *counts) {
    counts[0] = counts[1] = counts[2] = 0;
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < K; ++k) {
            int e = idx[(size_t)t * K + k];
            uint8_t c;
            if (resident[e]) {
                c = ORACLE_HIT;
            } else {
                float cf = conf_stride ? conf[(size_t)t * conf_stride + e] : conf[t];
                c = (cf < tau) ? ORACLE_LOWCONF : ORACLE_MISS_EXACT;
            }
            cls[(size_t)t * K + k] = c;
            counts[c] += 1;
        }
}

/* Exact expert output y_e = E_e(h) (Sec. 4.2), E a SwiGLU FFN.
 * w_gate, w_up: [I,d]; w_down: [d,I]; x: [d]; out: [d]. */
int oracle_swiglu_ffn(int d, int I, const float *w_gate, const float *w_up, const float *w_down,
                      const float *x, double *out) {
    double *a = (double *)malloc(sizeof(double) * (size_t)I);
    if (!a) return -1;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < I; ++i) {
        double g = dot_fd(w_gate + (size_t)i * d, x, d);
        double u = dot_fd(w_up + (size_t)i * d, x, d);
        a[i] = (g / (1.0 + exp(-g))) * u;
    }
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d; ++j) out[j] = dot_fdd(w_down + (size_t)j * I, a, I);
    free(a);
    return 0;
}

/* LoRE residual Delta_e(h) = B_e A_e h (Sec. 4.2), A: [r,d], B: [d,r]. */
int oracle_lore_delta(int d, int r, const float *A, const float *B, const float *x, double *out) {
    double *z = (double *)malloc(sizeof(double) * (size_t)r);
    if (!z) return -1;
    for (int q = 0; q < r; ++q) z[q] = dot_fd(A + (size_t)q * d, x, d);
#pragma omp parallel for schedule(static)
    for (int j = 0; j < d; ++j) out[j] = dot_fdd(B + (size_t)j * r, z, r);
    free(z);
    return 0;
}

/*
 * One layer call.
 *
 * Routing, classification and the residual-miss list are produced for all T tokens.
 * The expensive part (expert evaluation) is done for the n_sel tokens listed in sel[]
 * (sel == NULL means all tokens, n_sel is then ignored); y and y_full have one row per
 * listed token, in list order.
 *
 *   y_t      = s_t + sum_{k:HIT} g_k E_{e_k}(h_t) + sum_{k:LOWCONF} g_k ( s_t + B_{e_k} A_{e_k} h_t )
 *   y_full_t = y_t + sum_{k:MISS_EXACT} g_k E_{e_k}(h_t)            (what exact recovery adds later)
 *
 * w_gate/w_up/w_down are tables of N pointers; an entry may be NULL when that expert is
 * never evaluated.  Returns 0, or -(e+1) if expert e was needed but its pointer is NULL,
 * or -1000 on allocation failure.  y_full may be NULL (then MISS_EXACT experts are not needed).
 */
int oracle_layer(const oracle_cfg *cfg, int T, const float *h, const float *w_router,
                 const float *const *w_gate, const float *const *w_up, const float *const *w_down,
                 const float *s_gate, const float *s_up, const float *s_down,
                 const float *lore_A, const float *lore_B,
                 const uint8_t *resident, const float *conf,
                 int n_sel, const int32_t *sel,
                 double *logits, int32_t *idx, double *gate, uint8_t *cls, int32_t *counts,
                 int32_t *n_resid, int32_t *resid_tok, int32_t *resid_k, int32_t *resid_expert,
                 double *resid_gate, double *y, double *y_full) {
    const int d = cfg->d, N = cfg->n_experts, K = cfg->top_k, I = cfg->inter, Is = cfg->inter_shared,
              r = cfg->lore_rank;
    oracle_router_logits(T, d, N, h, w_router, logits);
    oracle_topk_gates(T, N, K, cfg->norm_topk, logits, idx, gate);
    oracle_classify(T, N, K, idx, resident, conf, cfg->conf_stride, cfg->tau, cls, counts);

    /* residual-miss set M (Sec. 4.3), listed in (t,k) order */
    int nr = 0;
    for (int t = 0; t < T; ++t)
        for (int k = 0; k < K; ++k)
            if (cls[(size_t)t * K + k] == ORACLE_MISS_EXACT) {
                resid_tok[nr] = t;
                resid_k[nr] = k;
                resid_expert[nr] = idx[(size_t)t * K + k];
                resid_gate[nr] = gate[(size_t)t * K + k];
                ++nr;
            }
    *n_resid = nr;

    int rows = sel ? n_sel : T;
    double *s = (double *)malloc(sizeof(double) * (size_t)d);
    double *o = (double *)malloc(sizeof(double) * (size_t)d);
    if (!s || !o) { free(s); free(o); return -1000; }
    int rc = 0;
    for (int row = 0; row < rows && rc == 0; ++row) {
        int t = sel ? sel[row] : row;
        const float *x = h + (size_t)t * d;
        double *yt = y + (size_t)row * d;
        double *yf = y_full ? y_full + (size_t)row * d : NULL;
        if (oracle_swiglu_ffn(d, Is, s_gate, s_up, s_down, x, s)) { rc = -1000; break; }
        for (int j = 0; j < d; ++j) yt[j] = s[j];           /* shared expert: always on */
        if (yf) for (int j = 0; j < d; ++j) yf[j] = 0.0;     /* exact-recovery part, added at the end */
        for (int k = 0; k < K; ++k) {
            int e = idx[(size_t)t * K + k];
            double g = gate[(size_t)t * K + k];
            uint8_t c = cls[(size_t)t * K + k];
            if (c == ORACLE_HIT || (c == ORACLE_MISS_EXACT && yf)) {
                if (!w_gate[e] || !w_up[e] || !w_down[e]) { rc = -(e + 1); break; }
                if (oracle_swiglu_ffn(d, I, w_gate[e], w_up[e], w_down[e], x, o)) { rc = -1000; break; }
                if (c == ORACLE_HIT) for (int j = 0; j < d; ++j) yt[j] += g * o[j];
                else                 for (int j = 0; j < d; ++j) yf[j] += g * o[j];
            } else if (c == ORACLE_LOWCONF) {
                if (oracle_lore_delta(d, r, lore_A + (size_t)e * r * d, lore_B + (size_t)e * d * r, x, o)) { rc = -1000; break; }
                for (int j = 0; j < d; ++j) yt[j] += g * (s[j] + o[j]);   /* y~_e = S(h) + B A h */
            }
        }
        if (yf && rc == 0) for (int j = 0; j < d; ++j) yf[j] += yt[j];
    }
    free(s);
    free(o);
    return rc;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
