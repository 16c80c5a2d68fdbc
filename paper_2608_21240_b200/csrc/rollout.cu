// Speculative prefetch rollout (Algorithm 1 of the paper, Sec. 4.1) on the device, for a batch of tokens.
// For depth l = 1 .. l_max, while a token still speculates:
//     pi^(l)  = router^(l)(h^(l-1)),  S^(l) = TopK(pi^(l), K)  -> enqueued,  C^(l) = sum_{i in S^(l)} pi^(l)_i
//     if l >= l_min and C^(l) < tau: the token stops (its current prediction is kept)
//     h^(l)   = Attn^(l)(h^(l-1)) + sum_{i in S^(l)} pi^(l)_i E~_i(h^(l-1)),   E~_i = S^(l) + B_i A_i
// Readings: Attn^(l) is not specified for a single state and is taken as the identity; the state is held in bf16
// between depths.  With these, a depth is the draft-confidence call followed by the LoRE-surrogate path of the layer
// call with every selected expert treated as a low-confidence miss, gates pi^(l)_i, and the shared expert weighted by
// C^(l) alone (the layer's own "1 +" term does not occur in the projection): the general-shape kernels are reused.
#include "spice_internal.cuh"

namespace spice {

// One thread per token: records the depth's prediction, applies the halting rule, and writes the classes that steer
// the projection (all LOWCONF for a token that continues, all MISS_EXACT -- i.e. nothing is added -- otherwise).
__global__ void __launch_bounds__(256) rollout_mask_kernel(int T, int K, int depth, int l_min, int l_max, float tau,
                                                           const float *__restrict__ conf_l, int32_t *__restrict__ active,
                                                           const int32_t *__restrict__ idx_ws, int32_t *__restrict__ idx_out,
                                                           float *__restrict__ conf_out, uint8_t *__restrict__ cls,
                                                           int32_t *__restrict__ depth_out) {
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= T) return;
    const bool on = depth == 1 ? true : active[t] != 0;
    bool cont = false;
    if (on) {
        const float c = conf_l[t];
        depth_out[t] = depth;
        conf_out[t] = c;
        cont = !(depth >= l_min && c < tau) && depth < l_max;   // (the last depth needs no further state)
        for (int k = 0; k < K; ++k) idx_out[(size_t)t * K + k] = idx_ws[(size_t)t * K + k];
        active[t] = (depth >= l_min && c < tau) ? 0 : 1;
    } else {
        conf_out[t] = 0.f;
        for (int k = 0; k < K; ++k) idx_out[(size_t)t * K + k] = -1;
        if (depth == 1) depth_out[t] = 0;
    }
    for (int k = 0; k < K; ++k) cls[(size_t)t * K + k] = cont ? SPICE_LOWCONF : SPICE_MISS_EXACT;
}

// Eq. 3: union of the predicted sets over the batch, per depth: mask[l, e] = 1 iff some token predicts expert e at depth l+1
__global__ void __launch_bounds__(256) prefetch_set_kernel(const int32_t *__restrict__ idx_hat, size_t per_depth, int n_depths, int N,
                                                           uint8_t *__restrict__ mask) {
    const size_t i = (size_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= per_depth * n_depths) return;
    const int e = idx_hat[i];
    if (e >= 0 && e < N) mask[(i / per_depth) * N + e] = 1;
}

int launch_prefetch_set(const Dims &dm, int l_max, const int32_t *idx_hat, uint8_t *mask, cudaStream_t st) {
    if (cudaMemsetAsync(mask, 0, (size_t)l_max * dm.N, st) != cudaSuccess) return -1;
    const size_t per_depth = (size_t)dm.T * dm.K, total = per_depth * l_max;
    prefetch_set_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(idx_hat, per_depth, l_max, dm.N, mask);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_rollout_mask(const Dims &dm, int depth, int l_min, int l_max, float tau, const float *conf_l, int32_t *active,
                        const int32_t *idx_ws, int32_t *idx_out, float *conf_out, uint8_t *cls, int32_t *depth_out,
                        cudaStream_t st) {
    rollout_mask_kernel<<<(dm.T + 255) / 256, 256, 0, st>>>(dm.T, dm.K, depth, l_min, l_max, tau, conf_l, active, idx_ws, idx_out,
                                                           conf_out, cls, depth_out);
    return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_rollout(const Dims &dm, const spice_layer_weights *w, int l_min, int l_max, float tau, __nv_bfloat16 *h_state,
                   __nv_bfloat16 *y_scratch, int32_t *idx_ws, float *gate_ws, uint8_t *cls_ws, float *conf_ws, float *logits_ws,
                   int32_t *active_ws, const Tables &tb, int32_t *idx_hat, float *conf, int32_t *depth, cudaStream_t st) {
    int launches = 0;
    const size_t n = (size_t)dm.T * dm.K;
    for (int l = 1; l <= l_max; ++l) {
        const spice_layer_weights &wl = w[l - 1];
        int k = launch_draft_confidence(dm, h_state, reinterpret_cast<const __nv_bfloat16 *>(wl.w_router), idx_ws, gate_ws,
                                        logits_ws, nullptr, conf_ws, st);
        if (k < 0) return -1;
        launches += k;
        rollout_mask_kernel<<<(dm.T + 255) / 256, 256, 0, st>>>(dm.T, dm.K, l, l_min, l_max, tau, conf_ws, active_ws, idx_ws,
                                                               idx_hat + (size_t)(l - 1) * n, conf + (size_t)(l - 1) * dm.T,
                                                               cls_ws, depth);
        if (cudaGetLastError() != cudaSuccess) return -1;
        ++launches;
        if (l == l_max) break;
        // projection of the tokens that continue: h += C S(h) + sum_k pi_k B_k A_k h
        if ((k = launch_group(dm, idx_ws, gate_ws, cls_ws, nullptr, tb, st)) < 0) return -1;
        launches += k;
        if ((k = launch_gateup(dm, KIND_SHARED, wl, h_state, tb, st)) < 0) return -1;
        launches += k;
        if ((k = launch_lore_a(dm, wl, h_state, tb, st)) < 0) return -1;
        launches += k;
        if ((k = launch_down(dm, KIND_SHARED | KIND_LOW, wl, tb, st)) < 0) return -1;
        launches += k;
        CombineArgs ca{KIND_SHARED | KIND_LOW, 0, gate_ws, cls_ws, nullptr, y_scratch, nullptr, h_state, /*shared_coef_low_sum=*/1};
        if ((k = launch_combine(dm, ca, tb, st)) < 0) return -1;
        launches += k;
    }
    return launches;
}

}  // namespace spice
