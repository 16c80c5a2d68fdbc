// spice_grouped_expert_ffn_static: the resident-expert FFN for callers that may not allocate.
//
// Every other entry point needs a spice_ctx, and creating one calls cudaMalloc for the workspace.
// Some hosts cannot do that: a serving process that gives each component a fixed arena and refuses
// driver allocations once it is up, or a process whose memory limit is enforced by failing
// cudaMalloc.  For them this file keeps the kernels' scratch (group table, permutation, SwiGLU
// activations, un-gated down-projected rows) in one file-scope device array of fixed size, which
// every GPU that loads the library holds until the process exits.  The kernels are the library's
// general-shape kernels, unchanged; only the place their scratch lives differs.
#include <mutex>

#include "spice_internal.cuh"

using namespace spice;

namespace {

constexpr size_t STATIC_SCRATCH_BYTES = 8u << 20;   // 8 MiB per GPU
constexpr int MAX_DEVICES = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

std::mutex g_setup_mutex;
void *g_scratch_addr[MAX_DEVICES] = {};   // device address of g_static_scratch on each device, once known

// Device address of the scratch array on the CURRENT device; looked up once per device.
cudaError_t scratch_address(int device, void **out) {
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[device]) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return cudaSuccess;
}

struct Carver {
    char *base;
    size_t off = 0;
    template <typename T>
    T *take(size_t n) {
        off = (off + 255) & ~size_t(255);
        T *p = reinterpret_cast<T *>(base + off);
        off += n * sizeof(T);
        return p;
    }
};

// lays the tables of one call out in the scratch array; returns the bytes needed
size_t carve_tables(const spice_layer_cfg &g, int T, char *base, Tables *tb) {
    const size_t n = (size_t)T * g.top_k;
    Carver cv{base};
    Tables t{};
    t.status = cv.take<int32_t>(4);
    t.hdr = cv.take<int32_t>(HDR_WORDS);
    t.groups = cv.take<GroupDesc>(1 + (size_t)g.n_slots + g.n_experts);
    t.perm_hit = cv.take<int32_t>(n);
    t.perm_low = cv.take<int32_t>(n);
    t.pos_of_entry = cv.take<int32_t>(n);
    t.coef_shared = cv.take<float>(T);
    t.act_hit = cv.take<float>(n * g.inter);
    t.part = cv.take<float>(n * g.d);
    t.act_shared = nullptr;   // the shared / LoRE parts are not computed by this entry point
    t.z_low = nullptr;
    t.part_shared = nullptr;
    if (tb) *tb = t;
    return (cv.off + 255) & ~size_t(255);
}

}  // namespace

extern "C" spice_status spice_grouped_expert_ffn_static(const spice_layer_cfg *cfg, const spice_layer_weights *w,
                                                        const spice_bf16 *h, const int32_t *idx, const float *gate,
                                                        const uint8_t *cls, const int32_t *slot, int32_t T, float *y,
                                                        int32_t *device_status, void *stream) {
    if (!cfg || T < 0) return SPICE_ERR_INVALID_ARG;
    if (cfg->d < 8 || cfg->d % 8 || cfg->inter < 8 || cfg->inter % 8) return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (cfg->n_experts < 1 || cfg->n_experts > 1024 || cfg->n_slots < 1 || cfg->n_slots > 1024 || cfg->top_k < 1 ||
        cfg->top_k > 32 || cfg->top_k > cfg->n_experts)
        return SPICE_ERR_UNSUPPORTED_SHAPE;
    if (T == 0) return SPICE_OK;
    if (T > 65535) return SPICE_ERR_INVALID_ARG;
    // the fixed array is all there is: a call that does not fit is refused, nothing is launched
    if (carve_tables(*cfg, T, nullptr, nullptr) > STATIC_SCRATCH_BYTES) return SPICE_ERR_WORKSPACE;
    auto aligned16 = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; };
    if (!w || !w->slot_w_gate_up || !w->slot_w_down || !h || !idx || !gate || !cls || !slot || !y ||
        !aligned16(w->slot_w_gate_up) || !aligned16(w->slot_w_down) || !aligned16(h) || !aligned16(y))
        return SPICE_ERR_INVALID_ARG;
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= MAX_DEVICES) return SPICE_ERR_CUDA;
    void *base = nullptr;
    if (scratch_address(device, &base) != cudaSuccess) return SPICE_ERR_CUDA;
    Tables tb;
    carve_tables(*cfg, T, static_cast<char *>(base), &tb);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the sticky status word must start at zero
    // (every other table is fully rewritten for the entries this call uses)
    if (cudaMemsetAsync(tb.status, 0, 4 * sizeof(int32_t), st) != cudaSuccess) return SPICE_ERR_CUDA;
    const Dims dm{T, cfg->d, cfg->n_experts, cfg->top_k, cfg->inter, cfg->inter_shared, cfg->lore_rank, cfg->n_slots};
    const __nv_bfloat16 *hb = reinterpret_cast<const __nv_bfloat16 *>(h);
    if (launch_group(dm, idx, gate, cls, slot, tb, st) < 0) return SPICE_ERR_CUDA;
    if (launch_gateup(dm, KIND_HIT, *w, hb, tb, st) < 0) return SPICE_ERR_CUDA;
    if (launch_down(dm, KIND_HIT, *w, tb, st) < 0) return SPICE_ERR_CUDA;
    CombineArgs ca{KIND_HIT, 1, gate, cls, y, nullptr, nullptr, nullptr};
    if (launch_combine(dm, ca, tb, st) < 0) return SPICE_ERR_CUDA;
    if (device_status &&
        cudaMemcpyAsync(device_status, tb.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return SPICE_ERR_CUDA;
    return SPICE_OK;
}

extern "C" size_t spice_static_scratch_bytes(void) { return STATIC_SCRATCH_BYTES; }
