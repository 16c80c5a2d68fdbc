"""Thin ctypes binding of libspice.so: argument marshalling only.

Every function named spice_* forwards to the C entry point of the same name (include/spice.h)
with torch tensors turned into device pointers; nothing of the layer is computed in Python.
`SpiceLayer` bundles a context with output allocation for convenience.  torch is used for
device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SPICE_LIB") or os.path.join(_PKG, "libspice.so")   # SPICE_LIB: an instrumented or older build

SPICE_OK = 0
HIT, MISS_EXACT, LOWCONF = 0, 1, 2


class SpiceError(RuntimeError):
    pass


class LayerCfg(C.Structure):
    """Mirror of spice_layer_cfg."""
    _fields_ = [("d", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32), ("inter", C.c_int32),
                ("inter_shared", C.c_int32), ("lore_rank", C.c_int32), ("n_slots", C.c_int32),
                ("norm_topk", C.c_int32), ("conf_stride", C.c_int32), ("tau", C.c_float)]


class LayerWeightsC(C.Structure):
    """Mirror of spice_layer_weights (device pointers)."""
    _fields_ = [("w_router", C.c_void_p), ("slot_w_gate_up", C.c_void_p), ("slot_w_down", C.c_void_p),
                ("slot_of_expert", C.c_void_p), ("shared_w_gate_up", C.c_void_p), ("shared_w_down", C.c_void_p),
                ("lore_A", C.c_void_p), ("lore_B", C.c_void_p)]


class LayerWeightsFp8C(C.Structure):
    """Mirror of spice_layer_weights_fp8 (device pointers)."""
    _fields_ = [("w_router", C.c_void_p), ("slot_q_gate_up", C.c_void_p), ("slot_s_gate_up", C.c_void_p),
                ("slot_q_down", C.c_void_p), ("slot_s_down", C.c_void_p), ("slot_of_expert", C.c_void_p),
                ("shared_q_gate_up", C.c_void_p), ("shared_s_gate_up", C.c_void_p), ("shared_q_down", C.c_void_p),
                ("shared_s_down", C.c_void_p), ("lore_A", C.c_void_p), ("lore_B", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Load libspice.so.  Raises if it has not been built: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SpiceError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_21240_b200.build` "
                             "(needs nvcc); the library has no CPU or PyTorch fallback")
        L = C.CDLL(LIB_PATH)
        L.spice_status_string.restype = C.c_char_p
        L.spice_version.restype = C.c_int32
        for name in ("spice_create", "spice_destroy", "spice_workspace_bytes", "spice_route_topk",
                     "spice_classify_misses", "spice_grouped_expert_ffn", "spice_lore_surrogate",
                     "spice_moe_layer_fwd", "spice_get_device_status", "spice_launch_count", "spice_set_option",
                     "spice_grouped_expert_ffn_static", "spice_draft_confidence", "spice_prefetch_rollout",
                     "spice_quantize_e4m3_rows", "spice_moe_layer_fwd_fp8"):
            getattr(L, name).restype = C.c_int
        L.spice_static_scratch_bytes.restype = C.c_size_t
        L.spice_lore_calibrate.restype = C.c_int
        L.spice_lore_calibrate_workspace_bytes.restype = C.c_size_t
        _lib = L
    return _lib


def _check(code: int, what: str) -> None:
    if code != SPICE_OK:
        raise SpiceError(f"{what}: {lib().spice_status_string(code).decode()} (status {code})")


def _ptr(t: Optional[torch.Tensor], dtype=None) -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    # (pinned host memory is device-accessible under unified addressing: a caller may let the kernels write small
    # results straight into it instead of copying them back)
    if not (t.is_cuda or t.is_pinned()) or not t.is_contiguous():
        raise SpiceError("tensors passed to libspice must be contiguous CUDA tensors (or pinned host tensors)")
    if dtype is not None and t.dtype != dtype:
        raise SpiceError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


# ------------------------------------------------------------------ C entry points, same names
def spice_create(cfg: LayerCfg, max_tokens: int, device: int = 0) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(lib().spice_create(C.byref(ctx), C.c_int32(device), C.byref(cfg), C.c_int32(max_tokens)), "spice_create")
    return ctx


def spice_destroy(ctx) -> None:
    _check(lib().spice_destroy(ctx), "spice_destroy")


def spice_workspace_bytes(ctx) -> int:
    n = C.c_size_t()
    _check(lib().spice_workspace_bytes(ctx, C.byref(n)), "spice_workspace_bytes")
    return n.value


def spice_launch_count(ctx) -> int:
    n = C.c_int64()
    _check(lib().spice_launch_count(ctx, C.byref(n)), "spice_launch_count")
    return n.value


OPT_PATH, OPT_SPIN_LIMIT, OPT_TC_WAIT_LIMIT = 0, 1, 2


def spice_set_option(ctx, option: int, value: int) -> None:
    _check(lib().spice_set_option(ctx, C.c_int32(option), C.c_int64(value)), "spice_set_option")


def spice_get_device_status(ctx) -> int:
    v = C.c_int32()
    _check(lib().spice_get_device_status(ctx, C.byref(v)), "spice_get_device_status")
    return v.value


def spice_route_topk(ctx, h, w_router, T, idx, gate, logits=None, stream=None) -> None:
    _check(lib().spice_route_topk(ctx, _ptr(h, torch.bfloat16), _ptr(w_router, torch.bfloat16), C.c_int32(T),
                                  _ptr(idx, torch.int32), _ptr(gate, torch.float32), _ptr(logits, torch.float32),
                                  _stream(stream)), "spice_route_topk")


def spice_draft_confidence(ctx, h_hat, w_draft_router, T, idx_hat, conf, pi_hat=None, stream=None) -> None:
    _check(lib().spice_draft_confidence(ctx, _ptr(h_hat, torch.bfloat16), _ptr(w_draft_router, torch.bfloat16), C.c_int32(T),
                                        _ptr(idx_hat, torch.int32), _ptr(pi_hat, torch.float32), _ptr(conf, torch.float32),
                                        _stream(stream)), "spice_draft_confidence")


def spice_min_lookahead_depth(n_prefetch, expert_bytes, pcie_bytes_per_s, t_comp_s) -> int:
    f = lib().spice_min_lookahead_depth
    f.restype = C.c_int32
    return int(f(C.c_int32(n_prefetch), C.c_double(expert_bytes), C.c_double(pcie_bytes_per_s), C.c_double(t_comp_s)))


def spice_prefetch_rollout(ctx, weights, x_current, T, l_min, l_max, tau, idx_hat, conf, depth, h_final=None,
                           prefetch_mask=None, stream=None) -> None:
    """weights: sequence of l_max LayerWeightsC structs (depth 1 first)."""
    arr = (LayerWeightsC * l_max)(*weights)
    _check(lib().spice_prefetch_rollout(ctx, arr, _ptr(x_current, torch.bfloat16), C.c_int32(T), C.c_int32(l_min),
                                        C.c_int32(l_max), C.c_float(tau), _ptr(idx_hat, torch.int32),
                                        _ptr(conf, torch.float32), _ptr(depth, torch.int32), _ptr(h_final, torch.bfloat16),
                                        _ptr(prefetch_mask, torch.uint8), _stream(stream)), "spice_prefetch_rollout")


def spice_lore_calibrate(h_cal, resid, rank, ridge=0.0, iterations=100, stream=None):
    """Fit the LoRE factors of one expert on the device.  h_cal [n,d] bf16, resid [n,d] fp32 (device tensors).
    Returns (A [rank,d] bf16, B [d,rank] bf16, loss tensor [2] = (objective, sum resid^2), status tensor [1])."""
    n, d = h_cal.shape
    dev = h_cal.device
    nbytes = int(lib().spice_lore_calibrate_workspace_bytes(C.c_int32(d), C.c_int32(n), C.c_int32(rank)))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    A = torch.empty(rank, d, dtype=torch.bfloat16, device=dev)
    Bm = torch.empty(d, rank, dtype=torch.bfloat16, device=dev)
    loss = torch.empty(2, dtype=torch.float32, device=dev)
    status = torch.empty(1, dtype=torch.int32, device=dev)
    with torch.cuda.device(dev):
        _check(lib().spice_lore_calibrate(C.c_int32(d), C.c_int32(n), C.c_int32(rank), C.c_float(ridge), C.c_int32(iterations),
                                          _ptr(h_cal, torch.bfloat16), _ptr(resid, torch.float32), _ptr(A, torch.bfloat16),
                                          _ptr(Bm, torch.bfloat16), _ptr(loss, torch.float32), _ptr(status, torch.int32),
                                          C.c_void_p(ws.data_ptr()), C.c_size_t(nbytes), _stream(stream)),
               "spice_lore_calibrate")
    return A, Bm, loss, status


def spice_classify_misses(ctx, idx, gate, slot_of_expert, conf, T, cls, slot, counts, resid_tok=None, resid_k=None,
                          resid_expert=None, resid_gate=None, stream=None) -> None:
    _check(lib().spice_classify_misses(ctx, _ptr(idx, torch.int32), _ptr(gate, torch.float32),
                                       _ptr(slot_of_expert, torch.int32), _ptr(conf, torch.float32), C.c_int32(T),
                                       _ptr(cls, torch.uint8), _ptr(slot, torch.int32), _ptr(counts, torch.int32),
                                       _ptr(resid_tok, torch.int32), _ptr(resid_k, torch.int32),
                                       _ptr(resid_expert, torch.int32), _ptr(resid_gate, torch.float32),
                                       _stream(stream)), "spice_classify_misses")


def spice_grouped_expert_ffn(ctx, weights: LayerWeightsC, h, idx, gate, cls, slot, T, y, stream=None) -> None:
    _check(lib().spice_grouped_expert_ffn(ctx, C.byref(weights), _ptr(h, torch.bfloat16), _ptr(idx, torch.int32),
                                          _ptr(gate, torch.float32), _ptr(cls, torch.uint8), _ptr(slot, torch.int32),
                                          C.c_int32(T), _ptr(y, torch.float32), _stream(stream)),
           "spice_grouped_expert_ffn")


def spice_grouped_expert_ffn_static(cfg: LayerCfg, weights: LayerWeightsC, h, idx, gate, cls, slot, T, y,
                                    device_status=None, stream=None) -> None:
    """The resident-expert FFN without a ctx and without any allocation (for hosts that may not call
    cudaMalloc): scratch lives in a fixed 8 MiB device array inside the library.  Calls on one GPU must
    not overlap; the first call on a GPU should precede any stream capture."""
    _check(lib().spice_grouped_expert_ffn_static(C.byref(cfg), C.byref(weights), _ptr(h, torch.bfloat16),
                                                 _ptr(idx, torch.int32), _ptr(gate, torch.float32),
                                                 _ptr(cls, torch.uint8), _ptr(slot, torch.int32), C.c_int32(T),
                                                 _ptr(y, torch.float32), _ptr(device_status, torch.int32),
                                                 _stream(stream)), "spice_grouped_expert_ffn_static")


def spice_static_scratch_bytes() -> int:
    return int(lib().spice_static_scratch_bytes())


def spice_lore_surrogate(ctx, weights: LayerWeightsC, h, idx, gate, cls, T, y, stream=None) -> None:
    _check(lib().spice_lore_surrogate(ctx, C.byref(weights), _ptr(h, torch.bfloat16), _ptr(idx, torch.int32),
                                      _ptr(gate, torch.float32), _ptr(cls, torch.uint8), C.c_int32(T),
                                      _ptr(y, torch.float32), _stream(stream)), "spice_lore_surrogate")


def spice_moe_layer_fwd(ctx, weights: LayerWeightsC, h, conf, T, y, y_cpu_residual=None, x_resid=None, idx=None,
                        gate=None, cls=None, counts=None, resid_tok=None, resid_k=None, resid_expert=None,
                        resid_gate=None, stream=None) -> None:
    _check(lib().spice_moe_layer_fwd(ctx, C.byref(weights), _ptr(h, torch.bfloat16), _ptr(conf, torch.float32),
                                     C.c_int32(T), _ptr(y_cpu_residual, torch.float32),
                                     _ptr(x_resid, torch.bfloat16), _ptr(y, torch.bfloat16), _ptr(idx, torch.int32),
                                     _ptr(gate, torch.float32), _ptr(cls, torch.uint8), _ptr(counts, torch.int32),
                                     _ptr(resid_tok, torch.int32), _ptr(resid_k, torch.int32),
                                     _ptr(resid_expert, torch.int32), _ptr(resid_gate, torch.float32),
                                     _stream(stream)), "spice_moe_layer_fwd")


def spice_quantize_e4m3_rows(w, q, scale, stream=None) -> None:
    """w [..., cols] bf16 -> q (uint8, same shape) and scale (fp32, shape without the last axis): E4M3 codes with one
    power-of-two scale per row."""
    cols = w.shape[-1]
    rows = w.numel() // cols
    with torch.cuda.device(w.device):
        _check(lib().spice_quantize_e4m3_rows(_ptr(w, torch.bfloat16), C.c_int64(rows), C.c_int32(cols), _ptr(q, torch.uint8),
                                              _ptr(scale, torch.float32), _stream(stream)), "spice_quantize_e4m3_rows")


def spice_moe_layer_fwd_fp8(ctx, weights: "LayerWeightsFp8C", h, conf, T, y, y_cpu_residual=None, x_resid=None, idx=None,
                            gate=None, cls=None, counts=None, resid_tok=None, resid_k=None, resid_expert=None,
                            resid_gate=None, stream=None) -> None:
    _check(lib().spice_moe_layer_fwd_fp8(ctx, C.byref(weights), _ptr(h, torch.bfloat16), _ptr(conf, torch.float32),
                                         C.c_int32(T), _ptr(y_cpu_residual, torch.float32),
                                         _ptr(x_resid, torch.bfloat16), _ptr(y, torch.bfloat16), _ptr(idx, torch.int32),
                                         _ptr(gate, torch.float32), _ptr(cls, torch.uint8), _ptr(counts, torch.int32),
                                         _ptr(resid_tok, torch.int32), _ptr(resid_k, torch.int32),
                                         _ptr(resid_expert, torch.int32), _ptr(resid_gate, torch.float32),
                                         _stream(stream)), "spice_moe_layer_fwd_fp8")


# ------------------------------------------------------------------ convenience wrappers
@dataclass
class LayerWeights:
    """Device tensors of one layer (bf16 unless noted); see spice_layer_weights."""
    w_router: torch.Tensor          # [N,d]
    slot_w_gate_up: torch.Tensor    # [S,2I,d]
    slot_w_down: torch.Tensor       # [S,d,I]
    slot_of_expert: torch.Tensor    # [N] int32
    shared_w_gate_up: torch.Tensor  # [2Is,d]
    shared_w_down: torch.Tensor     # [d,Is]
    lore_A: torch.Tensor            # [N,r,d]
    lore_B: torch.Tensor            # [N,d,r]

    def c_struct(self) -> LayerWeightsC:
        return LayerWeightsC(_ptr(self.w_router, torch.bfloat16), _ptr(self.slot_w_gate_up, torch.bfloat16),
                             _ptr(self.slot_w_down, torch.bfloat16), _ptr(self.slot_of_expert, torch.int32),
                             _ptr(self.shared_w_gate_up, torch.bfloat16), _ptr(self.shared_w_down, torch.bfloat16),
                             _ptr(self.lore_A, torch.bfloat16), _ptr(self.lore_B, torch.bfloat16))


@dataclass
class LayerWeightsFp8:
    """Device tensors of one layer at the 8-bit weight precision; see spice_layer_weights_fp8."""
    w_router: torch.Tensor          # [N,d] bf16
    slot_q_gate_up: torch.Tensor    # [S,2I,d] uint8 (E4M3)
    slot_s_gate_up: torch.Tensor    # [S,2I] fp32
    slot_q_down: torch.Tensor       # [S,d,I] uint8
    slot_s_down: torch.Tensor       # [S,d] fp32
    slot_of_expert: torch.Tensor    # [N] int32
    shared_q_gate_up: torch.Tensor  # [2Is,d] uint8
    shared_s_gate_up: torch.Tensor  # [2Is] fp32
    shared_q_down: torch.Tensor     # [d,Is] uint8
    shared_s_down: torch.Tensor     # [d] fp32
    lore_A: torch.Tensor            # [N,r,d] bf16
    lore_B: torch.Tensor            # [N,d,r] bf16

    def c_struct(self) -> LayerWeightsFp8C:
        u8, f32, bf = torch.uint8, torch.float32, torch.bfloat16
        return LayerWeightsFp8C(_ptr(self.w_router, bf), _ptr(self.slot_q_gate_up, u8), _ptr(self.slot_s_gate_up, f32),
                                _ptr(self.slot_q_down, u8), _ptr(self.slot_s_down, f32), _ptr(self.slot_of_expert, torch.int32),
                                _ptr(self.shared_q_gate_up, u8), _ptr(self.shared_s_gate_up, f32),
                                _ptr(self.shared_q_down, u8), _ptr(self.shared_s_down, f32), _ptr(self.lore_A, bf),
                                _ptr(self.lore_B, bf))


def quantize_layer(w: "LayerWeights") -> LayerWeightsFp8:
    """The 8-bit form of a bf16 weight set: four calls of spice_quantize_e4m3_rows (allocation of the outputs only)."""
    def qz(t):
        q = torch.empty(t.shape, dtype=torch.uint8, device=t.device)
        s = torch.empty(t.shape[:-1], dtype=torch.float32, device=t.device)
        spice_quantize_e4m3_rows(t, q, s)
        return q, s
    sgu, ssgu = qz(w.slot_w_gate_up)
    sd, ssd = qz(w.slot_w_down)
    hgu, shgu = qz(w.shared_w_gate_up)
    hd, shd = qz(w.shared_w_down)
    return LayerWeightsFp8(w.w_router, sgu, ssgu, sd, ssd, w.slot_of_expert, hgu, shgu, hd, shd, w.lore_A, w.lore_B)


@dataclass
class LayerOutputs:
    y: torch.Tensor
    idx: torch.Tensor
    gate: torch.Tensor
    cls: torch.Tensor
    counts: torch.Tensor
    resid_tok: torch.Tensor
    resid_k: torch.Tensor
    resid_expert: torch.Tensor
    resid_gate: torch.Tensor


def make_cfg(d, n_experts, top_k, inter, inter_shared, lore_rank, n_slots, tau, norm_topk=1, conf_per_expert=True):
    return LayerCfg(d, n_experts, top_k, inter, inter_shared, lore_rank, n_slots, norm_topk,
                    n_experts if conf_per_expert else 0, tau)


class SpiceLayer:
    """A spice_ctx plus output buffers; every method is one C call."""

    def __init__(self, cfg: LayerCfg, max_tokens: int, device: int = 0):
        self.cfg, self.max_tokens, self.device = cfg, max_tokens, device
        torch.cuda.set_device(device)
        self.ctx = spice_create(cfg, max_tokens, device)
        self.dev = torch.device("cuda", device)

    def close(self):
        if self.ctx is not None:
            spice_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _empty(self, shape, dtype):
        return torch.empty(shape, dtype=dtype, device=self.dev)

    def route_topk(self, h, w_router, want_logits=False, stream=None):
        T, K, N = h.shape[0], self.cfg.top_k, self.cfg.n_experts
        idx, gate = self._empty((T, K), torch.int32), self._empty((T, K), torch.float32)
        logits = self._empty((T, N), torch.float32) if want_logits else None
        spice_route_topk(self.ctx, h, w_router, T, idx, gate, logits, stream)
        return (idx, gate, logits) if want_logits else (idx, gate)

    def draft_confidence(self, h_hat, w_draft_router, want_pi=False, stream=None):
        T, K, N = h_hat.shape[0], self.cfg.top_k, self.cfg.n_experts
        idx, conf = self._empty((T, K), torch.int32), self._empty((T,), torch.float32)
        pi = self._empty((T, N), torch.float32) if want_pi else None
        spice_draft_confidence(self.ctx, h_hat, w_draft_router, T, idx, conf, pi, stream)
        return (idx, conf, pi) if want_pi else (idx, conf)

    def prefetch_rollout(self, weights, x_current, l_min, l_max, tau, stream=None):
        """weights: list of l_max LayerWeights (depth 1 first).  Returns (idx_hat, conf, depth, h_final)."""
        T, K = x_current.shape[0], self.cfg.top_k
        idx = self._empty((l_max, T, K), torch.int32)
        conf = self._empty((l_max, T), torch.float32)
        depth = self._empty((T,), torch.int32)
        h_final = self._empty((T, self.cfg.d), torch.bfloat16)
        self.prefetch_mask = self._empty((l_max, self.cfg.n_experts), torch.uint8)
        spice_prefetch_rollout(self.ctx, [w.c_struct() for w in weights], x_current, T, l_min, l_max, tau, idx, conf,
                               depth, h_final, self.prefetch_mask, stream)
        return idx, conf, depth, h_final

    def classify_misses(self, idx, gate, slot_of_expert, conf, stream=None):
        T, K = idx.shape
        cls, slot = self._empty((T, K), torch.uint8), self._empty((T, K), torch.int32)
        counts = torch.zeros(3, dtype=torch.int32, device=self.dev)
        n = max(T * K, 1)
        rt, rk, re_ = (self._empty((n,), torch.int32) for _ in range(3))
        rg = self._empty((n,), torch.float32)
        spice_classify_misses(self.ctx, idx, gate, slot_of_expert, conf, T, cls, slot, counts, rt, rk, re_, rg, stream)
        return cls, slot, counts, (rt, rk, re_, rg)

    def grouped_expert_ffn(self, w: LayerWeights, h, idx, gate, cls, slot, y, stream=None):
        spice_grouped_expert_ffn(self.ctx, w.c_struct(), h, idx, gate, cls, slot, h.shape[0], y, stream)
        return y

    def lore_surrogate(self, w: LayerWeights, h, idx, gate, cls, y, stream=None):
        spice_lore_surrogate(self.ctx, w.c_struct(), h, idx, gate, cls, h.shape[0], y, stream)
        return y

    def moe_layer_fwd(self, w: LayerWeights, h, conf, y_cpu_residual=None, x_resid=None, stream=None) -> LayerOutputs:
        T, K, d = h.shape[0], self.cfg.top_k, self.cfg.d
        n = max(T * K, 1)
        o = LayerOutputs(self._empty((T, d), torch.bfloat16), self._empty((T, K), torch.int32),
                         self._empty((T, K), torch.float32), self._empty((T, K), torch.uint8),
                         torch.zeros(3, dtype=torch.int32, device=self.dev), self._empty((n,), torch.int32),
                         self._empty((n,), torch.int32), self._empty((n,), torch.int32),
                         self._empty((n,), torch.float32))
        spice_moe_layer_fwd(self.ctx, w.c_struct(), h, conf, T, o.y, y_cpu_residual, x_resid, o.idx, o.gate, o.cls,
                            o.counts, o.resid_tok, o.resid_k, o.resid_expert, o.resid_gate, stream)
        return o

    def moe_layer_fwd_fp8(self, w: LayerWeightsFp8, h, conf, y_cpu_residual=None, x_resid=None, stream=None) -> LayerOutputs:
        T, K, d = h.shape[0], self.cfg.top_k, self.cfg.d
        n = max(T * K, 1)
        o = LayerOutputs(self._empty((T, d), torch.bfloat16), self._empty((T, K), torch.int32),
                         self._empty((T, K), torch.float32), self._empty((T, K), torch.uint8),
                         torch.zeros(3, dtype=torch.int32, device=self.dev), self._empty((n,), torch.int32),
                         self._empty((n,), torch.int32), self._empty((n,), torch.int32),
                         self._empty((n,), torch.float32))
        spice_moe_layer_fwd_fp8(self.ctx, w.c_struct(), h, conf, T, o.y, y_cpu_residual, x_resid, o.idx, o.gate, o.cls,
                                o.counts, o.resid_tok, o.resid_k, o.resid_expert, o.resid_gate, stream)
        return o

    def set_option(self, option: int, value: int) -> None:
        spice_set_option(self.ctx, option, value)

    def device_status(self) -> int:
        return spice_get_device_status(self.ctx)

    def launch_count(self) -> int:
        return spice_launch_count(self.ctx)


# ------------------------------------------------------------------ workload marshalling
def bf16_tensor(x_f32, dev="cuda") -> torch.Tensor:
    """fp32 numpy array holding bf16-representable values -> bf16 device tensor (bit exact)."""
    import numpy as np
    from . import workloads as W
    bits = W.bf16_bits(x_f32)
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)


def bits_tensor(bits, dev="cuda") -> torch.Tensor:
    import numpy as np
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)


def cfg_of(s, tau=None, norm_topk=None, conf_per_expert=True) -> LayerCfg:
    """spice_layer_cfg of a workloads.LayerShape."""
    return make_cfg(s.d, s.n_experts, s.top_k, s.inter, s.inter_shared, s.lore_rank, s.n_slots,
                    s.tau if tau is None else tau, s.norm_topk if norm_topk is None else norm_topk, conf_per_expert)


def upload(wl, dev="cuda", only=None) -> LayerWeights:
    """Copy a workloads.LayerWorkload's weights to the device in the library's layout.

    only: experts whose slot contents matter (see LayerWorkload.slot_pool_bits)."""
    gu, dn = wl.slot_pool_bits(only)
    sg, su, sd = wl.shared()
    A, Bm = wl.lore()
    return LayerWeights(
        w_router=bf16_tensor(wl.w_router, dev),
        slot_w_gate_up=bits_tensor(gu, dev),
        slot_w_down=bits_tensor(dn, dev),
        slot_of_expert=torch.from_numpy(wl.slot_of_expert.copy()).to(dev),
        shared_w_gate_up=torch.cat([bf16_tensor(sg, dev), bf16_tensor(su, dev)], 0).contiguous(),
        shared_w_down=bf16_tensor(sd, dev),
        lore_A=bf16_tensor(A, dev),
        lore_B=bf16_tensor(Bm, dev),
    )
