"""CPU oracle for the SPICE MoE-layer forward -- TEST INFRASTRUCTURE, not product code.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package.
It wraps `spice_oracle.c` (plain fp64 loops, see that file's header for the passages it
follows and the readings taken) through ctypes.  It imports nothing from the CUDA package.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spice_oracle.c")
_LIB = os.path.join(_HERE, "libspice_oracle.so")

HIT, MISS_EXACT, LOWCONF = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Cfg(C.Structure):
    _fields_ = [("d", C.c_int32), ("n_experts", C.c_int32), ("top_k", C.c_int32), ("inter", C.c_int32),
                ("inter_shared", C.c_int32), ("lore_rank", C.c_int32), ("norm_topk", C.c_int32),
                ("conf_stride", C.c_int32), ("tau", C.c_float)]


_lib = None


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_layer.restype = C.c_int
        _lib.oracle_swiglu_ffn.restype = C.c_int
        _lib.oracle_lore_delta.restype = C.c_int
        _lib.oracle_num_threads.restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


@dataclass
class LayerResult:
    logits: np.ndarray        # [T,N] f64
    idx: np.ndarray           # [T,K] i32, decreasing logit
    gate: np.ndarray          # [T,K] f64
    cls: np.ndarray           # [T,K] u8  (0 HIT, 1 MISS_EXACT, 2 LOWCONF)
    counts: np.ndarray        # [3] i32
    resid_tok: np.ndarray     # [n_resid] i32, (t,k) order
    resid_k: np.ndarray
    resid_expert: np.ndarray
    resid_gate: np.ndarray    # f64
    y: Optional[np.ndarray]        # [rows,d] f64 (GPU part of the layer output)
    y_full: Optional[np.ndarray]   # [rows,d] f64 (with the exact-recovery terms added)
    rows: np.ndarray          # token index of every row of y


def router_logits(h, w_router) -> np.ndarray:
    h, w = _f32(h), _f32(w_router)
    T, d = h.shape
    N = w.shape[0]
    out = np.empty((T, N), dtype=np.float64)
    _load().oracle_router_logits(C.c_int(T), C.c_int(d), C.c_int(N), _p(h), _p(w), _p(out))
    return out


def topk_gates(logits, K: int, norm_topk: int = 1):
    l = np.ascontiguousarray(logits, dtype=np.float64)
    T, N = l.shape
    idx = np.empty((T, K), dtype=np.int32)
    gate = np.empty((T, K), dtype=np.float64)
    _load().oracle_topk_gates(C.c_int(T), C.c_int(N), C.c_int(K), C.c_int(norm_topk), _p(l), _p(idx), _p(gate))
    return idx, gate


def draft_confidence(logits, K: int):
    """Sec. 4.1: pi_hat = softmax(logits), S_hat = TopK (Eq. 2), C = probability mass of S_hat (Eq. 5).
    Returns (idx_hat [T,K], pi_hat [T,N], conf [T])."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    T, N = l.shape
    idx = np.empty((T, K), dtype=np.int32)
    pi = np.empty((T, N), dtype=np.float64)
    conf = np.empty(T, dtype=np.float64)
    _load().oracle_draft_confidence(C.c_int(T), C.c_int(N), C.c_int(K), _p(l), _p(idx), _p(pi), _p(conf))
    return idx, pi, conf


def lore_calibrate(H, R, rank: int, ridge: float = 0.0):
    """LoRE calibration of one (layer, expert) pair (Sec. 4.2): the rank-r linear map Delta(h) = B A h that minimises
        sum_{h in D} || E(h) - S(h) - B A h ||_2^2
    over the calibration tokens, H [n,d] the hidden states and R [n,d] the residual targets E(h) - S(h).
    Written out as the closed-form minimiser (reduced-rank regression): the least-squares map W (R ~ H W), the fitted
    values H W, their r leading right singular vectors V; then B = V and A = (W V)^T.  With ridge > 0 the
    least-squares step is regularised: W = (H^T H + ridge * tr(H^T H)/d * I)^-1 H^T R.
    Returns (A [r,d], B [d,r], loss) in fp64; loss is the objective at (A, B)."""
    H = np.asarray(H, dtype=np.float64)
    R = np.asarray(R, dtype=np.float64)
    n, d = H.shape
    G = H.T @ H
    if ridge > 0.0:
        W = np.linalg.solve(G + ridge * np.trace(G) / d * np.eye(d), H.T @ R)
    else:
        W = np.linalg.lstsq(H, R, rcond=None)[0]
    fitted = H @ W
    _, _, Vt = np.linalg.svd(fitted, full_matrices=False)
    V = Vt[:rank].T
    B = V
    A = (W @ V).T
    loss = float(((R - (H @ A.T) @ B.T) ** 2).sum())
    return A, B, loss


def _round_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest bf16 (ties to even) of fp64 values, returned as fp64: the draft state is kept in bf16 between depths.
    A bf16 keeps 8 significant bits, so 45 of the 52 fraction bits of the fp64 pattern are dropped in ONE rounding
    (no detour over fp32, which would round twice).  Meant for finite values of normal bf16 magnitude (2^-126 .. 3.4e38);
    zeros keep their sign."""
    u = np.ascontiguousarray(x, dtype=np.float64).view(np.uint64)
    drop = np.uint64(45)
    half_minus_one = np.uint64((1 << 44) - 1)
    keep_mask = np.uint64(0xFFFFFFFFFFFFFFFF ^ ((1 << 45) - 1))
    r = (u + half_minus_one + ((u >> drop) & np.uint64(1))) & keep_mask
    return r.view(np.float64)


def prefetch_rollout(x, layers, top_k: int, l_min: int, l_max: int, tau: float):
    """Algorithm 1 (Sec. 4.1), per token, in the algorithm's own order and notation.

    x [T,d]: current hidden states.  layers[l-1] = dict(w_router, shared=(w_gate, w_up, w_down), lore_A, lore_B) of
    depth l.  For every depth l = 1..l_max while the token still speculates:
        pi^(l) = router^(l)(h^(l-1)); S^(l) = TopK(pi^(l), K); enqueue S^(l); C^(l) = sum_{i in S^(l)} pi^(l)_i;
        if l >= l_min and C^(l) < tau: stop (the current prediction is retained);
        h^(l) = Attn^(l)(h^(l-1)) + sum_{i in S^(l)} pi^(l)_i E~_i(h^(l-1)),  E~_i = S^(l) + B_i A_i.
    Readings: Attn^(l) is not specified for a single state and is taken as the identity; the state is held in bf16
    between depths (the library's activation type).  Returns (idx_hat [l_max,T,K] with -1 past a token's last depth,
    conf [l_max,T] with 0 there, depth [T] = number of predictions enqueued, h_final [T,d])."""
    h = _round_bf16(np.asarray(x, dtype=np.float64))
    T, d = h.shape
    idx_hat = np.full((l_max, T, top_k), -1, dtype=np.int32)
    conf = np.zeros((l_max, T), dtype=np.float64)
    depth = np.zeros(T, dtype=np.int32)
    active = np.ones(T, dtype=bool)
    for l in range(1, l_max + 1):
        L = layers[l - 1]
        logits = router_logits(h.astype(np.float32), L["w_router"])
        ix, pi, c = draft_confidence(logits, top_k)
        new_h = h.copy()
        for t in range(T):
            if not active[t]:
                continue
            idx_hat[l - 1, t] = ix[t]
            conf[l - 1, t] = c[t]
            depth[t] = l
            if l >= l_min and c[t] < tau:
                active[t] = False
                continue
            if l == l_max:
                continue        # the loop ends here: no further state is needed
            ht = h[t].astype(np.float32)
            s = swiglu_ffn(*L["shared"], ht)
            acc = h[t].copy()
            for k in range(top_k):
                i = int(ix[t, k])
                acc += pi[t, i] * (s + lore_delta(L["lore_A"][i], L["lore_B"][i], ht))
            new_h[t] = acc
        h = _round_bf16(new_h)
    return idx_hat, conf, depth, h


def prefetch_set(idx_hat, n_experts: int) -> np.ndarray:
    """Eq. 3: the prefetch intents are the union of the predicted sets.  Experts of different depths belong to different
    layers, so the union over the batch is kept per depth: mask[l-1, e] = 1 iff some token predicts expert e at depth l."""
    idx_hat = np.asarray(idx_hat)
    L = idx_hat.shape[0]
    mask = np.zeros((L, n_experts), dtype=np.uint8)
    for l in range(L):
        for e in idx_hat[l].ravel():
            if e >= 0:
                mask[l, int(e)] = 1
    return mask


def min_lookahead_depth(n_prefetch: int, expert_bytes: float, pcie_bytes_per_s: float, t_comp_s: float) -> int:
    """Eq. 4: H_min = ceil(P * M_e / (B_PCIe * T_comp)), the depth needed to hide P expert transfers per layer."""
    import math
    return int(math.ceil(n_prefetch * expert_bytes / (pcie_bytes_per_s * t_comp_s)))


# ---------------------------------------------------------------------------------------------------------------
# Second weight precision (the paper reports every result at BF16 and at one quantised precision, Sec. 5.1 / Table 1,
# and names that format without defining it).  Reading taken here: weights of the routed and shared experts stored as
# 8-bit floats in the E4M3 layout (1 sign, 4 exponent bits with bias 7, 3 fraction bits; no infinities; S.1111.111 is
# NaN; largest finite value 448; subnormals m/8 * 2^-6) with ONE power-of-two scale per output row:
#     s_r = 2^ceil(log2(max_j |W_rj| / 448))   (1 for an all-zero row),   q_rj = nearest E4M3 value of W_rj / s_r,
# ties to the even code, magnitudes above 448 saturate.  The layer on such weights is BY DEFINITION the layer of
# `layer()` above evaluated on the dequantised values s_r * q_rj (exact in fp32, since s_r is a power of two and q has
# four significant bits); router and LoRE factors keep their precision, so no routing decision depends on the format.


def _e4m3_finite_values() -> np.ndarray:
    """The 127 non-negative finite E4M3 values in code order (code = exponent field * 8 + fraction), as fp64."""
    vals = []
    for code in range(127):                      # code 127 = 1111.111 is NaN
        e, m = code >> 3, code & 7
        vals.append(m / 8.0 * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals, dtype=np.float64)


def e4m3_decode(codes) -> np.ndarray:
    """Value (fp64) of E4M3 bytes; 0x7F / 0xFF decode to NaN."""
    c = np.asarray(codes, dtype=np.uint8)
    mag = np.concatenate([_e4m3_finite_values(), [np.nan]])[c & 0x7F]
    return np.where(c & 0x80, -mag, mag)


def e4m3_encode(x) -> np.ndarray:
    """Nearest finite E4M3 value of every element of x (fp64 arithmetic), as bytes.  Written as the definition: among
    the two neighbouring representable magnitudes the nearer one wins, an exact tie goes to the one whose code is even
    (round-half-to-even), magnitudes beyond 448 give 448.  The sign is kept (also for zero); NaN gives 0x7F."""
    x = np.asarray(x, dtype=np.float64)
    table = _e4m3_finite_values()
    a = np.minimum(np.abs(x), table[-1])
    hi = np.searchsorted(table, a, side="left")          # first code whose value is >= a
    hi = np.minimum(hi, 126)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - table[lo], table[hi] - a
    take_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(take_hi, hi, lo).astype(np.uint8)
    code = np.where(np.isnan(x), np.uint8(0x7F), code)
    return (code | np.where(np.signbit(x) & ~np.isnan(x), np.uint8(0x80), np.uint8(0))).astype(np.uint8)


def quantize_e4m3_rows(W):
    """Per-row power-of-two scale and E4M3 codes of a weight matrix [..., rows, cols] (see the reading above).
    Returns (codes uint8 of W's shape, scale fp32 of W's shape without the last axis)."""
    W = np.asarray(W, dtype=np.float64)
    amax = np.abs(W).max(axis=-1)
    m, e = np.frexp(amax / 448.0)                        # amax / 448 = m * 2^e, m in [0.5, 1)
    exp = np.where(m == 0.5, e - 1, e)                   # ceil(log2(.)) without a logarithm
    scale = np.where(amax > 0, np.ldexp(1.0, exp), 1.0)
    return e4m3_encode(W / scale[..., None]), scale.astype(np.float32)


def dequantize_e4m3_rows(codes, scale) -> np.ndarray:
    """s_r * q_rj as fp32 (exact for power-of-two scales)."""
    v = e4m3_decode(codes) * np.asarray(scale, dtype=np.float64)[..., None]
    out = v.astype(np.float32)
    assert np.array_equal(out.astype(np.float64), v, equal_nan=True), "scale is not a power of two (or out of range)"
    return out


def classify(idx, resident, conf, tau: float, conf_stride: Optional[int] = None):
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, K = idx.shape
    res = np.ascontiguousarray(resident, dtype=np.uint8)
    N = res.shape[0]
    conf = _f32(conf)
    if conf_stride is None:
        conf_stride = 0 if conf.ndim == 1 else N
    cls = np.empty((T, K), dtype=np.uint8)
    counts = np.zeros(3, dtype=np.int32)
    _load().oracle_classify(C.c_int(T), C.c_int(N), C.c_int(K), _p(idx), _p(res), _p(conf),
                            C.c_int(conf_stride), C.c_float(tau), _p(cls), _p(counts))
    return cls, counts


def swiglu_ffn(w_gate, w_up, w_down, x) -> np.ndarray:
    wg, wu, wd, x = _f32(w_gate), _f32(w_up), _f32(w_down), _f32(x)
    I, d = wg.shape
    assert wu.shape == (I, d) and wd.shape == (d, I) and x.shape == (d,)
    out = np.empty(d, dtype=np.float64)
    rc = _load().oracle_swiglu_ffn(C.c_int(d), C.c_int(I), _p(wg), _p(wu), _p(wd), _p(x), _p(out))
    assert rc == 0
    return out


def lore_delta(A, B, x) -> np.ndarray:
    A, B, x = _f32(A), _f32(B), _f32(x)
    r, d = A.shape
    assert B.shape == (d, r) and x.shape == (d,)
    out = np.empty(d, dtype=np.float64)
    rc = _load().oracle_lore_delta(C.c_int(d), C.c_int(r), _p(A), _p(B), _p(x), _p(out))
    assert rc == 0
    return out


def layer(*, h, w_router, experts, shared, lore_A, lore_B, resident, conf, top_k: int, tau: float,
          norm_topk: int = 1, conf_stride: Optional[int] = None, tokens: Optional[Sequence[int]] = None,
          want_full: bool = True, skip_ffn: bool = False) -> LayerResult:
    """Evaluate one layer.

    experts: dict {e: (w_gate [I,d], w_up [I,d], w_down [d,I])} or a list of N such tuples;
             experts that are never evaluated may be absent.
    shared:  (s_gate [I_s,d], s_up [I_s,d], s_down [d,I_s]).
    tokens:  evaluate y / y_full only for these token indices (routing is always done for all).
    skip_ffn: routing + classification only (y, y_full are None).
    """
    h, w_router = _f32(h), _f32(w_router)
    T, d = h.shape
    N = w_router.shape[0]
    K = top_k
    resident = np.ascontiguousarray(resident, dtype=np.uint8)
    conf = _f32(conf)
    if conf_stride is None:
        conf_stride = 0 if conf.ndim == 1 else N
    sg, su, sd = (_f32(a) for a in shared)
    Is = sg.shape[0]
    lore_A, lore_B = _f32(lore_A), _f32(lore_B)
    r = lore_A.shape[1]
    if isinstance(experts, dict):
        items = experts
    else:
        items = {e: w for e, w in enumerate(experts) if w is not None}
    keep = []
    PA = C.c_void_p * N
    pg, pu, pd = PA(), PA(), PA()
    I = None
    for e, (g, u, w) in items.items():
        g, u, w = _f32(g), _f32(u), _f32(w)
        keep.append((g, u, w))
        I = g.shape[0]
        assert g.shape == (I, d) and u.shape == (I, d) and w.shape == (d, I)
        pg[e], pu[e], pd[e] = g.ctypes.data, u.ctypes.data, w.ctypes.data
    if I is None:
        I = 1
    cfg = _Cfg(d, N, K, I, Is, r, norm_topk, conf_stride, tau)
    if skip_ffn:
        sel = np.zeros(1, dtype=np.int32)   # non-NULL pointer, zero rows
    elif tokens is None:
        sel = np.arange(T, dtype=np.int32)
    else:
        sel = np.ascontiguousarray(tokens, dtype=np.int32)
    rows = 0 if skip_ffn else sel.shape[0]
    logits = np.empty((T, N), dtype=np.float64)
    idx = np.empty((T, K), dtype=np.int32)
    gate = np.empty((T, K), dtype=np.float64)
    cls = np.empty((T, K), dtype=np.uint8)
    counts = np.zeros(3, dtype=np.int32)
    n_resid = C.c_int32(0)
    rt = np.empty(T * K, dtype=np.int32)
    rk = np.empty(T * K, dtype=np.int32)
    re_ = np.empty(T * K, dtype=np.int32)
    rg = np.empty(T * K, dtype=np.float64)
    y = np.zeros((rows, d), dtype=np.float64)
    yf = np.zeros((rows, d), dtype=np.float64) if want_full else None
    rc = _load().oracle_layer(
        C.byref(cfg), C.c_int(T), _p(h), _p(w_router), pg, pu, pd, _p(sg), _p(su), _p(sd),
        _p(lore_A), _p(lore_B), _p(resident), _p(conf), C.c_int(rows), _p(sel),
        _p(logits), _p(idx), _p(gate), _p(cls), _p(counts), C.byref(n_resid),
        _p(rt), _p(rk), _p(re_), _p(rg), _p(y), _p(yf) if yf is not None else None)
    if rc != 0:
        raise RuntimeError(f"oracle_layer failed with code {rc} (-(e+1): weights of expert e missing)")
    n = n_resid.value
    return LayerResult(logits, idx, gate, cls, counts, rt[:n].copy(), rk[:n].copy(), re_[:n].copy(),
                       rg[:n].copy(), None if skip_ffn else y, None if (skip_ffn or yf is None) else yf, sel[:rows])
