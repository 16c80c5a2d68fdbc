"""Seeded synthetic inputs for one offloaded-MoE layer (shapes, residency, confidences).

This module only draws random numbers and lays them out.  It performs none of the
layer's arithmetic (no router products, no softmax, no expert evaluation), so the CPU
oracle and the CUDA path can both be fed from it without sharing any method code.

Every floating-point tensor is drawn in fp32 and rounded once to the nearest bf16 value
(round to nearest even); it is returned as fp32 holding exactly representable bf16
values, so the fp32 view handed to a CPU checker and the bf16 bit pattern uploaded to the
GPU describe the same numbers.

Workload shapes follow the two models the paper evaluates (Section 5.1): a
DeepSeek-V2-Lite-shaped layer and a Qwen2-57B-A14B-shaped layer, plus a tiny layer for
exhaustive checks.  Trained weights and the evaluation suites are replaced by
N(0, 0.02) weights, N(0, 1) activations and Beta(2, 2) draft confidences.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Sequence

import numpy as np

BASE_SEED = 20260821

# tensor identifiers that enter the seed sequence
_T_H, _T_ROUTER, _T_GATE, _T_UP, _T_DOWN = 1, 2, 3, 4, 5
_T_SGATE, _T_SUP, _T_SDOWN, _T_LORE_A, _T_LORE_B = 6, 7, 8, 9, 10
_T_RESIDENT, _T_CONF, _T_ZIPF = 11, 12, 13

WEIGHT_STD = 0.02


@dataclass(frozen=True)
class LayerShape:
    """Static description of one MoE layer (notation: d, N, K, I, I_s, r, S, tau)."""

    name: str
    d: int              # hidden width
    n_experts: int      # N routed experts
    top_k: int          # K experts selected per token
    inter: int          # I, routed-expert SwiGLU intermediate width
    inter_shared: int   # I_s, shared-expert intermediate width (all shared experts fused)
    lore_rank: int      # r, rank of the low-rank surrogate
    n_slots: int        # S, GPU-resident expert slots
    tau: float          # confidence threshold
    conf_dist: str = "beta22"   # "beta22" or "uniform"
    norm_topk: int = 1  # gates renormalised over the selected top-k
    cfg_id: int = 0


SHAPES: Dict[str, LayerShape] = {
    # config 1: tiny layer, everything brute-forceable
    "tiny": LayerShape("tiny", d=256, n_experts=8, top_k=2, inter=512, inter_shared=512,
                       lore_rank=16, n_slots=5, tau=0.5, conf_dist="uniform", cfg_id=1),
    # config 2: DeepSeek-V2-Lite-shaped decode layer
    "dsv2lite": LayerShape("dsv2lite", d=2048, n_experts=64, top_k=6, inter=1408,
                           inter_shared=2816, lore_rank=64, n_slots=32, tau=0.6, cfg_id=2),
    # config 3: Qwen2-57B-A14B-shaped decode layer
    "qwen2_57b": LayerShape("qwen2_57b", d=3584, n_experts=64, top_k=8, inter=2560,
                            inter_shared=20480, lore_rank=128, n_slots=24, tau=0.6, cfg_id=3),
    # config 4: DeepSeek-V2-Lite-shaped prefill layer, every expert resident
    "dsv2lite_prefill": LayerShape("dsv2lite_prefill", d=2048, n_experts=64, top_k=6,
                                   inter=1408, inter_shared=2816, lore_rank=64, n_slots=64,
                                   tau=0.6, cfg_id=4),
    # config 5: one layer of the 26-layer decode stack (40 % of experts in slots)
    "dsv2lite_stack": LayerShape("dsv2lite_stack", d=2048, n_experts=64, top_k=6, inter=1408,
                                 inter_shared=2816, lore_rank=64, n_slots=26, tau=0.6, cfg_id=5),
}


def scaled_shape(base: LayerShape, **kw) -> LayerShape:
    """A copy of `base` with some dimensions changed (used for ragged / edge-case tests)."""
    return replace(base, **kw)


# --------------------------------------------------------------------------- bf16 helpers
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Bit pattern (uint16) of values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("bf16_bits: input is not bf16-representable; call bf16_round first")
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Inverse of bf16_bits: widen uint16 bf16 patterns to fp32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([BASE_SEED, *key])))


def _normal(shape, std: float, *key: int) -> np.ndarray:
    g = _rng(*key)
    x = g.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        x *= np.float32(std)
    return bf16_round(x)


# --------------------------------------------------------------------------- the workload
@dataclass
class LayerWorkload:
    """All inputs of one layer call.  Expert weights are drawn lazily, per expert."""

    shape: LayerShape
    T: int
    variant: int = 0
    layer: int = 0                      # layer index inside a stack (enters every seed)
    zipf: bool = False                  # config 4: skewed router so expert loads are imbalanced
    h: np.ndarray = field(default=None, repr=False)               # [T, d]
    w_router: np.ndarray = field(default=None, repr=False)        # [N, d]
    slot_of_expert: np.ndarray = field(default=None, repr=False)  # [N] int32, -1 = not resident
    conf: np.ndarray = field(default=None, repr=False)            # [T, N] fp32
    _cache: dict = field(default_factory=dict, repr=False)
    _redraws: int = 0

    # ---- seeds
    def _key(self, tensor: int, index: int = 0):
        return (self.shape.cfg_id, self.variant, self.layer, tensor, index)

    # ---- lazily drawn weights (fp32 arrays holding bf16 values)
    def expert(self, e: int):
        """(w_gate [I,d], w_up [I,d], w_down [d,I]) of routed expert e."""
        k = ("expert", e)
        if k not in self._cache:
            s = self.shape
            self._cache[k] = (
                _normal((s.inter, s.d), WEIGHT_STD, *self._key(_T_GATE, e)),
                _normal((s.inter, s.d), WEIGHT_STD, *self._key(_T_UP, e)),
                _normal((s.d, s.inter), WEIGHT_STD, *self._key(_T_DOWN, e)),
            )
        return self._cache[k]

    def drop_expert(self, e: int) -> None:
        self._cache.pop(("expert", e), None)

    def shared(self):
        """(s_gate [I_s,d], s_up [I_s,d], s_down [d,I_s]) of the fused shared expert."""
        if "shared" not in self._cache:
            s = self.shape
            self._cache["shared"] = (
                _normal((s.inter_shared, s.d), WEIGHT_STD, *self._key(_T_SGATE)),
                _normal((s.inter_shared, s.d), WEIGHT_STD, *self._key(_T_SUP)),
                _normal((s.d, s.inter_shared), WEIGHT_STD, *self._key(_T_SDOWN)),
            )
        return self._cache["shared"]

    def lore(self):
        """(A [N,r,d], B [N,d,r]) low-rank surrogate factors for every routed expert."""
        if "lore" not in self._cache:
            s = self.shape
            self._cache["lore"] = (
                _normal((s.n_experts, s.lore_rank, s.d), WEIGHT_STD, *self._key(_T_LORE_A)),
                _normal((s.n_experts, s.d, s.lore_rank), WEIGHT_STD, *self._key(_T_LORE_B)),
            )
        return self._cache["lore"]

    # ---- residency
    @property
    def resident(self) -> np.ndarray:
        return (self.slot_of_expert >= 0).astype(np.uint8)

    def expert_of_slot(self) -> np.ndarray:
        s = self.shape
        out = np.full(s.n_slots, -1, dtype=np.int32)
        for e, sl in enumerate(self.slot_of_expert):
            if sl >= 0:
                out[sl] = e
        return out

    def set_residency(self, slot_of_expert: Sequence[int]) -> None:
        a = np.asarray(slot_of_expert, dtype=np.int32).copy()
        assert a.shape == (self.shape.n_experts,)
        used = a[a >= 0]
        assert used.size <= self.shape.n_slots and np.unique(used).size == used.size
        assert (used < self.shape.n_slots).all()
        self.slot_of_expert = a

    # ---- slot pool in the device layout: gate rows then up rows; down
    def slot_pool_bits(self, only=None):
        """bf16 bit patterns: slot_w_gate_up [S,2I,d], slot_w_down [S,d,I] (empty slots zero).

        only: if given, a set of expert ids; slots of other experts are left zero (they model stale
        prefetches that no token of the batch uses, so their contents are never read)."""
        s = self.shape
        gu = np.zeros((s.n_slots, 2 * s.inter, s.d), dtype=np.uint16)
        dn = np.zeros((s.n_slots, s.d, s.inter), dtype=np.uint16)
        for sl, e in enumerate(self.expert_of_slot()):
            if e < 0 or (only is not None and int(e) not in only):
                continue
            keep = ("expert", int(e)) in self._cache
            g, u, w = self.expert(int(e))
            gu[sl, : s.inter] = bf16_bits(g)
            gu[sl, s.inter:] = bf16_bits(u)
            dn[sl] = bf16_bits(w)
            if not keep:
                self.drop_expert(int(e))
        return gu, dn

    # ---- token redraw (used by callers that need well-separated router logits)
    def redraw_tokens(self, rows: Sequence[int]) -> None:
        """Replace the given rows of h by fresh draws (deterministic in the redraw count)."""
        self._redraws += 1
        for t in rows:
            row = _normal((self.shape.d,), 1.0, *self._key(_T_H, 1_000_003 * self._redraws + int(t)))
            if self.zipf:
                row[0] = 1.0
            self.h[int(t)] = row


def make_layer(shape_name: str | LayerShape, T: int, variant: int = 0, layer: int = 0,
               zipf: bool = False, n_resident: Optional[int] = None) -> LayerWorkload:
    """Draw h, router, residency table and confidences for one layer call.

    Residency: a seeded permutation pi of the experts; experts pi[0..S) are resident and
    slot_of_expert[pi[i]] = i, so slot order differs from expert order on purpose.
    Confidences: U(0,1) or Beta(2,2) per (token, expert); values within 1e-6 of tau are
    redrawn so the threshold comparison cannot depend on rounding.
    """
    s = SHAPES[shape_name] if isinstance(shape_name, str) else shape_name
    w = LayerWorkload(shape=s, T=T, variant=variant, layer=layer, zipf=zipf)
    w.h = _normal((T, s.d), 1.0, *w._key(_T_H))
    w.w_router = _normal((s.n_experts, s.d), WEIGHT_STD, *w._key(_T_ROUTER))
    if zipf:
        # expert popularity ~ rank^-1.1: a constant feature carries a per-expert log-bias
        g = _rng(*w._key(_T_ZIPF))
        rank = g.permutation(s.n_experts) + 1
        w.h[:, 0] = 1.0
        w.w_router[:, 0] = bf16_round((-1.1 * np.log(rank)).astype(np.float32))
    g = _rng(*w._key(_T_RESIDENT))
    perm = g.permutation(s.n_experts)
    nres = s.n_slots if n_resident is None else n_resident
    assert 0 <= nres <= s.n_slots
    soe = np.full(s.n_experts, -1, dtype=np.int32)
    soe[perm[:nres]] = np.arange(nres, dtype=np.int32)
    w.slot_of_expert = soe
    g = _rng(*w._key(_T_CONF))
    if s.conf_dist == "uniform":
        c = g.random(size=(T, s.n_experts))
    else:
        c = g.beta(2.0, 2.0, size=(T, s.n_experts))
    c = c.astype(np.float32)
    tau32 = np.float32(s.tau)
    bad = np.abs(c - tau32) < 1e-6
    while bad.any():
        c[bad] = g.random(size=int(bad.sum())).astype(np.float32)
        bad = np.abs(c - tau32) < 1e-6
    w.conf = c
    return w
