"""Helpers shared by the tests: run a synthetic workload through the CPU oracle and make
its router logits well separated (so that bit-exact routing parity is a fair demand)."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2608_21240_b200 import workloads as W

MARGIN = 1e-3


def bad_margin_rows(logits: np.ndarray, K: int, margin: float = MARGIN) -> np.ndarray:
    """Rows whose sorted logits have an adjacent gap < margin within the top K+1."""
    top = -np.sort(-logits, axis=1)[:, : K + 1]
    gaps = top[:, :-1] - top[:, 1:]
    return np.nonzero((gaps < margin).any(axis=1))[0]


def enforce_margins(wl: W.LayerWorkload, margin: float = MARGIN, max_rounds: int = 50) -> int:
    """Redraw tokens until every token's top-(K+1) logits are >= margin apart.

    The logits come from the oracle (fp64), the redraw from the generator; returns the
    number of token redraws."""
    n = 0
    for _ in range(max_rounds):
        logits = oracle.router_logits(wl.h, wl.w_router)
        bad = bad_margin_rows(logits, wl.shape.top_k, margin)
        if bad.size == 0:
            return n
        n += bad.size
        wl.redraw_tokens(bad)
    raise AssertionError("could not separate router logits")


def needed_experts(wl: W.LayerWorkload, idx: np.ndarray, tokens=None) -> set:
    rows = range(wl.T) if tokens is None else tokens
    return {int(e) for t in rows for e in idx[t]}


def run_oracle(wl: W.LayerWorkload, tokens=None, want_full: bool = True, conf=None, resident=None,
               lore=None, tau=None, norm_topk=None, skip_ffn=False) -> oracle.LayerResult:
    """Oracle result for a workload; only the experts some evaluated token selects are drawn."""
    s = wl.shape
    resident = wl.resident if resident is None else resident
    pre = oracle.layer(h=wl.h, w_router=wl.w_router, experts={}, shared=_tiny_shared(s),
                       lore_A=np.zeros((s.n_experts, 1, s.d), np.float32),
                       lore_B=np.zeros((s.n_experts, s.d, 1), np.float32),
                       resident=resident, conf=wl.conf if conf is None else conf, top_k=s.top_k,
                       tau=s.tau if tau is None else tau,
                       norm_topk=s.norm_topk if norm_topk is None else norm_topk, skip_ffn=True)
    if skip_ffn:
        return pre
    rows = range(wl.T) if tokens is None else tokens
    need = set()
    for t in rows:
        for k in range(s.top_k):
            c = pre.cls[t, k]
            if c == oracle.HIT or (c == oracle.MISS_EXACT and want_full):
                need.add(int(pre.idx[t, k]))
    experts = {e: wl.expert(e) for e in sorted(need)}
    A, B = wl.lore() if lore is None else lore
    return oracle.layer(h=wl.h, w_router=wl.w_router, experts=experts, shared=wl.shared(), lore_A=A, lore_B=B,
                        resident=resident, conf=wl.conf if conf is None else conf, top_k=s.top_k,
                        tau=s.tau if tau is None else tau,
                        norm_topk=s.norm_topk if norm_topk is None else norm_topk,
                        tokens=tokens, want_full=want_full)


def _tiny_shared(s):
    return (np.zeros((1, s.d), np.float32), np.zeros((1, s.d), np.float32), np.zeros((s.d, 1), np.float32))


# ------------------------------------------------------------------ config 5: the 26-layer decode stack
STACK_LAYERS = 26
STACK_HIT_RATE = 0.7


def rms_normalise(x: np.ndarray) -> np.ndarray:
    """Weight-less RMSNorm (eps 1e-6) between layers: harness glue, not part of the layer call.
    Needed because 26 un-normalised SwiGLU layers with N(0, 0.02) weights would not keep O(1) inputs."""
    x = x.astype(np.float64)
    return x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-6)


def stack_layer(l: int, x: np.ndarray, T: int = 8, variant: int = 0):
    """Inputs and oracle result of layer l of the stack, given the residual stream x [T,d] (fp64).

    Residency is chosen GIVEN the routing: the distinct selected experts are shuffled and made resident until
    >= 70 % of the T*K picks hit; the other slots hold unselected experts (stale prefetches).  Every miss is
    low-confidence with probability 1/2 (conf ~ U(0,tau)) else exact (conf ~ U(tau,1)).
    Returns (workload, oracle result with y and y_full for all tokens, number of redrawn tokens)."""
    s = W.SHAPES["dsv2lite_stack"]
    wl = W.make_layer(s, T, variant=variant, layer=l, n_resident=0)
    wl.h = W.bf16_round(rms_normalise(x).astype(np.float32))
    redrawn = enforce_margins(wl)
    pre = oracle.layer(h=wl.h, w_router=wl.w_router, experts={}, shared=_tiny_shared(s),
                       lore_A=np.zeros((s.n_experts, 1, s.d), np.float32), lore_B=np.zeros((s.n_experts, s.d, 1), np.float32),
                       resident=np.zeros(s.n_experts, np.uint8), conf=wl.conf, top_k=s.top_k, tau=s.tau, skip_ffn=True)
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([W.BASE_SEED, 5, variant, l, 99])))
    picks = pre.idx.ravel()
    selected = rng.permutation(np.unique(picks))
    resident, hits = [], 0
    for e in selected:
        if hits >= STACK_HIT_RATE * picks.size or len(resident) >= s.n_slots:
            break
        resident.append(int(e))
        hits += int((picks == e).sum())
    others = [int(e) for e in rng.permutation(s.n_experts) if e not in set(selected.tolist())]
    resident += others[: s.n_slots - len(resident)]
    soe = np.full(s.n_experts, -1, np.int32)
    soe[np.array(resident)] = rng.permutation(len(resident)).astype(np.int32)
    wl.set_residency(soe)
    tau = np.float32(s.tau)
    for t in range(T):
        for e in pre.idx[t]:
            if soe[e] < 0:
                lo = rng.random() < 0.5
                wl.conf[t, e] = np.float32(rng.uniform(0.0, tau * 0.999) if lo else rng.uniform(tau * 1.001, 1.0))
    ref = run_oracle(wl, want_full=True)
    return wl, ref, redrawn
