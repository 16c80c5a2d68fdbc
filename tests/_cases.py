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
