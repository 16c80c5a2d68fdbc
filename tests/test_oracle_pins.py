"""Pins for the CPU oracle: it is checked against things other than itself -- brute-force
dense evaluation through an independent numpy path, invariants, closed forms, special
cases that reduce to the textbook MoE layer, and a hand-computed example."""
import os

import numpy as np
import pytest

import oracle
from paper_2608_21240_b200 import workloads as W
from tests._cases import enforce_margins

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ independent numpy path
def np_silu(v):
    return v / (1.0 + np.exp(-v))


def np_ffn(wg, wu, wd, X):
    """SwiGLU FFN for a batch, all in fp64 numpy matmuls.  X: [T,d] -> [T,d]."""
    X = X.astype(np.float64)
    a = np_silu(X @ wg.astype(np.float64).T) * (X @ wu.astype(np.float64).T)
    return a @ wd.astype(np.float64).T


def np_dense_gates(h, w_router, K, norm_topk=1):
    """Dense [T,N] gate matrix built by sorting full-softmax probabilities."""
    logits = h.astype(np.float64) @ w_router.astype(np.float64).T
    z = logits - logits.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    order = np.argsort(-p, axis=1, kind="stable")[:, :K]
    G = np.zeros_like(p)
    for t in range(h.shape[0]):
        sel = order[t]
        G[t, sel] = p[t, sel] / p[t, sel].sum() if norm_topk else p[t, sel]
    return G, order


def tiny(T=4, variant=0, **kw):
    s = W.scaled_shape(W.SHAPES["tiny"], **kw) if kw else W.SHAPES["tiny"]
    wl = W.make_layer(s, T, variant=variant)
    enforce_margins(wl)
    return wl


def run(wl, resident=None, conf=None, lore=None, tau=None, norm_topk=1, tokens=None):
    s = wl.shape
    A, B = wl.lore() if lore is None else lore
    return oracle.layer(h=wl.h, w_router=wl.w_router, experts=[wl.expert(e) for e in range(s.n_experts)],
                        shared=wl.shared(), lore_A=A, lore_B=B,
                        resident=wl.resident if resident is None else resident,
                        conf=wl.conf if conf is None else conf, top_k=s.top_k,
                        tau=s.tau if tau is None else tau, norm_topk=norm_topk, tokens=tokens)


def dense_layer(wl, norm_topk=1):
    s = wl.shape
    G, order = np_dense_gates(wl.h, wl.w_router, s.top_k, norm_topk)
    y = np_ffn(*wl.shared(), wl.h)
    for e in range(s.n_experts):
        y = y + G[:, [e]] * np_ffn(*wl.expert(e), wl.h)
    return y, G, order


def rel(a, b):
    return np.abs(a - b).max() / max(np.abs(b).max(), 1e-30)


# ------------------------------------------------------------------ P1 brute force
@pytest.mark.parametrize("variant,norm_topk", [(0, 1), (1, 1), (2, 0)])
def test_p1_all_resident_equals_bruteforce_dense(variant, norm_topk):
    wl = tiny(T=5, variant=variant)
    res = run(wl, resident=np.ones(wl.shape.n_experts, np.uint8), norm_topk=norm_topk)
    y, G, order = dense_layer(wl, norm_topk)
    assert rel(res.y, y) < 1e-9
    assert rel(res.y_full, y) < 1e-9
    assert (res.idx == order).all()
    assert res.counts.tolist() == [wl.T * wl.shape.top_k, 0, 0] and res.resid_tok.size == 0


def test_router_logits_match_numpy_matmul():
    wl = tiny(T=7)
    ref = wl.h.astype(np.float64) @ wl.w_router.astype(np.float64).T
    assert np.abs(oracle.router_logits(wl.h, wl.w_router) - ref).max() < 1e-12


def test_ffn_and_lore_match_numpy():
    wl = tiny(T=3)
    for e in (0, 3):
        ref = np_ffn(*wl.expert(e), wl.h[1:2])[0]
        assert rel(oracle.swiglu_ffn(*wl.expert(e), wl.h[1]), ref) < 1e-10
    A, B = wl.lore()
    ref = B[2].astype(np.float64) @ (A[2].astype(np.float64) @ wl.h[0].astype(np.float64))
    assert rel(oracle.lore_delta(A[2], B[2], wl.h[0]), ref) < 1e-10
    # a transposed operand would give the wrong shape/values: asymmetric check
    wg, wu, wd = wl.expert(1)
    assert rel(oracle.swiglu_ffn(wg, wu, wd, wl.h[0]), np_ffn(wu, wg, wd, wl.h[0:1])[0]) > 1e-3


# ------------------------------------------------------------------ P2 gate invariants
@pytest.mark.parametrize("K", [1, 2, 3, 8])
def test_p2_gate_invariants(K):
    rng = np.random.default_rng(5)
    logits = rng.normal(size=(9, 8)) * 2.0
    idx, gate = oracle.topk_gates(logits, K, 1)
    assert np.allclose(gate.sum(axis=1), 1.0, atol=1e-12)
    assert (gate > 0).all() and (np.diff(gate, axis=1) <= 1e-15).all()
    for t in range(9):
        assert len(set(idx[t])) == K and idx[t].min() >= 0 and idx[t].max() < 8
        assert (np.sort(logits[t])[::-1][:K] == logits[t, idx[t]]).all()
    if K == 8:   # K = N: gates are the full softmax
        p = np.exp(logits - logits.max(1, keepdims=True))
        p /= p.sum(1, keepdims=True)
        assert np.allclose(np.take_along_axis(p, idx, 1), gate, atol=1e-13)
    if K == 1:
        assert (gate == 1.0).all()
    # shift invariance
    idx2, gate2 = oracle.topk_gates(logits + 3.25, K, 1)
    assert (idx2 == idx).all() and np.allclose(gate2, gate, atol=1e-13)
    # un-normalised variant = full softmax probabilities of the winners
    idx3, gate3 = oracle.topk_gates(logits, K, 0)
    p = np.exp(logits - logits.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    assert (idx3 == idx).all() and np.allclose(np.take_along_axis(p, idx, 1), gate3, atol=1e-13)


def test_topk_ties_prefer_lower_index():
    logits = np.array([[1.0, 3.0, 3.0, 0.5, 3.0, 2.0]])
    idx, gate = oracle.topk_gates(logits, 4, 1)
    assert idx.tolist() == [[1, 2, 4, 5]]


# ------------------------------------------------------------------ P3 all-hit = textbook MoE
def test_p3_all_hit_ignores_conf_tau_lore():
    wl = tiny(T=4)
    ones = np.ones(wl.shape.n_experts, np.uint8)
    base = run(wl, resident=ones)
    A, B = wl.lore()
    other = run(wl, resident=ones, conf=np.zeros_like(wl.conf), tau=2.0, lore=(A * 3, B * -2))
    assert np.array_equal(base.y, other.y) and other.counts[2] == 0


# ------------------------------------------------------------------ P4 rank-sufficient LoRE
def test_p4_rank_sufficient_lore_reproduces_exact_expert():
    wl = tiny(T=4)
    s = wl.shape
    H = wl.h.astype(np.float64).T                      # [d,T]
    Hp = np.linalg.pinv(H)                             # [T,d], Hp @ H = I_T
    SH = np_ffn(*wl.shared(), wl.h).T                  # [d,T]
    A = np.zeros((s.n_experts, s.lore_rank, s.d))
    B = np.zeros((s.n_experts, s.d, s.lore_rank))
    for e in range(s.n_experts):
        A[e, : wl.T] = Hp
        B[e, :, : wl.T] = np_ffn(*wl.expert(e), wl.h).T - SH
    # fp32 storage of A,B costs ~1e-7 relative; keep fp64 by calling with float32 copies and loose bound
    all_hit = run(wl, resident=np.ones(s.n_experts, np.uint8))
    for mask_seed in range(3):
        rng = np.random.default_rng(mask_seed)
        resident = (rng.random(s.n_experts) < 0.4).astype(np.uint8)
        res = run(wl, resident=resident, conf=np.zeros_like(wl.conf), tau=0.5, lore=(A, B))
        assert res.counts[1] == 0 and res.counts[2] > 0
        assert rel(res.y, all_hit.y) < 2e-5
    none = run(wl, resident=np.zeros(s.n_experts, np.uint8), conf=np.zeros_like(wl.conf), tau=0.5, lore=(A, B))
    assert none.counts.tolist() == [0, 0, wl.T * s.top_k]
    assert rel(none.y, all_hit.y) < 2e-5


def test_p4b_identity_lore_full_rank():
    """r = d, A = I: B A h = B h, so a linear 'expert minus shared' map is reproduced exactly."""
    s = W.scaled_shape(W.SHAPES["tiny"], d=32, inter=16, inter_shared=16, lore_rank=32)
    wl = W.make_layer(s, 3)
    enforce_margins(wl)
    rng = np.random.default_rng(0)
    Bm = rng.normal(size=(s.n_experts, s.d, s.d)).astype(np.float32)
    A = np.broadcast_to(np.eye(s.d, dtype=np.float32), (s.n_experts, s.d, s.d)).copy()
    res = run(wl, resident=np.zeros(s.n_experts, np.uint8), conf=np.zeros_like(wl.conf), tau=0.5, lore=(A, Bm))
    S = np_ffn(*wl.shared(), wl.h)
    exp = np.zeros_like(S)
    for t in range(wl.T):
        exp[t] = S[t]
        for k in range(s.top_k):
            e = res.idx[t, k]
            exp[t] += res.gate[t, k] * (S[t] + Bm[e].astype(np.float64) @ wl.h[t].astype(np.float64))
    assert rel(res.y, exp) < 1e-10


# ------------------------------------------------------------------ P5 / P6 closed forms
def test_p5_all_miss_high_conf_gives_shared_only():
    wl = tiny(T=4)
    s = wl.shape
    res = run(wl, resident=np.zeros(s.n_experts, np.uint8), conf=np.ones_like(wl.conf), tau=0.5)
    S = np_ffn(*wl.shared(), wl.h)
    assert rel(res.y, S) < 1e-10
    assert res.resid_tok.size == wl.T * s.top_k and res.counts.tolist() == [0, wl.T * s.top_k, 0]
    dense, _, _ = dense_layer(wl)
    assert rel(res.y_full, dense) < 1e-9
    # residual list is in (t,k) order and carries the routing
    assert (res.resid_tok == np.repeat(np.arange(wl.T), s.top_k)).all()
    assert (res.resid_k == np.tile(np.arange(s.top_k), wl.T)).all()
    assert (res.resid_expert == res.idx.ravel()).all() and np.array_equal(res.resid_gate, res.gate.ravel())


def test_p6_all_miss_low_conf_zero_lore_gives_twice_shared():
    wl = tiny(T=4)
    s = wl.shape
    A, B = wl.lore()
    res = run(wl, resident=np.zeros(s.n_experts, np.uint8), conf=np.zeros_like(wl.conf), tau=0.5,
              lore=(A * 0, B * 0))
    S = np_ffn(*wl.shared(), wl.h)
    assert rel(res.y, 2 * S) < 1e-10
    assert res.resid_tok.size == 0


# ------------------------------------------------------------------ P7 threshold edges
def test_p7_threshold_edges():
    idx = np.array([[0, 1, 2, 3]], dtype=np.int32)
    resident = np.array([1, 0, 0, 0], np.uint8)
    tau = np.float32(0.6)
    conf = np.array([[0.0, tau, np.nextafter(tau, np.float32(0)), np.nan]], dtype=np.float32)
    cls, counts = oracle.classify(idx, resident, conf, float(tau))
    assert cls.tolist() == [[oracle.HIT, oracle.MISS_EXACT, oracle.LOWCONF, oracle.MISS_EXACT]]
    assert counts.tolist() == [1, 2, 1]
    cls0, _ = oracle.classify(idx, resident, np.abs(np.nan_to_num(conf)), 0.0)
    assert (cls0[0, 1:] == oracle.MISS_EXACT).all()           # tau = 0: nothing is low-confidence
    cls2, _ = oracle.classify(idx, resident, np.nan_to_num(conf), 1.5)
    assert (cls2[0, 1:] == oracle.LOWCONF).all()              # tau > 1: every miss is
    # one scalar confidence per token (conf_stride = 0)
    cls3, _ = oracle.classify(np.array([[1, 2], [1, 2]], np.int32), resident, np.array([0.1, 0.9], np.float32), 0.6)
    assert cls3.tolist() == [[oracle.LOWCONF] * 2, [oracle.MISS_EXACT] * 2]


# ------------------------------------------------------------------ P8 linearity
def test_p8_lore_term_is_linear_and_residual_is_exact_sum():
    wl = tiny(T=4, variant=3)
    s = wl.shape
    A, B = wl.lore()
    r1 = run(wl)
    r0 = run(wl, lore=(A, B * 0))
    r3 = run(wl, lore=(A, B * 3))
    assert r1.counts[2] > 0 and r1.counts[1] > 0 and r1.counts[0] > 0
    assert rel(r3.y - r0.y, 3 * (r1.y - r0.y)) < 1e-9
    extra = np.zeros_like(r1.y)
    for t, k, e, g in zip(r1.resid_tok, r1.resid_k, r1.resid_expert, r1.resid_gate):
        assert r1.idx[t, k] == e and r1.cls[t, k] == oracle.MISS_EXACT
        extra[t] += g * np_ffn(*wl.expert(e), wl.h[t:t + 1])[0]
    assert rel(r1.y_full - r1.y, extra) < 1e-9


# ------------------------------------------------------------------ P9 symmetries
def test_p9_token_permutation_and_batch_independence():
    wl = tiny(T=5, variant=1)
    full = run(wl)
    for t in range(wl.T):
        one = oracle.layer(h=wl.h[t:t + 1], w_router=wl.w_router,
                           experts=[wl.expert(e) for e in range(wl.shape.n_experts)], shared=wl.shared(),
                           lore_A=wl.lore()[0], lore_B=wl.lore()[1], resident=wl.resident,
                           conf=wl.conf[t:t + 1], top_k=wl.shape.top_k, tau=wl.shape.tau)
        assert np.array_equal(one.y[0], full.y[t]) and (one.idx[0] == full.idx[t]).all()
    sub = run(wl, tokens=[3, 1])
    assert np.array_equal(sub.y, full.y[[3, 1]]) and np.array_equal(sub.y_full, full.y_full[[3, 1]])


def test_p9_expert_relabelling():
    wl = tiny(T=4, variant=2)
    s = wl.shape
    base = run(wl)
    perm = np.random.default_rng(1).permutation(s.n_experts)      # new expert j = old expert perm[j]
    A, B = wl.lore()
    res = oracle.layer(h=wl.h, w_router=wl.w_router[perm], experts=[wl.expert(int(perm[j])) for j in range(s.n_experts)],
                       shared=wl.shared(), lore_A=A[perm], lore_B=B[perm], resident=wl.resident[perm],
                       conf=wl.conf[:, perm], top_k=s.top_k, tau=s.tau)
    assert (perm[res.idx] == base.idx).all() and (res.cls == base.cls).all()
    assert rel(res.y, base.y) < 1e-12


# ------------------------------------------------------------------ P10 closed forms
def test_p10_zero_input_gives_zero_output():
    wl = tiny(T=2)
    wl.h[:] = 0
    res = run(wl)
    assert np.abs(res.y).max() == 0.0


def test_p10_hand_computed_example():
    rows = []
    with open(os.path.join(GOLD, "swiglu_hand_example.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if len(line) == 4:
                rows.append((line[0], int(line[1]), float(line[2]), float(line[3])))
    assert len(rows) == 5
    h = np.array([[1.0, 2.0]], np.float32)
    wr = np.eye(2, dtype=np.float32)
    e1 = (np.array([[1, 0.5]], np.float32), np.array([[0.5, 0.25]], np.float32), np.array([[2], [-1]], np.float32))
    e0 = (np.array([[-1, 0.5]], np.float32), np.array([[1, 1]], np.float32), np.array([[1], [3]], np.float32))
    sh = (np.array([[1, 0]], np.float32), np.array([[0, 1]], np.float32), np.array([[1], [1]], np.float32))
    A = np.array([[[9, 9]], [[1, 1]]], np.float32)
    B = np.array([[[9], [9]], [[0.5], [-0.5]]], np.float32)
    for case, norm, y0, y1 in rows:
        resident = np.array([0, 1 if case == "hit" else 0], np.uint8)
        conf = np.array([[0.9, 0.1 if case == "lowconf" else 0.9]], np.float32)
        res = oracle.layer(h=h, w_router=wr, experts=[e0, e1], shared=sh, lore_A=A, lore_B=B, resident=resident,
                           conf=conf, top_k=1, tau=0.5, norm_topk=norm)
        assert res.idx.tolist() == [[1]]
        assert np.allclose(res.y[0], [y0, y1], rtol=0, atol=1e-14), (case, norm, res.y)
        assert res.resid_tok.size == (1 if case == "exact" else 0)


# ------------------------------------------------------------------ P12 y_full vs dense
@pytest.mark.parametrize("seed", [0, 1])
def test_p12_y_full_equals_dense_when_nothing_is_substituted(seed):
    wl = tiny(T=4, variant=seed)
    resident = (np.random.default_rng(seed).random(wl.shape.n_experts) < 0.5).astype(np.uint8)
    res = run(wl, resident=resident, tau=0.0)
    assert res.counts[2] == 0 and res.counts[1] > 0
    dense, _, _ = dense_layer(wl)
    assert rel(res.y_full, dense) < 1e-9


# ------------------------------------------------------------------ draft-router confidence (Sec. 4.1, Eq. 2 and Eq. 5)
def test_p13_draft_confidence_hand_example():
    """Logits ln(1..4): the distribution is (0.1, 0.2, 0.3, 0.4) by inspection, so the top two experts are 3 and 2
    and the confidence is 0.7; with K = N the mass is 1, with K = 1 it is the largest probability."""
    logits = np.log(np.array([[1.0, 2.0, 3.0, 4.0]]))
    idx, pi, conf = oracle.draft_confidence(logits, 2)
    assert idx.tolist() == [[3, 2]]
    assert np.allclose(pi, [[0.1, 0.2, 0.3, 0.4]], atol=1e-15)
    assert abs(conf[0] - 0.7) < 1e-15
    assert abs(oracle.draft_confidence(logits, 4)[2][0] - 1.0) < 1e-15
    assert abs(oracle.draft_confidence(logits, 1)[2][0] - 0.4) < 1e-15


@pytest.mark.parametrize("N,K", [(8, 2), (64, 6), (64, 8), (10, 10)])
def test_p13_draft_confidence_invariants(N, K):
    rng = np.random.default_rng(5 + N + K)
    logits = rng.standard_normal((7, N)) * 1.3
    idx, pi, conf = oracle.draft_confidence(logits, K)
    # a distribution; independent numpy path: sort the softmax, add the K largest
    assert np.allclose(pi.sum(axis=1), 1.0, atol=1e-14) and (pi >= 0).all()
    z = np.exp(logits - logits.max(axis=1, keepdims=True))
    p = z / z.sum(axis=1, keepdims=True)
    assert np.allclose(conf, np.sort(p, axis=1)[:, ::-1][:, :K].sum(axis=1), atol=1e-14)
    assert np.array_equal(idx, np.argsort(-logits, axis=1, kind="stable")[:, :K])
    # shift invariance, bounds, monotone in K, uniform logits give K / N
    assert np.allclose(oracle.draft_confidence(logits + 3.25, K)[2], conf, atol=1e-14)
    assert (conf <= 1.0 + 1e-15).all() and (conf >= K / N - 1e-15).all()
    if K > 1:
        assert (oracle.draft_confidence(logits, K - 1)[2] < conf).all()
    assert np.allclose(oracle.draft_confidence(np.full((2, N), 0.37), K)[2], K / N, atol=1e-15)
    # the selected set and its probabilities are those of the router of Eq. 1 with un-normalised gates
    idx1, gate1 = oracle.topk_gates(logits, K, norm_topk=0)
    assert np.array_equal(idx1, idx) and np.allclose(gate1.sum(axis=1), conf, atol=1e-14)


def test_p13_draft_confidence_ties_prefer_lower_index():
    logits = np.array([[0.5, 1.0, 1.0, 0.5, 1.0]])
    idx, pi, conf = oracle.draft_confidence(logits, 2)
    assert idx.tolist() == [[1, 2]]


# ------------------------------------------------------------------ Algorithm 1: speculative prefetch rollout
def _rollout_layers(rng, L, N, d, Is, r, shared_scale=0.3, lore_scale=0.3, same_router=False):
    wr = W.bf16_round(rng.standard_normal((N, d)).astype(np.float32))
    out = []
    for _ in range(L):
        out.append(dict(
            w_router=wr if same_router else W.bf16_round(rng.standard_normal((N, d)).astype(np.float32)),
            shared=tuple(W.bf16_round((rng.standard_normal(sz) * shared_scale).astype(np.float32)) for sz in ((Is, d), (Is, d), (d, Is))),
            lore_A=W.bf16_round((rng.standard_normal((N, r, d)) * lore_scale).astype(np.float32)),
            lore_B=W.bf16_round((rng.standard_normal((N, d, r)) * lore_scale).astype(np.float32))))
    return out


def test_p14_rollout_depth_one_is_the_draft_confidence():
    rng = np.random.default_rng(14)
    N, d, K, T = 10, 32, 3, 6
    layers = _rollout_layers(rng, 1, N, d, 16, 4)
    x = W.bf16_round(rng.standard_normal((T, d)).astype(np.float32))
    idx, conf, depth, h = oracle.prefetch_rollout(x, layers, K, 1, 1, 0.5)
    ix, pi, c = oracle.draft_confidence(oracle.router_logits(x, layers[0]["w_router"]), K)
    assert np.array_equal(idx[0], ix) and np.array_equal(conf[0], c) and (depth == 1).all() and np.array_equal(h, x)


def test_p14_rollout_halting_rule():
    """tau = 0 never halts (depth = l_max); tau > 1 halts as soon as l >= l_min, keeping the prediction made there;
    in between, a token stops exactly at the first depth >= l_min whose confidence is below tau."""
    rng = np.random.default_rng(15)
    N, d, K, T, L = 12, 32, 2, 9, 5
    layers = _rollout_layers(rng, L, N, d, 16, 4)
    x = W.bf16_round(rng.standard_normal((T, d)).astype(np.float32))
    idx, conf, depth, _ = oracle.prefetch_rollout(x, layers, K, 2, L, 0.0)
    assert (depth == L).all() and (idx >= 0).all()
    idx, conf, depth, _ = oracle.prefetch_rollout(x, layers, K, 3, L, 1.5)
    assert (depth == 3).all() and (idx[:3] >= 0).all() and (idx[3:] == -1).all() and (conf[3:] == 0).all()
    tau = float(np.median(conf[:3]))
    idx2, conf2, depth2, _ = oracle.prefetch_rollout(x, layers, K, 2, L, tau)
    for t in range(T):
        below = [l for l in range(2, L + 1) if conf2[l - 1, t] < tau and depth2[t] >= l]
        assert depth2[t] == (below[0] if below else L)
        assert (idx2[depth2[t]:, t] == -1).all() and (idx2[:depth2[t], t] >= 0).all()
    assert len(set(depth2.tolist())) > 1      # the threshold actually separates the tokens


def test_p14_rollout_state_projection_matches_numpy():
    """One projection step written out with numpy matmuls: h1 = h0 + C S(h0) + sum_i pi_i B_i A_i h0 (Attn = identity),
    and its two special cases: zero LoRE (shared expert only) and zero shared expert (low-rank maps only)."""
    rng = np.random.default_rng(16)
    N, d, K, T, Is, r = 8, 24, 3, 4, 16, 5
    x = W.bf16_round(rng.standard_normal((T, d)).astype(np.float32))
    for shared_scale, lore_scale in ((0.3, 0.3), (0.3, 0.0), (0.0, 0.3)):
        layers = _rollout_layers(rng, 2, N, d, Is, r, shared_scale, lore_scale)
        _, _, depth, h1 = oracle.prefetch_rollout(x, layers, K, 2, 2, 0.0)
        L0 = layers[0]
        logits = x.astype(np.float64) @ L0["w_router"].astype(np.float64).T
        p = np.exp(logits - logits.max(axis=1, keepdims=True))
        p /= p.sum(axis=1, keepdims=True)
        sel = np.argsort(-logits, axis=1, kind="stable")[:, :K]
        S = np_ffn(*L0["shared"], x)
        want = x.astype(np.float64).copy()
        for t in range(T):
            want[t] += p[t, sel[t]].sum() * S[t]
            for i in sel[t]:
                want[t] += p[t, i] * (L0["lore_B"][i].astype(np.float64) @ (L0["lore_A"][i].astype(np.float64) @ x[t].astype(np.float64)))
        assert (depth == 2).all()
        assert np.abs(h1 - want).max() <= 2.0 ** -8 * np.abs(want).max()      # h1 is the bf16 rounding of `want`


def test_p14_rollout_fixed_point_when_nothing_is_added():
    """Zero shared expert and zero LoRE: the state never moves, so with one router for all depths every depth
    predicts the same set with the same confidence."""
    rng = np.random.default_rng(17)
    N, d, K, T, L = 9, 16, 2, 5, 4
    layers = _rollout_layers(rng, L, N, d, 8, 3, 0.0, 0.0, same_router=True)
    x = W.bf16_round(rng.standard_normal((T, d)).astype(np.float32))
    idx, conf, depth, h = oracle.prefetch_rollout(x, layers, K, 1, L, 0.0)
    assert np.array_equal(h, x) and all(np.array_equal(idx[l], idx[0]) and np.array_equal(conf[l], conf[0]) for l in range(L))


def test_p14_rollout_state_rounding_is_nearest_even_bf16():
    """The bf16 rounding of the draft state between depths, pinned on hand-written values (a bf16 keeps 8 significant
    bits: the spacing in [1, 2) is 2^-7, so 1 + 2^-8 lies exactly between 1 and 1 + 2^-7).  Truncation fails the
    round-up rows, round-half-up fails the first tie, round-half-down the second; a detour over fp32 fails the last two
    rows, which sit within 2^-30 of a tie (fp32 would first round them ONTO the tie)."""
    f = oracle._round_bf16
    u = 2.0 ** -7                      # one bf16 step in [1, 2)
    rows = [
        (1.0, 1.0),                            # representable
        (-3.140625, -3.140625),                # representable, negative (-(3 + 9/64): 8 significant bits)
        (1.0 + 0.5 * u, 1.0),                  # tie, even mantissa below   -> down
        (1.0 + 1.5 * u, 1.0 + 2 * u),          # tie, even mantissa above   -> up
        (-(1.0 + 1.5 * u), -(1.0 + 2 * u)),    # the same tie, negative: magnitude rounds, sign kept
        (1.0 + 0.5 * u + 2.0 ** -20, 1.0 + u),       # just above a tie -> up
        (1.0 + 0.5 * u - 2.0 ** -20, 1.0),           # just below a tie -> down
        (1.0 + 0.75 * u, 1.0 + u),             # above half -> up (truncation would give 1)
        (1.0 + 0.25 * u, 1.0),                 # below half -> down
        (255.5, 256.0),                        # tie at the top of a binade (255 = 11111111b is odd) carries into the exponent
        (2.0 ** -100 * (1.0 + 0.75 * u), 2.0 ** -100 * (1.0 + u)),   # the same away from 1
        (1.0 + 0.5 * u + 2.0 ** -30, 1.0 + u),       # above the tie by less than an fp32 ulp (2^-23): still up
        (1.0 + 1.5 * u - 2.0 ** -30, 1.0 + u),       # below the tie by less than an fp32 ulp: still down
    ]
    x = np.array([a for a, _ in rows], dtype=np.float64)
    want = np.array([b for _, b in rows], dtype=np.float64)
    got = f(x)
    assert got.dtype == np.float64 and np.array_equal(got, want), list(zip(x.tolist(), got.tolist(), want.tolist()))
    assert np.array_equal(f(got), got)                       # idempotent
    assert np.signbit(f(np.array([-0.0]))[0]) and f(np.array([0.0]))[0] == 0.0
    # every result has at most 8 significant bits: scaled to [128, 256) it is an integer
    rng = np.random.default_rng(141)
    r = f(rng.standard_normal(1000) * 10.0 ** rng.integers(-3, 4, 1000))
    m, _ = np.frexp(r)
    assert np.array_equal(m * 256.0, np.round(m * 256.0))
    # and it agrees with the generator's fp32 -> bf16 rounding wherever the input is an fp32 value
    x32 = (rng.standard_normal(1000) * 3.0).astype(np.float32)
    assert np.array_equal(f(x32.astype(np.float64)), W.bf16_round(x32).astype(np.float64))


# ------------------------------------------------------------------ LoRE calibration (Sec. 4.2, the fitting objective)
def _lore_loss(H, R, A, B):
    return float(((R - (H @ A.T) @ B.T) ** 2).sum())


def test_p15_lore_calibration_is_eckart_young_for_orthonormal_inputs():
    """H with orthonormal columns and an exactly linear target R = H M^T: the objective is ||M - BA||_F^2, whose minimiser
    over rank-r maps is the truncated SVD of M (Eckart-Young), with loss = sum of the discarded squared singular values."""
    rng = np.random.default_rng(21)
    n, d, r = 40, 12, 4
    H = np.linalg.qr(rng.standard_normal((n, d)))[0]
    M = rng.standard_normal((d, d))
    A, B, loss = oracle.lore_calibrate(H, H @ M.T, r)
    U, S, Vt = np.linalg.svd(M)
    assert np.allclose(B @ A, (U[:, :r] * S[:r]) @ Vt[:r], atol=1e-10)
    assert abs(loss - (S[r:] ** 2).sum()) <= 1e-10 * (S ** 2).sum()


def test_p15_lore_calibration_recovers_a_rank_r_residual_exactly_and_improves_with_rank():
    rng = np.random.default_rng(22)
    n, d, r = 60, 16, 3
    H = rng.standard_normal((n, d)) * np.linspace(0.3, 2.0, d)        # anisotropic inputs
    A0, B0 = rng.standard_normal((r, d)), rng.standard_normal((d, r))
    R = (H @ A0.T) @ B0.T
    A, B, loss = oracle.lore_calibrate(H, R, r)
    assert loss <= 1e-18 * (R ** 2).sum() and np.allclose(B @ A, B0 @ A0, atol=1e-9)
    # a generic (full-rank, noisy) target: the loss falls with the rank and reaches ordinary least squares at r = d
    R = rng.standard_normal((n, d)) + H @ rng.standard_normal((d, d))
    losses = [oracle.lore_calibrate(H, R, k)[2] for k in range(1, d + 1)]
    assert all(a >= b - 1e-9 for a, b in zip(losses, losses[1:]))
    ols = float(((R - H @ np.linalg.lstsq(H, R, rcond=None)[0]) ** 2).sum())
    assert abs(losses[-1] - ols) <= 1e-9 * ols


def test_p15_lore_calibration_is_a_minimum():
    """No rank-r perturbation of the returned factors lowers the objective (first-order optimality, probed at random),
    and random rank-r maps are worse."""
    rng = np.random.default_rng(23)
    n, d, r = 50, 10, 2
    H = rng.standard_normal((n, d)) * np.linspace(0.5, 1.5, d)
    R = rng.standard_normal((n, d)) + H @ rng.standard_normal((d, d)) * 0.5
    A, B, loss = oracle.lore_calibrate(H, R, r)
    assert abs(loss - _lore_loss(H, R, A, B)) <= 1e-9 * loss
    for _ in range(200):
        dA, dB = rng.standard_normal(A.shape), rng.standard_normal(B.shape)
        for eps in (1e-3, 1e-2, 1e-1):
            assert _lore_loss(H, R, A + eps * dA, B + eps * dB) >= loss - 1e-9 * loss
    assert min(_lore_loss(H, R, rng.standard_normal(A.shape), rng.standard_normal(B.shape)) for _ in range(50)) > loss


def test_p16_prefetch_set_and_minimum_lookahead_depth():
    """Eq. 3 on a hand example, and Eq. 4 on the numbers of a worked case: 2 experts of 17.3 MB per layer over a 25 GB/s
    link need 1.384 ms; with 0.5 ms of compute per layer that is 3 layers of lookahead (2.77 -> 3), with 1.4 ms it is 1."""
    idx_hat = np.array([[[3, 1], [1, 0]], [[2, 2], [-1, -1]]])        # depth 1: tokens {3,1}, {1,0}; depth 2: {2,2}, stopped
    assert oracle.prefetch_set(idx_hat, 5).tolist() == [[1, 1, 0, 1, 0], [0, 0, 1, 0, 0]]
    assert oracle.min_lookahead_depth(2, 17.3e6, 25e9, 0.5e-3) == 3
    assert oracle.min_lookahead_depth(2, 17.3e6, 25e9, 1.4e-3) == 1
    assert oracle.min_lookahead_depth(0, 17.3e6, 25e9, 1e-3) == 0


# ---------------------------------------------------------------------------------------------------------------
# P17: the 8-bit weight format (E4M3 codes, one power-of-two scale per output row) that stands in for the paper's
# second, quantised weight precision (Sec. 5.1, Table 1).  The format's constants below are written by hand from its
# definition (1-4-3 bits, bias 7, no infinities, largest finite value 448, subnormal step 2^-9).
def test_p17_e4m3_code_values_by_hand():
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x0F: 1.875 * 2.0 ** -6, 0x30: 0.5, 0x38: 1.0,
            0x39: 1.125, 0x3F: 1.875, 0x40: 2.0, 0x44: 3.0, 0x78: 256.0, 0x7E: 448.0, 0xB8: -1.0, 0xFE: -448.0, 0x81: -2.0 ** -9}
    codes = np.array(sorted(hand), dtype=np.uint8)
    assert oracle.e4m3_decode(codes).tolist() == [hand[int(c)] for c in codes]
    assert np.isnan(oracle.e4m3_decode(np.array([0x7F, 0xFF], np.uint8))).all()
    assert np.signbit(oracle.e4m3_decode(np.array([0x80], np.uint8))[0])               # -0
    # strictly increasing in the code, and every finite code survives decode -> encode
    allc = np.arange(256, dtype=np.uint8)
    fin = allc[(allc & 0x7F) != 0x7F]
    v = oracle.e4m3_decode(fin)
    assert (np.diff(v[:127]) > 0).all() and np.array_equal(oracle.e4m3_encode(v), fin)


def test_p17_e4m3_rounding_is_nearest_even_and_saturates():
    enc = lambda *xs: oracle.e4m3_encode(np.array(xs, dtype=np.float64)).tolist()
    # halfway between 1.0 (0x38) and 1.125 (0x39): the even code 0x38; between 1.125 and 1.25 (0x3A): the even code 0x3A
    assert enc(1.0625, 1.1875, -1.0625, -1.1875) == [0x38, 0x3A, 0xB8, 0xBA]
    assert enc(1.0625 + 1e-9, 1.0625 - 1e-9, 1.1875 - 1e-9) == [0x39, 0x38, 0x39]
    # across a binade: 1.875 (0x3F) | 2.0 (0x40): halfway 1.9375 -> even code 0x40
    assert enc(1.9375, 1.93, 1.94) == [0x40, 0x3F, 0x40]
    # subnormals: half the smallest step ties to zero, one and a half steps tie to code 2
    assert enc(2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -10 + 1e-12, 2.0 ** -11) == [0x00, 0x02, 0x01, 0x00]
    # the last normal step of the subnormal range: 7/8 * 2^-6 (0x07) | 2^-6 (0x08)
    assert enc(7.5 * 2.0 ** -9) == [0x08]
    # saturation instead of NaN / infinity; NaN stays NaN
    assert enc(448.0, 449.0, 480.0, 1e30, -1e30, np.inf) == [0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0x7E]
    assert enc(np.nan) == [0x7F] and enc(-0.0) == [0x80]


def test_p17_e4m3_encode_agrees_with_the_library_cast():
    """An independent implementation of the same rounding: torch's float8_e4m3fn cast (CPU).  It does not saturate, so
    the comparison is made where no saturation occurs (|x| <= 448)."""
    import torch
    rng = np.random.default_rng(171)
    x = np.concatenate([rng.standard_normal(200000) * rng.choice([1e-3, 0.02, 1.0, 50.0, 150.0], 200000),
                        np.linspace(-448.0, 448.0, 20001), oracle.e4m3_decode(np.arange(0, 127, dtype=np.uint8)),
                        0.5 * (oracle.e4m3_decode(np.arange(0, 126, dtype=np.uint8)) + oracle.e4m3_decode(np.arange(1, 127, dtype=np.uint8)))])
    x = x[np.abs(x) <= 448.0]
    ours = oracle.e4m3_encode(x)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(ours, lib)


def test_p17_row_scales_and_round_trip():
    rng = np.random.default_rng(172)
    Wm = (rng.standard_normal((40, 256)) * 0.02 * rng.choice([1e-3, 1.0, 30.0], (40, 1))).astype(np.float32)
    Wm[3] = 0.0                               # an all-zero row
    Wm[4, :] = 0.0
    Wm[4, 7] = 448.0 * 2.0 ** -5              # row maximum exactly 448 * 2^k: the scale is 2^k, the code 0x7E
    q, s = oracle.quantize_e4m3_rows(Wm)
    assert q.shape == Wm.shape and q.dtype == np.uint8 and s.shape == (40,) and s.dtype == np.float32
    m, _ = np.frexp(s.astype(np.float64))
    assert (m == 0.5).all()                                              # powers of two
    assert s[3] == 1.0 and (q[3] & 0x7F).max() == 0 and s[4] == np.float32(2.0 ** -5) and q[4, 7] == 0x7E
    scaled_max = np.abs(Wm.astype(np.float64)).max(axis=1) / s
    nz = scaled_max > 0
    assert (scaled_max[nz] > 224.0).all() and (scaled_max[nz] <= 448.0).all()    # the largest element lands in the top binade
    back = oracle.dequantize_e4m3_rows(q, s)
    assert back.dtype == np.float32
    err = np.abs(back.astype(np.float64) - Wm)
    # nearest value: half a step of 4 significant bits where the scaled value is normal, half a subnormal step below
    bound = np.maximum(2.0 ** -4 * np.abs(Wm), 2.0 ** -10 * s[:, None])
    assert (err <= bound).all() and err.max() > 0
    # dequantised weights are a fixed point of quantise -> dequantise (the codes may move by one exponent step where a
    # row's maximum rounded down to 224 * s, which the scale rule then reads as 448 * s/2; the VALUES do not move)
    q2, s2 = oracle.quantize_e4m3_rows(back)
    assert np.array_equal(oracle.dequantize_e4m3_rows(q2, s2), back)
    assert ((s2 == s) | (s2 == s / 2)).all() and (s2 == s).sum() >= 30
    # and they are bf16 values (four significant bits times a power of two), so the GPU's bf16 kernels can take them as they are
    assert np.array_equal(W.bf16_round(back), back)
    # batched shapes quantise row by row
    q3, s3 = oracle.quantize_e4m3_rows(Wm.reshape(4, 10, 256))
    assert np.array_equal(q3.reshape(40, 256), q) and np.array_equal(s3.reshape(40), s)


def test_p17_layer_on_quantised_weights_is_the_layer_on_their_dequantised_values():
    """The layer at the second precision is defined through the same equations on s_r * q_rj; with weights that are
    already representable (scale 1) it IS the bf16 layer, and in general it stays close to it: the per-weight relative
    error of at most 2^-4 averages out over the d-term dot products."""
    wl = W.make_layer("tiny", 4, variant=17)
    s = wl.shape

    def deq(w):
        return oracle.dequantize_e4m3_rows(*oracle.quantize_e4m3_rows(w))

    kw = dict(h=wl.h, w_router=wl.w_router, lore_A=wl.lore()[0], lore_B=wl.lore()[1], resident=wl.resident, conf=wl.conf,
              top_k=s.top_k, tau=s.tau)
    base = oracle.layer(experts=[wl.expert(e) for e in range(s.n_experts)], shared=wl.shared(), **kw)
    q8 = oracle.layer(experts=[tuple(deq(w) for w in wl.expert(e)) for e in range(s.n_experts)],
                      shared=tuple(deq(w) for w in wl.shared()), **kw)
    assert np.array_equal(q8.idx, base.idx) and np.array_equal(q8.cls, base.cls) and np.array_equal(q8.gate, base.gate)
    rel = np.abs(q8.y - base.y).max() / np.abs(base.y).max()
    assert 1e-4 < rel < 0.1, rel
    # representable weights: quantisation is the identity, so the two layers coincide bit for bit
    rep = [tuple(deq(w) for w in wl.expert(e)) for e in range(s.n_experts)]
    again = oracle.layer(experts=[tuple(deq(w) for w in ws) for ws in rep], shared=tuple(deq(deq(w)) for w in wl.shared()), **kw)
    assert np.array_equal(again.y, q8.y)
