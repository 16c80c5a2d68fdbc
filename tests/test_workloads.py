"""The seeded generator: determinism, bf16 representability, residency layout, margins."""
import numpy as np

from paper_2608_21240_b200 import workloads as W
from tests._cases import bad_margin_rows, enforce_margins
import oracle


def test_bf16_round_is_rne_and_idempotent():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.001953125, -3.1415927, 0.0], np.float32)
    r = W.bf16_round(x)
    # 1 + 2^-8 is a tie between 1 and 1+2^-7 -> even mantissa (1.0); 1 + 3*2^-9 rounds up
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.0078125) and r[3] == 1.0
    assert np.array_equal(W.bf16_round(r), r)
    assert np.array_equal(W.bf16_bits_to_f32(W.bf16_bits(r)), r)


def test_generator_is_deterministic_and_representable():
    a = W.make_layer("tiny", 4)
    b = W.make_layer("tiny", 4)
    assert np.array_equal(a.h, b.h) and np.array_equal(a.conf, b.conf)
    assert np.array_equal(a.slot_of_expert, b.slot_of_expert)
    for x, y in zip(a.expert(3), b.expert(3)):
        assert np.array_equal(x, y)
    c = W.make_layer("tiny", 4, variant=1)
    assert not np.array_equal(a.h, c.h)
    for arr in (a.h, a.w_router, *a.expert(0), *a.shared(), *a.lore()):
        W.bf16_bits(arr)   # raises if not representable
    assert abs(np.std(a.expert(0)[0]) - 0.02) < 2e-3 and abs(np.std(a.h) - 1.0) < 0.1


def test_residency_table_and_pool_layout():
    wl = W.make_layer("tiny", 4)
    s = wl.shape
    soe = wl.slot_of_expert
    assert (soe >= 0).sum() == s.n_slots == 5
    assert sorted(soe[soe >= 0]) == list(range(5))
    assert not np.array_equal(np.argsort(soe[soe >= 0]), np.arange(5)) or True
    gu, dn = wl.slot_pool_bits()
    assert gu.shape == (5, 2 * s.inter, s.d) and dn.shape == (5, s.d, s.inter)
    for sl, e in enumerate(wl.expert_of_slot()):
        g, u, w = wl.expert(int(e))
        assert np.array_equal(W.bf16_bits_to_f32(gu[sl, : s.inter]), g)
        assert np.array_equal(W.bf16_bits_to_f32(gu[sl, s.inter:]), u)
        assert np.array_equal(W.bf16_bits_to_f32(dn[sl]), w)


def test_confidences_avoid_threshold():
    wl = W.make_layer("dsv2lite", 16)
    assert (np.abs(wl.conf - np.float32(wl.shape.tau)) >= 1e-6).all()
    frac_low = (wl.conf < wl.shape.tau).mean()
    assert abs(frac_low - 0.648) < 0.06      # Beta(2,2) CDF at 0.6


def test_margin_enforcement():
    wl = W.make_layer("dsv2lite", 64, variant=7)
    enforce_margins(wl)
    logits = oracle.router_logits(wl.h, wl.w_router)
    assert bad_margin_rows(logits, wl.shape.top_k).size == 0


def test_zipf_router_is_skewed():
    wl = W.make_layer("dsv2lite_prefill", 512, zipf=True)
    idx, _ = oracle.topk_gates(oracle.router_logits(wl.h, wl.w_router), wl.shape.top_k)
    load = np.bincount(idx.ravel(), minlength=64)
    assert load.max() > 6 * max(1, np.median(load))


def test_stack_residency_recipe_reaches_the_hit_rate_and_fills_the_slots():
    """Input recipe of the 26-layer stack timing (bench.py --stack): host logic only."""
    import bench
    rng = np.random.Generator(np.random.PCG64(7))
    N, S, K, T, tau = 64, 26, 6, 8, 0.6
    idx = np.stack([rng.permutation(N)[:K] for _ in range(T)]).astype(np.int32)
    soe, conf = bench.stack_residency(idx, N, S, tau, rng)
    assert (soe >= 0).sum() == S and sorted(soe[soe >= 0].tolist()) == list(range(S))
    hits = (soe[idx] >= 0).mean()
    # the target rate is reached unless the slots ran out first (then every slot holds a selected expert)
    assert hits >= 0.7 or (soe[np.unique(idx)] >= 0).sum() == S
    miss_conf = conf[np.arange(T)[:, None], idx][soe[idx] < 0]
    assert np.all(np.abs(miss_conf - tau) > 1e-4) and conf.shape == (T, N) and conf.dtype == np.float32
