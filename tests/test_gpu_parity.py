"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Routing and classification must be bit-exact; outputs must satisfy
max|gpu - oracle| <= 1e-2 * max|oracle| + 1e-3."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21240_b200 import binding as B
from paper_2608_21240_b200 import workloads as W
from tests._cases import enforce_margins, run_oracle
from tests._gpu import (GATE_ATOL, LOGIT_ATOL, Y_ATOL, Y_RTOL, bf16_tensor, cfg_of, check_routing, upload, y_close)

pytestmark = pytest.mark.gpu

DECODE_CASES = [("tiny", 4), ("dsv2lite", 1), ("dsv2lite", 4), ("dsv2lite", 16), ("dsv2lite", 33), ("dsv2lite", 64),
                ("qwen2_57b", 1), ("qwen2_57b", 8), ("qwen2_57b", 32)]


def _layer_case(name, T, variant=0, margin=1e-3, **mk):
    wl = W.make_layer(name, T, variant=variant, **mk)
    enforce_margins(wl, margin)
    return wl


@pytest.mark.parametrize("name,T", DECODE_CASES + [("dsv2lite_prefill", 4096)])
def test_route_topk_bit_exact(name, T):
    wl = _layer_case(name, T, zipf=(name == "dsv2lite_prefill"))
    s = wl.shape
    ref_logits = oracle.router_logits(wl.h, wl.w_router)
    ref_idx, ref_gate = oracle.topk_gates(ref_logits, s.top_k, 1)
    L = B.SpiceLayer(cfg_of(s), T)
    idx, gate, logits = L.route_topk(bf16_tensor(wl.h), bf16_tensor(wl.w_router), want_logits=True)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert np.abs(gate.cpu().numpy() - ref_gate).max() <= GATE_ATOL
    assert np.abs(logits.cpu().numpy() - ref_logits).max() <= LOGIT_ATOL
    assert L.device_status() == 0
    L.close()


@pytest.mark.parametrize("N,K,d,T,norm", [(10, 3, 264, 5, 0), (64, 1, 512, 3, 1), (7, 7, 128, 2, 1),
                                           (160, 6, 1024, 70, 1), (1024, 32, 64, 3, 0)])
def test_route_topk_odd_shapes(N, K, d, T, norm):
    s = W.scaled_shape(W.SHAPES["tiny"], d=d, n_experts=N, top_k=K, n_slots=min(5, N), norm_topk=norm)
    wl = _layer_case(s, T, variant=3, margin=1e-3 if N < 1024 else 1e-5)   # 33 of 1024 logits cannot be 1e-3 apart
    ref_idx, ref_gate = oracle.topk_gates(oracle.router_logits(wl.h, wl.w_router), K, norm)
    L = B.SpiceLayer(cfg_of(s), T)
    idx, gate = L.route_topk(bf16_tensor(wl.h), bf16_tensor(wl.w_router))
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    assert np.abs(gate.cpu().numpy() - ref_gate).max() <= GATE_ATOL
    L.close()


def test_route_topk_ties_go_to_lower_index():
    s = W.scaled_shape(W.SHAPES["tiny"], d=64, n_experts=12, top_k=4)
    wr = np.zeros((12, 64), np.float32)
    wr[[1, 2, 4], 0] = 3.0       # three equal winners
    wr[5, 0] = 2.0
    h = np.zeros((2, 64), np.float32)
    h[:, 0] = 1.0
    L = B.SpiceLayer(cfg_of(s), 2)
    idx, gate = L.route_topk(bf16_tensor(h), bf16_tensor(wr))
    ref_idx, ref_gate = oracle.topk_gates(oracle.router_logits(h, wr), 4, 1)
    assert idx.cpu().numpy().tolist() == [[1, 2, 4, 5]] * 2 == ref_idx.tolist()
    assert np.abs(gate.cpu().numpy() - ref_gate).max() <= GATE_ATOL
    L.close()


@pytest.mark.parametrize("name,T", DECODE_CASES)
def test_classify_bit_exact(name, T):
    wl = _layer_case(name, T, variant=1)
    s = wl.shape
    ref = run_oracle(wl, skip_ffn=True)
    L = B.SpiceLayer(cfg_of(s), T)
    idx = torch.from_numpy(ref.idx).cuda()
    gate = torch.from_numpy(ref.gate.astype(np.float32)).cuda()
    cls, slot, counts, (rt, rk, re_, rg) = L.classify_misses(idx, gate, torch.from_numpy(wl.slot_of_expert).cuda(),
                                                             torch.from_numpy(wl.conf).cuda())
    assert np.array_equal(cls.cpu().numpy(), ref.cls)
    exp_slot = np.where(ref.cls == oracle.HIT, wl.slot_of_expert[ref.idx], -1)
    assert np.array_equal(slot.cpu().numpy(), exp_slot)
    assert counts.cpu().numpy().tolist() == ref.counts.tolist()
    n = int(ref.counts[1])
    assert np.array_equal(rt.cpu().numpy()[:n], ref.resid_tok) and np.array_equal(rk.cpu().numpy()[:n], ref.resid_k)
    assert np.array_equal(re_.cpu().numpy()[:n], ref.resid_expert)
    assert np.array_equal(rg.cpu().numpy()[:n], ref.resid_gate.astype(np.float32))
    assert L.device_status() == 0
    L.close()


def test_classify_threshold_edges_and_scalar_conf():
    s = W.scaled_shape(W.SHAPES["tiny"], n_experts=8, top_k=4, tau=0.6)
    tau = np.float32(0.6)
    idx = np.array([[0, 1, 2, 3], [4, 5, 6, 7]], np.int32)
    soe = np.array([2, -1, -1, -1, -1, 0, -1, -1], np.int32)
    conf = np.full((2, 8), 0.9, np.float32)
    conf[0, 1] = tau
    conf[0, 2] = np.nextafter(tau, np.float32(0))
    conf[0, 3] = np.nan
    conf[1, 4] = 0.0
    gate = np.full((2, 4), 0.25, np.float32)
    ref_cls, ref_counts = oracle.classify(idx, (soe >= 0).astype(np.uint8), conf, float(tau))
    L = B.SpiceLayer(cfg_of(s, tau=float(tau)), 2)
    cls, slot, counts, _ = L.classify_misses(*(torch.from_numpy(a).cuda() for a in (idx, gate, soe, conf)))
    assert cls.cpu().numpy().tolist() == ref_cls.tolist() == [[0, 1, 2, 1], [2, 0, 1, 1]]
    assert counts.cpu().numpy().tolist() == ref_counts.tolist()
    L.close()
    # one confidence per token
    L = B.SpiceLayer(cfg_of(s, tau=float(tau), conf_per_expert=False), 2)
    c1 = np.array([0.1, 0.9], np.float32)
    cls, _, _, _ = L.classify_misses(*(torch.from_numpy(a).cuda() for a in (idx, gate, soe, c1)))
    ref_cls, _ = oracle.classify(idx, (soe >= 0).astype(np.uint8), c1, float(tau))
    assert np.array_equal(cls.cpu().numpy(), ref_cls)
    L.close()


@pytest.mark.parametrize("name,T", [("tiny", 6), ("dsv2lite", 8), ("tiny", 300)])
def test_a_token_of_nans_stays_in_its_own_row(name, T):
    """Tokens are independent (Sec. 2.1: every token is routed and combined on its own).  A token whose hidden state
    is NaN selects the experts 0..K-1 (NaN never wins a comparison, equal logits go to the smaller index) and gets a
    NaN output; routing, classes and outputs of every OTHER token equal the oracle's for the clean batch.  Covers the
    fused decode kernel (every group is multiplied with all token columns) and the large-batch path (tensor-core
    router, grouped GEMMs)."""
    wl = _layer_case(name, T, variant=31)
    s = wl.shape
    ref = run_oracle(wl, want_full=False)
    bad = 2
    h = wl.h.copy()
    h[bad, :] = np.nan
    L = B.SpiceLayer(cfg_of(s), T)
    out = L.moe_layer_fwd(upload(wl), bf16_tensor(h), torch.from_numpy(wl.conf).cuda())
    torch.cuda.synchronize()
    keep = np.arange(T) != bad
    idx, cls, y = out.idx.cpu().numpy(), out.cls.cpu().numpy(), out.y.float().cpu().numpy()
    assert idx[bad].tolist() == list(range(s.top_k))
    assert np.array_equal(idx[keep], ref.idx[keep]) and np.array_equal(cls[keep], ref.cls[keep])
    assert np.isnan(y[bad]).all() and np.isfinite(y[keep]).all()
    err, bound = y_close(y[keep], ref.y[keep])
    assert err <= bound, (err, bound)
    assert L.device_status() == 0
    L.close()


def _fwd_and_check(wl, tokens=None, y_cpu=None, general_path=False, **ora):
    s = wl.shape
    ref = run_oracle(wl, tokens=tokens, **ora)
    L = B.SpiceLayer(cfg_of(s, tau=ora.get("tau"), norm_topk=ora.get("norm_topk")), wl.T)
    if general_path:
        L.set_option(B.OPT_PATH, 1)
    w = upload(wl)
    if "resident" in ora:
        raise AssertionError("change residency through wl.set_residency so the pool matches")
    conf = torch.from_numpy(np.ascontiguousarray(ora.get("conf", wl.conf))).cuda()
    out = L.moe_layer_fwd(w, bf16_tensor(wl.h), conf, y_cpu_residual=y_cpu)
    torch.cuda.synchronize()
    check_routing(out, ref, wl.T, s.top_k)
    y = out.y.float().cpu().numpy()
    if tokens is not None:
        y = y[np.asarray(tokens)]
    assert np.isfinite(y).all()
    err, bound = y_close(y, ref.y if y_cpu is None else ref.y + y_cpu.cpu().numpy()[ref.rows])
    assert err <= bound, f"max err {err:.3e} > bound {bound:.3e}"
    assert L.device_status() == 0
    return L, w, out, ref


@pytest.mark.parametrize("name,T", DECODE_CASES)
def test_moe_layer_fwd_matches_oracle(name, T):
    wl = _layer_case(name, T)
    L, w, out, ref = _fwd_and_check(wl, want_full=False)
    assert ref.counts[0] > 0
    L.close()


def _residency_with_unused_first_slots(wl, n_first):
    """Residency in which the first slots hold experts that no token of the batch routes to (as many as there are, at
    most n_first), the remaining slots experts that are used.  From the oracle's own routing."""
    s = wl.shape
    idx, _ = oracle.topk_gates(oracle.router_logits(wl.h, wl.w_router), s.top_k, s.norm_topk)
    used = np.zeros(s.n_experts, dtype=bool)
    used[np.unique(idx)] = True
    cold = [e for e in range(s.n_experts) if not used[e]][:n_first]
    hot = [e for e in range(s.n_experts) if used[e]][: s.n_slots - len(cold)]
    soe = np.full(s.n_experts, -1, dtype=np.int32)
    for sl, e in enumerate(cold + hot):
        soe[e] = sl
    wl.set_residency(soe)
    return len(cold)


@pytest.mark.parametrize("name,T,zipf", [("dsv2lite", 16, False), ("dsv2lite", 24, False), ("dsv2lite", 32, False),
                                         ("dsv2lite", 40, True), ("dsv2lite", 64, True)])
def test_slots_streamed_before_the_routing_is_known_but_chosen_by_no_token(name, T, zipf):
    """Once a slot is unlikely to go unused (16 tokens on this shape), the decode kernel streams the gate/up tiles of the
    first slots before the routing tables exist.  Here the first slots hold experts that no token chose: their tiles are computed and dropped,
    their down tiles are empty, and every output still matches the oracle."""
    wl = _layer_case(name, T, variant=9, zipf=zipf)   # (a skewed router leaves experts unused at the larger batches)
    n_cold = _residency_with_unused_first_slots(wl, 3)
    assert n_cold >= 1, "the batch uses every expert: pick another variant"
    L, w, out, ref = _fwd_and_check(wl, want_full=False)
    assert ref.counts[0] > 0
    # the same call twice more: bit-identical (the empty groups leave no state behind)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    for _ in range(2):
        again = L.moe_layer_fwd(w, h, conf)
        assert torch.equal(again.y, out.y) and torch.equal(again.cls, out.cls)
    # whatever the unused slots hold never reaches an output: NaN weights in them change nothing
    w.slot_w_gate_up[:n_cold] = float("nan")
    w.slot_w_down[:n_cold] = float("nan")
    poisoned = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert torch.equal(poisoned.y, out.y) and bool(torch.isfinite(poisoned.y.float()).all())
    assert L.device_status() == 0
    L.close()


@pytest.mark.parametrize("name,T", [("tiny", 4), ("dsv2lite", 4), ("dsv2lite", 16)])
def test_moe_layer_fwd_general_kernels_match_oracle(name, T):
    """The any-shape kernels (forced) against the oracle, and against the fused decode kernel."""
    wl = _layer_case(name, T)
    L, w, out, ref = _fwd_and_check(wl, want_full=False, general_path=True)
    n_general = L.launch_count()
    L.set_option(B.OPT_PATH, 0)
    fused = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda())
    assert L.launch_count() - n_general == 1 and n_general > 1
    assert torch.equal(fused.idx, out.idx) and torch.equal(fused.gate, out.gate) and torch.equal(fused.cls, out.cls)
    diff = (fused.y.float() - out.y.float()).abs().max().item()
    assert diff <= 1e-2 * out.y.float().abs().max().item() + 1e-3
    L.close()


@pytest.mark.parametrize("name,T", [("tiny", 4), ("dsv2lite", 1), ("dsv2lite", 16), ("qwen2_57b", 8)])
def test_mma_sync_decode_kernel_matches_oracle_and_tcgen05_kernel(name, T):
    """The mma.sync decode kernel (forced) against the oracle, and against the default tcgen05 decode kernel."""
    wl = _layer_case(name, T, variant=2)
    s = wl.shape
    ref = run_oracle(wl, want_full=False)
    L = B.SpiceLayer(cfg_of(s), T)
    w = upload(wl)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    new = L.moe_layer_fwd(w, h, conf)
    L.set_option(B.OPT_PATH, 3)
    n0 = L.launch_count()
    old = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.launch_count() - n0 == 1 and L.device_status() == 0
    for out in (new, old):
        check_routing(out, ref, T, s.top_k)
        err, bound = y_close(out.y.float().cpu().numpy(), ref.y)
        assert err <= bound, f"max err {err:.3e} > bound {bound:.3e}"
    assert torch.equal(new.idx, old.idx) and torch.equal(new.gate, old.gate) and torch.equal(new.cls, old.cls)
    L.close()


@pytest.mark.parametrize("T", [3, 5, 13, 32, 37])
def test_moe_layer_fwd_ragged_token_counts_and_dims(T):
    s = W.scaled_shape(W.SHAPES["tiny"], d=264, n_experts=10, top_k=3, inter=200, inter_shared=328, lore_rank=24,
                       n_slots=4)
    wl = _layer_case(s, T, variant=T)
    L, *_ = _fwd_and_check(wl, want_full=False)
    L.close()


@pytest.mark.parametrize("T", [16, 48])
def test_expired_dependency_wait_reports_timeout_and_recovers(T):
    """A wait that cannot be satisfied within its poll limit ends the kernel with a status, not a hang.  (48 tokens: the
    routing is spread over the grid and slots stream ahead of it, so the wait runs out with tiles in flight.)"""
    wl = _layer_case("dsv2lite", T, variant=11)
    s = wl.shape
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    good = L.moe_layer_fwd(w, h, conf)
    assert L.device_status() == 0
    L.set_option(B.OPT_SPIN_LIMIT, 1)          # one poll: the router cannot be done by then
    L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 6               # SPICE_ERR_TIMEOUT
    L.set_option(B.OPT_SPIN_LIMIT, 1 << 20)
    again = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    assert torch.equal(again.y, good.y) and torch.equal(again.idx, good.idx)
    # the kernel that gave up resets the dependency counters itself: a call that follows WITHOUT a status read in
    # between is complete and correct, and the status word still tells that an earlier call timed out
    L.set_option(B.OPT_SPIN_LIMIT, 1)
    L.moe_layer_fwd(w, h, conf)
    L.set_option(B.OPT_SPIN_LIMIT, 1 << 20)
    third = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert torch.equal(third.y, good.y) and torch.equal(third.cls, good.cls)
    assert L.device_status() == 6 and L.device_status() == 0
    L.close()


def test_expired_pipeline_wait_of_the_large_batch_gemm_reports_timeout_and_recovers():
    """The same for the grouped GEMM kernel of batches above 64 tokens: with a limit of one poll a role's wait on its
    shared-memory barrier (e.g. the tensor-core warp's wait for the first tile copy) runs out, the thread block records
    SPICE_ERR_TIMEOUT, lets its copies and MMAs in flight finish, frees its TMEM and returns; nothing hangs, and the
    next call with the default limit gives the first call's bits."""
    wl = _layer_case("tiny", 200, variant=12)
    s = wl.shape
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    good = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    L.set_option(B.OPT_TC_WAIT_LIMIT, 1)
    L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 6               # SPICE_ERR_TIMEOUT
    L.set_option(B.OPT_TC_WAIT_LIMIT, 1 << 22)
    again = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    assert torch.equal(again.y, good.y) and torch.equal(again.idx, good.idx) and torch.equal(again.cls, good.cls)
    L.close()


def test_moe_layer_fwd_degenerate_residency():
    s = W.SHAPES["tiny"]
    # all hit
    wl = _layer_case(W.scaled_shape(s, n_slots=8), 4, variant=5)
    L, w, out, ref = _fwd_and_check(wl, want_full=False)
    assert ref.counts.tolist() == [8, 0, 0]
    L.close()
    # nothing resident: all misses, mixed low-confidence / exact
    wl = _layer_case(s, 4, variant=6, n_resident=0)
    L, w, out, ref = _fwd_and_check(wl, want_full=False)
    assert ref.counts[0] == 0 and ref.counts[1] > 0 and ref.counts[2] > 0
    L.close()
    # all misses low-confidence (tau > 1) and all exact (tau = 0)
    for tau in (1.5, 0.0):
        wl = _layer_case(s, 4, variant=7, n_resident=0)
        L, w, out, ref = _fwd_and_check(wl, want_full=False, tau=tau)
        assert ref.counts[2 if tau > 1 else 1] == 8
        L.close()


def test_moe_layer_fwd_unnormalised_gates_and_cpu_residual_and_resid_stream():
    wl = _layer_case("tiny", 4, variant=8)
    s = wl.shape
    ref = run_oracle(wl, want_full=True, norm_topk=0)
    # exact-recovery outputs computed elsewhere are merged by the layer call
    y_cpu = torch.from_numpy((ref.y_full - ref.y).astype(np.float32)).cuda()
    L = B.SpiceLayer(cfg_of(s, norm_topk=0), wl.T)
    w = upload(wl)
    x0 = torch.randn(wl.T, s.d, device="cuda").bfloat16()
    x = x0.clone()
    out = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda(), y_cpu_residual=y_cpu, x_resid=x)
    check_routing(out, ref, wl.T, s.top_k)
    err, bound = y_close(out.y.float().cpu().numpy(), ref.y_full)
    assert err <= bound
    errx, boundx = y_close(x.float().cpu().numpy(), x0.float().cpu().numpy().astype(np.float64) + ref.y_full)
    assert errx <= boundx + 2e-2    # bf16 rounding of the O(1) residual stream
    L.close()


@pytest.mark.parametrize("T", [7, 17, 48])
def test_tcgen05_decode_kernel_all_token_widths_scalar_conf_full_softmax_and_residuals(T):
    """The tcgen05 decode kernel at 16, 32 and 64 token columns, on a shape with ragged tiles (I = 192: 3 gate/up
    tiles; I_s = 320; r = 24 on plain maps), one confidence per token, full-softmax gates, CPU residual and residual stream."""
    s = W.scaled_shape(W.SHAPES["tiny"], d=320, n_experts=12, top_k=3, inter=192, inter_shared=320, lore_rank=24,
                       n_slots=5)
    wl = _layer_case(s, T, variant=20 + T)
    conf1 = np.ascontiguousarray(wl.conf[:, 0])
    ref = run_oracle(wl, want_full=True, norm_topk=0, conf=conf1)
    y_cpu = torch.from_numpy((ref.y_full - ref.y).astype(np.float32)).cuda()
    L = B.SpiceLayer(cfg_of(s, norm_topk=0, conf_per_expert=False), T)
    w = upload(wl)
    x0 = torch.randn(T, s.d, device="cuda").bfloat16()
    x = x0.clone()
    n0 = L.launch_count()
    out = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(conf1).cuda(), y_cpu_residual=y_cpu, x_resid=x)
    torch.cuda.synchronize()
    assert L.launch_count() - n0 == 1 and L.device_status() == 0
    check_routing(out, ref, T, s.top_k)
    err, bound = y_close(out.y.float().cpu().numpy(), ref.y_full)
    assert err <= bound, f"max err {err:.3e} > bound {bound:.3e}"
    errx, boundx = y_close(x.float().cpu().numpy(), x0.float().cpu().numpy().astype(np.float64) + ref.y_full)
    assert errx <= boundx + 2e-2    # bf16 rounding of the O(1) residual stream
    # the general kernels agree on every routing decision
    L.set_option(B.OPT_PATH, 1)
    gen = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(conf1).cuda(), y_cpu_residual=y_cpu)
    assert L.launch_count() - n0 > 2
    assert torch.equal(gen.idx, out.idx) and torch.equal(gen.gate, out.gate) and torch.equal(gen.cls, out.cls)
    L.close()


@pytest.mark.parametrize("name,T", [("tiny", 4), ("dsv2lite", 16), ("qwen2_57b", 8), ("dsv2lite", 300)])
def test_draft_confidence_matches_oracle_and_feeds_the_layer(name, T):
    """Sec. 4.1, Eq. 2 and Eq. 5: predicted set bit-exact, confidence and distribution within fp32 rounding; the
    confidences are accepted by the layer call in both layouts."""
    wl = _layer_case(name, T, variant=31)
    s = wl.shape
    logits = oracle.router_logits(wl.h, wl.w_router)
    ref_idx, ref_pi, ref_conf = oracle.draft_confidence(logits, s.top_k)
    L = B.SpiceLayer(cfg_of(s), T)
    h, wr = bf16_tensor(wl.h), bf16_tensor(wl.w_router)
    idx, conf, pi = L.draft_confidence(h, wr, want_pi=True)
    idx2, conf2 = L.draft_confidence(h, wr)
    torch.cuda.synchronize()
    assert np.array_equal(idx.cpu().numpy(), ref_idx) and torch.equal(idx, idx2) and torch.equal(conf, conf2)
    assert np.abs(conf.cpu().numpy().astype(np.float64) - ref_conf).max() <= s.top_k * GATE_ATOL
    assert np.abs(pi.cpu().numpy().astype(np.float64) - ref_pi).max() <= GATE_ATOL
    # the router of Eq. 1 on the same inputs selects the same experts; its un-normalised gates are pi_hat's entries
    Lf = B.SpiceLayer(cfg_of(s, norm_topk=0), T)
    ridx, rgate = Lf.route_topk(h, wr)
    assert torch.equal(ridx, idx) and torch.equal(rgate, torch.gather(pi, 1, idx.long()))
    Lf.close()
    if T <= 64:
        # per-token confidence and per-(token, expert) probabilities as the `conf` input of the layer
        w = upload(wl)
        ref1 = run_oracle(wl, want_full=False, conf=conf.cpu().numpy())    # the same fp32 numbers decide on both sides
        L1 = B.SpiceLayer(cfg_of(s, conf_per_expert=False), T)
        out1 = L1.moe_layer_fwd(w, h, conf)
        assert np.array_equal(out1.cls.cpu().numpy(), ref1.cls)
        L1.close()
        out2 = L.moe_layer_fwd(w, h, pi)
        ref2 = run_oracle(wl, want_full=False, conf=pi.cpu().numpy())
        assert np.array_equal(out2.cls.cpu().numpy(), ref2.cls)
    L.close()


def _rollout_case(shape, T, L, variant, l_min):
    """Layers of depths 1..L from the seeded generator, a threshold that splits the tokens, and a check (through the
    oracle) that every decision the rollout takes has a margin that rounding cannot cross: 1e-3 between logits at depth 1
    (fp32 summation order), 5e-3 at later depths and 1e-3 between a confidence and the threshold (the draft state is bf16
    and the GPU also rounds the intermediate activations to bf16, which moves later logits by up to ~1e-3)."""
    for v in range(variant, variant + 300):
        wls = [W.make_layer(shape, T, variant=v, layer=l) for l in range(L)]
        enforce_margins(wls[0])
        layers = [dict(w_router=wl.w_router, shared=wl.shared(), lore_A=wl.lore()[0], lore_B=wl.lore()[1]) for wl in wls]
        x = wls[0].h
        _, conf0, _, _ = oracle.prefetch_rollout(x, layers, shape.top_k, l_min, L, 0.0)
        cs = np.sort(conf0[l_min - 1:].ravel())
        tau = float(0.5 * (cs[cs.size // 2 - 1] + cs[cs.size // 2]))      # between two observed confidences
        ok = np.abs(conf0 - tau).min() > 1e-3
        for l in range(1, L + 1):
            _, _, depth, h_prev = oracle.prefetch_rollout(x, layers[:l], shape.top_k, min(l_min, l), l, tau)
            lg = np.sort(oracle.router_logits(h_prev.astype(np.float32), layers[l - 1]["w_router"]), axis=1)[:, ::-1]
            gaps = (lg[:, :shape.top_k] - lg[:, 1:shape.top_k + 1]).min(axis=1)
            ok = ok and bool((gaps[depth == l] >= (1e-3 if l == 1 else 5e-3)).all())
        if ok:
            return wls, layers, x, tau
    raise AssertionError("no variant with safe margins found")


@pytest.mark.parametrize("name,T,L,l_min", [("tiny", 6, 3, 1), ("tiny", 9, 4, 2), ("dsv2lite", 4, 3, 2)])
def test_prefetch_rollout_matches_oracle(name, T, L, l_min):
    """Algorithm 1: predicted sets and halting depths bit-exact, confidences within fp32 rounding, the draft state after
    the last projection within the output tolerance."""
    s = W.SHAPES[name]
    wls, layers, x, tau = _rollout_case(s, T, L, 40, l_min)
    ref_idx, ref_conf, ref_depth, ref_h = oracle.prefetch_rollout(x, layers, s.top_k, l_min, L, tau)
    assert len(set(ref_depth.tolist())) > 1, "the threshold should stop some tokens early"
    Lyr = B.SpiceLayer(cfg_of(s), T)
    ws = [upload(wl) for wl in wls]
    n0 = Lyr.launch_count()
    idx, conf, depth, h_final = Lyr.prefetch_rollout(ws, bf16_tensor(x), l_min, L, tau)
    torch.cuda.synchronize()
    # one fused launch per projecting depth + the last depth's router, confidence and halting kernels + the prefetch set
    assert Lyr.device_status() == 0 and Lyr.launch_count() - n0 == (L - 1) + 3 + 1
    assert np.array_equal(depth.cpu().numpy(), ref_depth)
    assert np.array_equal(idx.cpu().numpy(), ref_idx)
    dconf = np.abs(conf.cpu().numpy().astype(np.float64) - ref_conf)
    assert dconf[0].max() <= s.top_k * GATE_ATOL and dconf.max() <= 1e-3      # later depths inherit the bf16 state's rounding
    err, bound = y_close(h_final.float().cpu().numpy(), ref_h)
    assert err <= bound + 2e-2, f"max err {err:.3e}"      # + bf16 rounding of the O(1) state
    # Eq. 3: the per-depth union of the predicted sets
    assert np.array_equal(Lyr.prefetch_mask.cpu().numpy(), oracle.prefetch_set(ref_idx, s.n_experts))
    # depth 1 is the draft-confidence call
    i1, c1 = Lyr.draft_confidence(bf16_tensor(x), ws[0].w_router)
    assert torch.equal(i1, idx[0]) and torch.equal(c1, conf[0])
    # the same rollout on the general-shape kernels
    Lyr.set_option(B.OPT_PATH, 1)
    n1 = Lyr.launch_count()
    gidx, gconf, gdepth, gh = Lyr.prefetch_rollout(ws, bf16_tensor(x), l_min, L, tau)
    torch.cuda.synchronize()
    assert Lyr.launch_count() - n1 == 3 * L + 5 * (L - 1) + 1
    assert torch.equal(gidx, idx) and torch.equal(gdepth, depth)
    assert (gconf[0] - conf[0]).abs().max().item() <= s.top_k * GATE_ATOL and (gconf - conf).abs().max().item() <= 1e-3
    err, bound = y_close(gh.float().cpu().numpy(), ref_h)
    assert err <= bound + 2e-2
    Lyr.set_option(B.OPT_PATH, 0)
    # argument errors launch nothing
    with pytest.raises(B.SpiceError):
        Lyr.prefetch_rollout(ws, bf16_tensor(x), L + 1, L, tau)
    Lyr.close()


@pytest.mark.parametrize("name,T", [("dsv2lite", 4), ("tiny", 200)])
def test_split_exports_compose_to_the_fused_call(name, T):
    """The four split exports applied in turn give the fused call's result: on a decode batch (fused decode kernel
    against the general kernels) and on a batch above 64 tokens (both sides on the tensor-core kernels)."""
    wl = _layer_case(name, T, variant=2)
    s = wl.shape
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h = bf16_tensor(wl.h)
    conf = torch.from_numpy(wl.conf).cuda()
    fused = L.moe_layer_fwd(w, h, conf)
    idx, gate = L.route_topk(h, w.w_router)
    cls, slot, counts, resid = L.classify_misses(idx, gate, w.slot_of_expert, conf)
    assert torch.equal(idx, fused.idx) and torch.equal(cls, fused.cls) and torch.equal(counts, fused.counts)
    if T <= 64:
        assert torch.equal(gate, fused.gate)          # same logit arithmetic on both sides
    else:
        assert (gate - fused.gate).abs().max().item() <= 7e-5   # the fused call's logits come from the tensor cores
    y = torch.zeros(wl.T, s.d, device="cuda")
    L.grouped_expert_ffn(w, h, idx, gate, cls, slot, y)
    y_hit = y.clone()
    L.lore_surrogate(w, h, idx, gate, cls, y)
    torch.cuda.synchronize()
    ref = run_oracle(wl, want_full=False)
    err, bound = y_close(y.cpu().numpy(), ref.y)
    assert err <= bound
    assert (y.bfloat16().float() - fused.y.float()).abs().max().item() <= Y_RTOL * fused.y.float().abs().max().item() + Y_ATOL
    # the routed part alone: oracle with the shared/LoRE part removed = hits only
    hits_only = np.zeros_like(ref.y)
    for t in range(wl.T):
        for k in range(s.top_k):
            if ref.cls[t, k] == oracle.HIT:
                e = int(ref.idx[t, k])
                hits_only[t] += ref.gate[t, k] * oracle.swiglu_ffn(*wl.expert(e), wl.h[t])
    err, bound = y_close(y_hit.cpu().numpy(), hits_only)
    assert err <= bound
    L.close()


def test_batch_independence_and_repeatability():
    wl = _layer_case("dsv2lite", 16, variant=4)
    s = wl.shape
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h = bf16_tensor(wl.h)
    conf = torch.from_numpy(wl.conf).cuda()
    a = L.moe_layer_fwd(w, h, conf)
    b = L.moe_layer_fwd(w, h, conf)
    assert torch.equal(a.y, b.y), "two runs on the same inputs must be bit-identical"
    for t in (0, 7, 15):
        one = L.moe_layer_fwd(w, h[t:t + 1].contiguous(), conf[t:t + 1].contiguous())
        assert torch.equal(one.idx[0], a.idx[t]) and torch.equal(one.cls[0], a.cls[t])
        diff = (one.y[0].float() - a.y[t].float()).abs().max().item()
        assert diff <= 1e-2 * a.y[t].float().abs().max().item() + 1e-3
    L.close()


@pytest.mark.parametrize("T", [1, 4, 16, 64])
def test_repeated_calls_over_rotating_weight_sets_are_bit_identical(T):
    """240 back-to-back layer calls that rotate through 4 independent weight sets (2.6 GB, so every call streams its
    weights from HBM with a cold L2, as in a decode loop): every output of every later pass equals the first pass bit
    for bit.  Inside the fused decode kernel the activations of a group are written by ordinary stores of one CTA and
    fetched by TMA copies of others, ordered by a release / acquire pair on the group's counter and a proxy fence on the
    reader's side; a gap in that ordering would show here as a rare stale tile."""
    s = W.SHAPES["dsv2lite"]
    sets = [W.make_layer(s, T, variant=300 + i) for i in range(4)]
    ws = [upload(wl) for wl in sets]
    structs = [w.c_struct() for w in ws]
    L = B.SpiceLayer(cfg_of(s), T)
    h, conf = bf16_tensor(sets[0].h), torch.from_numpy(sets[0].conf).cuda()
    n_pass = 60
    ys = torch.empty(n_pass, 4, T, s.d, dtype=torch.bfloat16, device="cuda")
    idx = torch.empty(n_pass, 4, T, s.top_k, dtype=torch.int32, device="cuda")
    cls = torch.empty(n_pass, 4, T, s.top_k, dtype=torch.uint8, device="cuda")
    st = torch.cuda.current_stream()
    n0 = L.launch_count()
    for p in range(n_pass):
        for i in range(4):
            B.spice_moe_layer_fwd(L.ctx, structs[i], h, conf, T, ys[p, i], idx=idx[p, i], cls=cls[p, i], stream=st)
    torch.cuda.synchronize()
    assert L.device_status() == 0 and L.launch_count() - n0 == 4 * n_pass     # one fused kernel per call
    assert bool(torch.isfinite(ys[0].float()).all()) and int((cls[0] == 0).sum()) > 0
    assert not torch.equal(ys[0, 0], ys[0, 1])                                   # the sets really differ
    same = (ys == ys[0:1]).flatten(1).all(dim=1)
    assert bool(same.all()), f"passes that differ from the first: {torch.nonzero(~same).flatten().tolist()[:10]}"
    assert bool((idx == idx[0:1]).all()) and bool((cls == cls[0:1]).all())
    L.close()


@pytest.mark.parametrize("name,T", [("dsv2lite", 8), ("tiny", 150)])
def test_layer_calls_replay_from_a_cuda_graph(name, T):
    """Three layer calls (residual stream updated in place) captured into one CUDA graph and replayed: same bits as the
    eager calls.  The calls make no host synchronisation and take every pointer at call time.  Batch 8: the fused decode
    kernel.  Batch 150: the large-batch path, whose shared expert and LoRE groups run on the context's side stream
    (the fork and the join are captured as edges of the graph)."""
    s = W.SHAPES[name]
    wls = [W.make_layer(s, T, variant=200 + i) for i in range(3)]
    ws = [upload(wl) for wl in wls]
    structs = [w.c_struct() for w in ws]
    L = B.SpiceLayer(cfg_of(s), T)
    h, conf = bf16_tensor(wls[0].h), torch.from_numpy(wls[0].conf).cuda()
    ys = [torch.empty(T, s.d, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    x = torch.zeros(T, s.d, dtype=torch.bfloat16, device="cuda")

    def run():
        for i in range(3):
            B.spice_moe_layer_fwd(L.ctx, structs[i], h, conf, T, ys[i], x_resid=x, stream=torch.cuda.current_stream())

    run()
    torch.cuda.synchronize()
    ref, xref = [y.clone() for y in ys], x.clone()
    x.zero_()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(g, stream=side):
        run()
    for _ in range(2):
        x.zero_()
        for y in ys:
            y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert all(torch.equal(a, b) for a, b in zip(ys, ref)) and torch.equal(x, xref)
    assert L.device_status() == 0
    L.close()


def test_zero_tokens_and_argument_errors():
    s = W.SHAPES["tiny"]
    wl = W.make_layer(s, 4)
    L = B.SpiceLayer(cfg_of(s), 4)
    w = upload(wl)
    h0 = torch.empty(0, s.d, dtype=torch.bfloat16, device="cuda")
    c0 = torch.empty(0, s.n_experts, device="cuda")
    out = L.moe_layer_fwd(w, h0, c0)
    assert out.counts.cpu().tolist() == [0, 0, 0] and L.launch_count() == 0
    with pytest.raises(B.SpiceError):   # more tokens than the ctx was created for
        L.moe_layer_fwd(w, bf16_tensor(np.zeros((5, s.d), np.float32)), torch.zeros(5, s.n_experts, device="cuda"))
    with pytest.raises(B.SpiceError):   # misaligned activation pointer
        buf = torch.zeros(4 * s.d + 8, dtype=torch.bfloat16, device="cuda")
        L.moe_layer_fwd(w, buf[1:1 + 4 * s.d].view(4, s.d), torch.zeros(4, s.n_experts, device="cuda"))
    with pytest.raises(B.SpiceError):
        B.SpiceLayer(cfg_of(W.scaled_shape(s, d=100)), 4)      # d not a multiple of 8
    with pytest.raises(B.SpiceError):
        B.SpiceLayer(cfg_of(W.scaled_shape(s, top_k=9)), 4)    # K > N
    L.close()


def test_corrupt_slot_table_sets_status_without_faulting():
    wl = _layer_case("tiny", 4, variant=9)
    s = wl.shape
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    ref = run_oracle(wl, skip_ffn=True)
    e_bad = int(ref.idx[0, 0])
    w.slot_of_expert[e_bad] = s.n_slots + 3          # points outside the pool
    out = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda())
    torch.cuda.synchronize()
    assert L.device_status() == 5                    # SPICE_ERR_BAD_TABLE, sticky until read
    assert L.device_status() == 0
    cls = out.cls.cpu().numpy()
    assert (cls[ref.idx == e_bad] == B.MISS_EXACT).all()
    assert torch.isfinite(out.y.float()).all()
    L.close()


def _config4_sample(idx, n_experts, n_random=64, seed=4):
    """Tokens for the oracle at 4096 tokens, chosen from the ORACLE's routing so that every expert's row range is looked
    at from both ends: per expert its first and its last token (the first and the last 128-row tile of its group hold
    them whenever the group is laid out in token order), one token out of every 128 of its list (a group of m tokens
    spans ceil(m / 128) tiles), every token of an expert that has at most four, plus random tokens."""
    rng = np.random.default_rng(seed)
    T = idx.shape[0]
    pick = set(rng.choice(T, size=n_random, replace=False).tolist())
    for e in range(n_experts):
        toks = np.nonzero((idx == e).any(axis=1))[0]
        if toks.size == 0:
            continue
        pick.update(toks[::128].tolist())
        pick.update((int(toks[0]), int(toks[-1])))
        if toks.size <= 4:
            pick.update(toks.tolist())
    return sorted(pick)


def test_config4_prefill_4096_tokens_skewed_loads_sampled_against_oracle():
    """DeepSeek-V2-Lite-shaped layer, 4096 tokens, Zipf-skewed router, every expert resident.
    Routing / classification are compared for all tokens.  Outputs: against the oracle on a sample that touches both
    ends and every 128th row of every expert's group, and -- because the grouping of such batches places rows by
    atomics, so that no host-side choice can name the tile a token lands in -- ALL 4096 tokens of the tensor-core path
    against the general-shape kernels (GPU against GPU at the output tolerance), which therefore covers every 128-row
    tile of every group, the last partial tile of the hottest expert and the smallest group included."""
    wl = _layer_case("dsv2lite_prefill", 4096, zipf=True)
    s = wl.shape
    pre = run_oracle(wl, skip_ffn=True)
    tokens = _config4_sample(pre.idx, s.n_experts)
    assert 150 <= len(tokens) <= 400
    ref = run_oracle(wl, tokens=tokens, want_full=False)
    load = np.bincount(ref.idx.ravel(), minlength=s.n_experts)
    assert load.max() > 8 * max(1, load.min())            # loads really are imbalanced
    assert load.max() > 3000 and load.min() < 128          # a group of dozens of tiles and one smaller than a tile
    assert ref.counts.tolist() == [4096 * s.top_k, 0, 0]
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    n0 = L.launch_count()
    out = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    n_tc = L.launch_count() - n0
    check_routing(out, ref, wl.T, s.top_k)
    y = out.y.float().cpu().numpy()
    assert np.isfinite(y).all()
    err, bound = y_close(y[np.asarray(tokens)], ref.y)
    assert err <= bound, (err, bound)
    assert L.device_status() == 0
    # every token, every tile: the same call on the general-shape kernels
    L.set_option(B.OPT_PATH, 1)
    gen = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    assert L.device_status() == 0 and L.launch_count() - n0 - n_tc > 0
    assert torch.equal(gen.idx, out.idx) and torch.equal(gen.cls, out.cls)
    yg = gen.y.float().cpu().numpy()
    errg, boundg = y_close(yg[np.asarray(tokens)], ref.y)
    assert errg <= boundg, (errg, boundg)
    diff = np.abs(yg - y).max(axis=1)
    assert diff.max() <= Y_RTOL * np.abs(yg).max() + Y_ATOL, (int(diff.argmax()), float(diff.max()))
    L.close()


def test_large_batch_with_misses_multi_cta_tables_sampled_against_oracle():
    """3000 tokens of the small layer with 5 of 8 experts resident: 6000 (token, expert) entries take the multi-CTA
    classification / grouping kernels, and every class occurs.  Routing, classes, counts and the ORDERED residual-miss list
    are compared for all tokens (also through the split exports), outputs for a sample."""
    wl = _layer_case("tiny", 3000, variant=13)
    s = wl.shape
    tokens = sorted(np.random.default_rng(5).choice(3000, size=40, replace=False).tolist())
    ref = run_oracle(wl, tokens=tokens, want_full=False)
    assert min(ref.counts.tolist()) > 200
    L = B.SpiceLayer(cfg_of(s), wl.T)
    w = upload(wl)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    out = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    check_routing(out, ref, wl.T, s.top_k)
    err, bound = y_close(out.y.float().cpu().numpy()[np.asarray(tokens)], ref.y)
    assert err <= bound, (err, bound)
    idx, gate = L.route_topk(h, w.w_router)
    cls, slot, counts, resid = L.classify_misses(idx, gate, w.slot_of_expert, conf)
    assert torch.equal(cls, out.cls) and torch.equal(counts, out.counts)
    n_miss = int(counts[1].item())
    assert torch.equal(resid[0][:n_miss], out.resid_tok[:n_miss]) and torch.equal(resid[2][:n_miss], out.resid_expert[:n_miss])
    # the general kernels on the tables the multi-CTA grouping built
    L.set_option(B.OPT_PATH, 1)
    gen = L.moe_layer_fwd(w, h, conf)
    assert (gen.y.float() - out.y.float()).abs().max().item() <= Y_RTOL * out.y.float().abs().max().item() + Y_ATOL
    assert L.device_status() == 0
    L.close()


def test_config5_decode_stack_teacher_forced_per_layer():
    """26 layers of DeepSeek-V2-Lite shape, batch 8, slot cache of 26 experts with ~70 % hits.  Each GPU layer
    call gets the oracle chain's input for that layer (bf16-level output error must not be allowed to flip later
    routing decisions), the exact-recovery outputs as y_cpu_residual, and the residual stream to update."""
    from tests._cases import STACK_LAYERS, stack_layer
    s = W.SHAPES["dsv2lite_stack"]
    T = 8
    x = W.make_layer(s, T, variant=55).h.astype(np.float64)          # embedding-like start of the stream
    L = B.SpiceLayer(cfg_of(s), T)
    tot = np.zeros(3, np.int64)
    for l in range(STACK_LAYERS):
        wl, ref, _ = stack_layer(l, x, T)
        need = {int(e) for e, c in zip(ref.idx.ravel(), ref.cls.ravel()) if c == oracle.HIT}
        w = upload(wl, only=need)
        y_cpu = torch.from_numpy((ref.y_full - ref.y).astype(np.float32)).cuda()
        xr = bf16_tensor(W.bf16_round(x.astype(np.float32)))
        out = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda(), y_cpu_residual=y_cpu, x_resid=xr)
        torch.cuda.synchronize()
        check_routing(out, ref, T, s.top_k)
        err, bound = y_close(out.y.float().cpu().numpy(), ref.y_full)
        assert err <= bound, (l, err, bound)
        x_next = x + ref.y_full
        errx = np.abs(xr.float().cpu().numpy() - x_next).max()
        assert errx <= 1e-2 * np.abs(x_next).max() + 1e-3 + 2.0 ** -8 * np.abs(x_next).max()   # + bf16 rounding of x
        tot += ref.counts
        x = x_next
        del w
    hit_rate = tot[0] / tot.sum()
    assert 0.6 <= hit_rate <= 0.85 and tot[1] > 0 and tot[2] > 0
    assert L.device_status() == 0
    L.close()


@pytest.mark.parametrize("T,dims", [
    (300, {}),                                                                   # tiny shape, several tokens per expert
    (200, dict(d=264, n_experts=10, top_k=3, inter=200, inter_shared=328, lore_rank=24, n_slots=4)),   # ragged tiles
    (1000, dict(d=512, n_experts=16, top_k=4, inter=384, inter_shared=768, lore_rank=32, n_slots=9)),
])
def test_tensor_core_path_matches_oracle_and_general_path(T, dims):
    """Batches beyond the decode kernel run the exact experts on the tcgen05 grouped GEMM; same answers as
    the oracle (sampled tokens) and as the general-shape kernels (all tokens)."""
    s = W.scaled_shape(W.SHAPES["tiny"], **dims) if dims else W.SHAPES["tiny"]
    wl = _layer_case(s, T, variant=31)
    tokens = sorted(np.random.default_rng(T).choice(T, size=16, replace=False).tolist())
    L, w, out, ref = _fwd_and_check(wl, tokens=tokens, want_full=False)
    assert ref.counts[0] > 0 and ref.counts[2] > 0
    n_tc = L.launch_count()
    L.set_option(B.OPT_PATH, 1)
    gen = L.moe_layer_fwd(w, bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda())
    torch.cuda.synchronize()
    assert torch.equal(gen.idx, out.idx) and torch.equal(gen.cls, out.cls)
    diff = (gen.y.float() - out.y.float()).abs().max().item()
    assert diff <= 1e-2 * gen.y.float().abs().max().item() + 1e-3, diff
    assert L.device_status() == 0 and n_tc > 0
    L.close()
