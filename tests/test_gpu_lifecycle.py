"""Context life cycle and call mixing: contexts are created and destroyed repeatedly without leaking device memory, one
context serves 16-bit and 8-bit calls of different batch sizes in any order, and calls on a non-default stream give the
default stream's bits."""
import numpy as np
import pytest
import torch

from paper_2608_21240_b200 import binding as B
from paper_2608_21240_b200 import workloads as W
from tests._gpu import bf16_tensor, cfg_of, upload

pytestmark = pytest.mark.gpu


def test_create_destroy_does_not_leak_device_memory():
    s = W.SHAPES["dsv2lite"]
    torch.cuda.synchronize()
    L = B.SpiceLayer(cfg_of(s), 64)
    ws = B.spice_workspace_bytes(L.ctx)
    L.close()
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(40):
        L = B.SpiceLayer(cfg_of(s), 64)
        L.close()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert ws > 0 and free0 - free1 < ws // 2, (free0, free1, ws)


def test_one_context_serves_mixed_calls_in_any_order():
    s = W.SHAPES["dsv2lite"]
    wl = W.make_layer(s, 40, variant=500)
    w16 = upload(wl)
    w8 = B.quantize_layer(w16)
    L = B.SpiceLayer(cfg_of(s), 200)
    h_all, conf_all = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()

    def run(kind, T):
        h, conf = h_all[:T].contiguous(), conf_all[:T].contiguous()
        out = (L.moe_layer_fwd_fp8 if kind == 8 else L.moe_layer_fwd)(w8 if kind == 8 else w16, h, conf)
        return out.y.clone(), out.idx.clone(), out.cls.clone()

    plan = [(16, 1), (8, 1), (16, 16), (8, 16), (16, 40), (8, 27), (16, 3), (8, 3)]
    first = {}
    for kind, T in plan:
        first[(kind, T)] = run(kind, T)
    torch.cuda.synchronize()
    assert L.device_status() == 0
    rng = np.random.default_rng(7)
    for _ in range(3):
        for j in rng.permutation(len(plan)):
            kind, T = plan[j]
            y, idx, cls = run(kind, T)
            ref = first[(kind, T)]
            assert torch.equal(y, ref[0]) and torch.equal(idx, ref[1]) and torch.equal(cls, ref[2]), (kind, T)
    # routing does not depend on the weight precision
    assert torch.equal(first[(16, 16)][1], first[(8, 16)][1]) and torch.equal(first[(16, 16)][2], first[(8, 16)][2])
    assert L.device_status() == 0
    L.close()


def test_calls_on_another_stream_give_the_same_bits():
    s = W.SHAPES["tiny"]
    for T in (4, 150):        # fused decode kernel; large-batch path with its side-stream fork
        wl = W.make_layer(s, T, variant=510)
        w = upload(wl)
        L = B.SpiceLayer(cfg_of(s), T)
        h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
        a = L.moe_layer_fwd(w, h, conf)
        torch.cuda.synchronize()
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            b = L.moe_layer_fwd(w, h, conf, stream=st)
        st.synchronize()
        assert torch.equal(a.y, b.y) and torch.equal(a.idx, b.idx) and torch.equal(a.counts, b.counts)
        assert L.device_status() == 0
        L.close()


def test_spread_routing_with_outputs_in_pinned_host_memory_or_not_wanted():
    """At more than 32 tokens the decode kernel exchanges the routing between thread blocks through the context's own arrays;
    the caller's idx / gate / cls are only written: they may live in pinned host memory, and y does not depend on whether
    they were asked for."""
    s = W.SHAPES["dsv2lite"]
    T = 48
    wl = W.make_layer(s, T, variant=520)
    w = upload(wl)
    L = B.SpiceLayer(cfg_of(s), T)
    h, conf = bf16_tensor(wl.h), torch.from_numpy(wl.conf).cuda()
    ref = L.moe_layer_fwd(w, h, conf)
    torch.cuda.synchronize()
    n = T * s.top_k
    idx = torch.empty(n, dtype=torch.int32).pin_memory()
    gate = torch.empty(n, dtype=torch.float32).pin_memory()
    cls = torch.empty(n, dtype=torch.uint8).pin_memory()
    y = torch.empty(T, s.d, dtype=torch.bfloat16, device="cuda")
    B.spice_moe_layer_fwd(L.ctx, w.c_struct(), h, conf, T, y, idx=idx, gate=gate, cls=cls)
    torch.cuda.synchronize()
    assert torch.equal(y, ref.y)
    assert torch.equal(idx.view(T, -1), ref.idx.cpu().view(T, -1)) and torch.equal(gate.view(T, -1), ref.gate.cpu().view(T, -1))
    assert torch.equal(cls.view(T, -1), ref.cls.cpu().view(T, -1))
    y2 = torch.empty_like(y)
    B.spice_moe_layer_fwd(L.ctx, w.c_struct(), h, conf, T, y2)
    torch.cuda.synchronize()
    assert torch.equal(y2, ref.y) and L.device_status() == 0
    L.close()
