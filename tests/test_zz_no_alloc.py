"""spice_grouped_expert_ffn_static: the entry point for hosts that may not allocate (no ctx, no
cudaMalloc; scratch in a fixed device array of the library).  It must give what the ctx-based
spice_grouped_expert_ffn gives, call after call, although every call reuses the same array."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_21240_b200 import binding as B
from paper_2608_21240_b200 import workloads as W
from tests._cases import enforce_margins, run_oracle

pytestmark = pytest.mark.gpu


def _case(name, T, variant):
    wl = W.make_layer(name, T, variant=variant)
    enforce_margins(wl)
    s = wl.shape
    L = B.SpiceLayer(B.cfg_of(s), T)
    w = B.upload(wl)
    h = B.bf16_tensor(wl.h)
    idx, gate = L.route_topk(h, w.w_router)
    cls, slot, counts, _ = L.classify_misses(idx, gate, w.slot_of_expert, torch.from_numpy(wl.conf).cuda())
    assert int(counts[0]) > 0
    y_ref = torch.full((T, s.d), 0.25, device="cuda")     # y is accumulated into: start from a non-zero value
    L.grouped_expert_ffn(w, h, idx, gate, cls, slot, y_ref)
    torch.cuda.synchronize()
    # the oracle's value of the same sum: the exactly executed (resident) experts only, gate-weighted (Sec. 4.2)
    ref = run_oracle(wl, skip_ffn=True)
    assert np.array_equal(idx.cpu().numpy(), ref.idx) and np.array_equal(cls.cpu().numpy(), ref.cls)
    hits_only = np.zeros((T, s.d))
    for t in range(T):
        for k in range(s.top_k):
            if ref.cls[t, k] == oracle.HIT:
                hits_only[t] += ref.gate[t, k] * oracle.swiglu_ffn(*wl.expert(int(ref.idx[t, k])), wl.h[t])
    return L, s, w, h, idx, gate, cls, slot, y_ref, hits_only


def test_static_scratch_entry_point_matches_ctx_entry_point_on_consecutive_calls():
    assert B.spice_static_scratch_bytes() == 8 << 20
    # two different layers back to back: the second call finds the first call's tables in the array
    for name, T, variant in (("dsv2lite", 16, 21), ("tiny", 4, 22), ("dsv2lite", 16, 21)):
        L, s, w, h, idx, gate, cls, slot, y_ref, hits_only = _case(name, T, variant)
        bound_o = 1e-2 * np.abs(hits_only).max() + 1e-3
        assert np.abs(y_ref.cpu().numpy() - 0.25 - hits_only).max() <= bound_o
        status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        for _ in range(2):
            y = torch.full((T, s.d), 0.25, device="cuda")
            B.spice_grouped_expert_ffn_static(B.cfg_of(s), w.c_struct(), h, idx, gate, cls, slot, T, y, status)
            torch.cuda.synchronize()
            err = (y - y_ref).abs().max().item()
            bound = 1e-2 * y_ref.abs().max().item() + 1e-3
            assert err <= bound, (name, err, bound)
            err_o = np.abs(y.cpu().numpy().astype(np.float64) - 0.25 - hits_only).max()      # against the CPU oracle
            assert err_o <= bound_o, (name, err_o, bound_o)
            assert int(status[0]) == 0
        L.close()


def test_static_scratch_entry_point_rejects_what_does_not_fit():
    s = W.SHAPES["dsv2lite"]
    wl = W.make_layer(s, 1)
    w = B.upload(wl)
    T = 1024     # 6144 entries * (1408 + 2048) * 4 bytes = 85 MB > 8 MiB
    z = lambda *shape, dt: torch.zeros(*shape, dtype=dt, device="cuda")
    with pytest.raises(B.SpiceError, match="workspace"):
        B.spice_grouped_expert_ffn_static(B.cfg_of(s), w.c_struct(), z(T, s.d, dt=torch.bfloat16),
                                          z(T, s.top_k, dt=torch.int32), z(T, s.top_k, dt=torch.float32),
                                          z(T, s.top_k, dt=torch.uint8), z(T, s.top_k, dt=torch.int32), T,
                                          z(T, s.d, dt=torch.float32))
