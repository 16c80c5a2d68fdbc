"""The C-ABI library loads without a GPU and exports every entry point that include/spice.h declares;
host-side argument checks answer without touching a device."""
import ctypes as C
import os
import re

from paper_2608_21240_b200 import binding as B
from paper_2608_21240_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spice.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spice_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    cuda_build.build()
    lib = B.lib()
    names = declared_functions()
    assert {"spice_route_topk", "spice_classify_misses", "spice_grouped_expert_ffn", "spice_lore_surrogate",
            "spice_moe_layer_fwd", "spice_create", "spice_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in spice.h but not exported"


def test_host_side_checks_need_no_device():
    lib = B.lib()
    assert lib.spice_version() >= 100
    assert lib.spice_status_string(0) == b"ok" and b"unsupported" in lib.spice_status_string(2)
    ctx = C.c_void_p()
    good = B.make_cfg(256, 8, 2, 512, 512, 16, 5, 0.5)
    assert lib.spice_create(C.byref(ctx), 0, None, 4) == 1                 # NULL cfg
    assert lib.spice_create(C.byref(ctx), 0, C.byref(good), 0) == 1        # max_tokens < 1
    for field, val in (("d", 100), ("inter", 12), ("top_k", 9), ("n_experts", 2000), ("n_slots", 0), ("lore_rank", 4)):
        bad = B.make_cfg(256, 8, 2, 512, 512, 16, 5, 0.5)
        setattr(bad, field, val)
        assert lib.spice_create(C.byref(ctx), 0, C.byref(bad), 4) == 2, field   # unsupported shape
    assert lib.spice_destroy(None) == 0
    assert lib.spice_route_topk(None, None, None, 1, None, None, None, None) == 1
    assert lib.spice_moe_layer_fwd(None, None, None, None, 1, None, None, None, None, None, None, None, None, None,
                                   None, None, None) == 1
    assert lib.spice_static_scratch_bytes() == 8 << 20
    # the entry point without a ctx refuses a call that does not fit its fixed array before anything else
    assert lib.spice_grouped_expert_ffn_static(C.byref(B.make_cfg(2048, 64, 6, 1408, 2816, 64, 32, 0.6)), None, None,
                                               None, None, None, None, 4096, None, None, None) == 3


def test_binding_refuses_host_tensors():
    import pytest
    import torch
    with pytest.raises(B.SpiceError):
        B._ptr(torch.zeros(4))


def test_min_lookahead_depth_is_eq4_host_arithmetic():
    """Eq. 4 needs no device: checked against the oracle's ceiling formula on a grid of values, and on bad arguments."""
    import itertools
    import oracle
    from paper_2608_21240_b200 import binding as B
    for P, Me, Bw, Tc in itertools.product((0, 1, 2, 6), (17.3e6, 55e6), (12e9, 25e9, 50e9), (0.2e-3, 0.5e-3, 1.4e-3, 5e-3)):
        assert B.spice_min_lookahead_depth(P, Me, Bw, Tc) == oracle.min_lookahead_depth(P, Me, Bw, Tc)
    assert B.spice_min_lookahead_depth(2, 17.3e6, 25e9, 0.5e-3) == 3
    assert B.spice_min_lookahead_depth(2, 17.3e6, 0.0, 0.5e-3) == -1 and B.spice_min_lookahead_depth(-1, 1.0, 1.0, 1.0) == -1
