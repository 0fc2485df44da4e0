"""CPU checks of the C-ABI library: it loads, exports every declared symbol, and its
pure host helpers agree with the oracle.  No kernel is launched here."""
import os
import re

import pytest

from oracle import freebalance_oracle as O
from paper_2608_14205_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(inc, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(fb_[a-z_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert "fb_predict_load" in names and "fb_plan_swaps" in names and "fb_route_dispatch" in names
    L = B.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in the header but not exported"
    assert sorted(B.EXPORTS) == names


def test_budget_helper_matches_eq10():
    for t, d in [(500_000, 100_000), (100, 100), (100, 250), (0, 0), (2**63, 1)]:
        assert B.fb_budget_ns(t, d) == O.budget_ns(t, d)


@pytest.mark.parametrize("alpha,fs,size,rpn", [((2000, 2000), (1111, 1111), 44_040_192, 0),
                                               ((10, 1000), (1000, 4000), 500, 2),
                                               ((0, 0), (0, 0), 0, 0), ((0, 7), (1, 3), 1, 4),
                                               ((5, 5), (10**6, 10**6), 9 * 2**20, 0)])
def test_cost_helper_matches_eq9(alpha, fs, size, rpn):
    b = B.make_budget(alpha_ns=alpha, fs_per_byte=fs, expert_bytes=size, ranks_per_node=rpn)
    ob = O.Budget(alpha_ns=alpha, fs_per_byte=fs, expert_bytes=size, ranks_per_node=rpn)
    for a, bb in [(0, 1), (1, 2), (3, 4), (0, 7)]:
        assert B.fb_swap_cost_ns(b, a, bb) == O.swap_cost_ns(ob, a, bb)


def test_cost_helper_reports_overflow():
    b = B.make_budget(alpha_ns=(0, 0), fs_per_byte=(2**63, 2**63), expert_bytes=2**62)
    assert B.fb_swap_cost_ns(b, 0, 1) == 0


def test_status_strings():
    L = B.lib()
    seen = {L.fb_status_string(s).decode() for s in range(8)}
    assert len(seen) == 8 and all(seen)


def test_create_rejects_bad_shapes_before_touching_a_device():
    import ctypes
    h = ctypes.c_void_p()
    L = B.lib()
    bad = [dict(E=300), dict(k=9), dict(k=0), dict(R=3), dict(R=128, E=128), dict(d=100), dict(E=8, k=9),
           dict(gate=1, n_group=3), dict(gate=1, n_group=8, topk_group=9), dict(gate=1, n_group=8, topk_group=1, k=8, E=32)]
    for kw in bad:
        base = dict(T_max=128, d=64, E=8, k=2, R=4, gate=0, n_group=1, topk_group=1, renorm=1, route_scale=1.0)
        base.update(kw)
        cfg = B.FbConfig(*[base[f] for f, _ in B.FbConfig._fields_])
        st = L.fb_create(ctypes.byref(h), ctypes.byref(cfg), 0)
        assert st in (B.FB_ERR_INVALID_ARG, B.FB_ERR_UNSUPPORTED_SHAPE), (kw, st)
        assert not h.value
    assert L.fb_create(None, None, 0) == B.FB_ERR_INVALID_ARG
    assert L.fb_destroy(None) == B.FB_OK
