"""The C-ABI library loads without a GPU and exports every symbol that
include/lt.h declares; host-only entry points and argument validation work."""
import ctypes as C
import os
import re

import pytest

import paper_2410_13846_b200 as lt
from paper_2410_13846_b200 import build
from oracle import lt_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "lt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lt_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = _declared_symbols()
    assert {"lt_lazy_scores", "lt_select_lazy", "lt_kv_append", "lt_hybrid_decode_attn", "lt_stream_init",
            "lt_workspace_bytes", "lt_ring_slot", "lt_status_string", "lt_check"} <= set(names)
    L = C.CDLL(lt.lib_path())
    for n in names:
        assert hasattr(L, n), f"{n} declared in lt.h but not exported"


def test_ring_slot_matches_integer_model():
    for S, R in [(0, 1), (4, 60), (4, 2044), (3, 7), (0, 5)]:
        for p in list(range(0, 3 * (S + R) + 5)) + [10**6, 2**31 - 2]:
            assert lt.ring_slot(p, S, R) == O.ring_slot(p, S, R)
    assert lt.ring_slot(-1, 4, 4) == -1 and lt.ring_slot(3, -1, 4) == -1 and lt.ring_slot(3, 4, 0) == -1


def test_status_strings_and_version():
    assert lt.version() >= 100
    seen = {lt.status_string(i) for i in range(7)}
    assert len(seen) == 7 and lt.status_string(0) == "ok" and "unknown" in lt.status_string(99)


def test_workspace_bytes_and_shape_validation():
    s = lt.Shape(32, 8, 32, 8, 128, 4, 2044, 32768 + 128)
    nb = lt.workspace_bytes(s, 32768, 64)
    assert nb > 256 and nb % 256 == 0
    assert lt.workspace_bytes(s, 0, 0) <= nb
    bad = [dict(n_layers=0), dict(n_layers=129), dict(head_dim=96), dict(n_q_heads=30), dict(n_recent=0),
           dict(n_sink=-1), dict(dtype=7), dict(full_capacity=0), dict(batch=0)]
    for kw in bad:
        d = dict(s.__dict__); d.update(kw)
        with pytest.raises(lt.LtError):
            lt.workspace_bytes(lt.Shape(**d), 128, 8)


def test_host_side_errors_come_before_any_launch():
    """Null pointers, n_lazy outside [0, L], w_last > n_ctx and a missing
    workspace are rejected on the host (no GPU is present in this test)."""
    L = lt.lib()
    s = lt.Shape(2, 1, 4, 2, 64, 4, 60, 512, lt.LT_F32)
    cs = s.c()
    fake = C.c_void_p(0x1000)           # never dereferenced: validation fails first
    tab = (C.c_void_p * 2)(0x1000, 0x2000)
    assert L.lt_select_lazy(fake, 2, 1, 4, 3, fake, None, None) == 1       # n_lazy > L
    assert L.lt_select_lazy(fake, 2, 1, 4, -1, fake, None, None) == 1
    assert L.lt_select_lazy(None, 2, 1, 4, 1, fake, None, None) == 1
    assert L.lt_select_lazy(fake, 200, 1, 4, 1, fake, None, None) == 2      # too many layers
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 512, 513, 0, 2, fake, fake, 1 << 20, None) == 1   # w_last > n_ctx
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 600, 16, 0, 2, fake, fake, 1 << 20, None) == 1    # n_ctx > capacity
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 512, 16, 0, 2, fake, None, 0, None) == 3          # no workspace
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 512, 16, 0, 2, fake, C.c_void_p(0x1000), 300, None) == 3  # too small
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 512, 16, 1, 2, fake, fake, 1 << 20, None) == 1    # layer range
    assert L.lt_lazy_scores(C.byref(cs), fake, tab, 512, 16, 0, 0, fake, fake, 1 << 20, None) == 1
    tab_null = (C.c_void_p * 2)(0x1000, None)
    assert L.lt_lazy_scores(C.byref(cs), fake, tab_null, 512, 16, 0, 2, fake, fake, 1 << 20, None) == 1   # scored layer missing
    assert L.lt_lazy_scores(C.byref(cs), fake, tab_null, 512, 16, 1, 1, fake, fake, 1 << 20, None) == 1
    # a missing entry outside the scored range is fine: the call gets past the table check (and stops at the workspace)
    assert L.lt_lazy_scores(C.byref(cs), fake, tab_null, 512, 16, 0, 1, fake, None, 0, None) == 3
    tab_misaligned = (C.c_void_p * 2)(0x1004, 0x2000)
    assert L.lt_hybrid_decode_attn(C.byref(cs), fake, tab_misaligned, tab, None, None, fake, fake, fake, 0, 0, 0, 2,
                                   fake, 1 << 20, None) == 1
    assert L.lt_hybrid_decode_attn(C.byref(cs), fake, tab, tab, None, None, fake, fake, fake, 0, 0, 1, 2,
                                   fake, 1 << 20, None) == 1                                     # layer range
    assert L.lt_hybrid_decode_attn(C.byref(cs), fake, tab, tab, None, None, fake, fake, fake, 5, 0, 0, 2,
                                   fake, 1 << 20, None) == 2                                     # out dtype
    assert L.lt_hybrid_decode_attn(C.byref(cs), fake, tab, tab, None, None, fake, fake, fake, 0, 0, 0, 2,
                                   C.c_void_p(0x1000), 256, None) == 3                           # ws too small
    assert L.lt_kv_append(C.byref(cs), fake, fake, fake, None, tab, tab, None, None, 0, 2, 1, None, None) == 1
    assert L.lt_kv_append(C.byref(cs), fake, fake, fake, fake, None, None, None, None, 0, 2, 1, None, None) == 1
    assert L.lt_stream_init(C.byref(cs), fake, tab, tab, fake, None, tab, None, None) == 1
    assert L.lt_workspace_init(None, 0, None) == 3
    # the layered step: same checks as lt_decode_step, and its workspace must have a slot region per layer
    need, need_l = C.c_size_t(0), C.c_size_t(0)
    big = lt.Shape(8, 2, 8, 2, 128, 4, 60, 40000)
    assert L.lt_workspace_bytes(C.byref(big.c()), 0, 0, C.byref(need)) == 0
    assert L.lt_workspace_bytes_layers(C.byref(big.c()), 0, 0, C.byref(need_l)) == 0 and need_l.value > need.value
    assert L.lt_workspace_bytes_layers(C.byref(big.c()), 0, 0, None) == 1
    tab8 = (C.c_void_p * 8)(*[0x1000 * (i + 1) for i in range(8)])
    args = lambda ws_bytes, begin=0, count=1, q=fake: (C.byref(big.c()), q, fake, fake, tab8, tab8, None, None, fake, fake, fake,
                                                        0, begin, count, 0, 1, C.c_void_p(0x1000), ws_bytes, None)
    assert L.lt_decode_step_layers(*args(need.value)) == 3                      # plain workspace: no per-layer slots
    assert L.lt_decode_step_layers(*args(need_l.value, begin=8)) == 1           # layer range
    assert L.lt_decode_step_layers(*args(need_l.value, q=None)) == 1            # null q


def test_binding_refuses_cpu_tensors():
    import torch
    s = lt.Shape(1, 1, 1, 1, 64, 0, 4, 8, lt.LT_F32)
    with pytest.raises(ValueError):
        lt.select_lazy(torch.zeros(1), 1, 1, 1, 0, torch.zeros(1, dtype=torch.uint8))
