"""The allocation-free decode entry point (collected last on purpose).

lt_hybrid_decode_attn_static serves hosts that are given pointers but may not
allocate device memory: an engine that already handed all free HBM to its
KV-cache pool, or a plug-in living inside another program's memory plan.  Its
split-KV scratch is a fixed array inside the library.  The GPU test calls it
through the C ABI twice in a row, on different inputs, and compares each result
with the ordinary entry point (which gets a caller-owned workspace); the second
call finds the first call's partials still in the array and must not be
affected by them.  Both entry points run the same deterministic kernel, so the
results are compared bit for bit.
"""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from paper_2410_13846_b200 import binding


def test_oversized_shape_is_refused_before_any_device_work():
    # the 32K benchmark stack needs ~69 MB of partials: more than the fixed array
    big = lt.Shape(32, 8, 32, 8, 128, 4, 2044, 32768 + 128)
    assert lt.workspace_bytes(big) > binding.STATIC_SCRATCH_BYTES
    import ctypes as C
    L = lt.lib()
    fake = C.c_void_p(0x1000)
    tab = (C.c_void_p * 32)(*([0x1000] * 32))
    st = L.lt_hybrid_decode_attn_static(C.byref(big.c()), fake, tab, tab, tab, tab, fake, fake, fake, 0, 0, 0, 32,
                                        None, None)
    assert st == 3          # LT_ERR_WORKSPACE


def test_refused_call_needs_no_device_and_enqueues_nothing():
    # every host-side check comes before the first CUDA call: on a machine without a GPU an invalid
    # call still gets its own status, not a CUDA error
    import ctypes as C
    small = lt.Shape(2, 1, 4, 2, 128, 4, 60, 512)
    L = lt.lib()
    fake = C.c_void_p(0x1000)
    tab = (C.c_void_p * 2)(0x1000, 0x2000)
    call = lambda *a: L.lt_hybrid_decode_attn_static(C.byref(small.c()), *a)  # noqa: E731
    assert call(None, tab, tab, tab, tab, fake, fake, fake, 0, 0, 0, 2, None, None) == 1       # q missing
    assert call(fake, tab, tab, tab, tab, fake, fake, fake, 7, 0, 0, 2, None, None) == 2       # out dtype
    assert call(fake, tab, tab, tab, tab, fake, fake, fake, 0, 0, 1, 2, None, None) == 1       # layer range
    assert call(fake, tab, tab, tab, tab, fake, fake, fake, 0, 0, 0, 2, C.c_void_p(0x1002), None) == 1  # dev_error misaligned


@pytest.mark.gpu
def test_static_entry_matches_workspace_entry_twice_in_a_row():
    from tests.gpu_util import Stack
    torch.manual_seed(21)
    L, B, Hq, Hkv, D, S, R, cap = 3, 2, 8, 2, 128, 4, 60, 3000
    st = Stack(L, B, Hq, Hkv, D, S, R, cap)
    assert lt.workspace_bytes(st.shape) <= binding.STATIC_SCRATCH_BYTES
    st.set_mask([0, 1, 0])
    for l in range(L):
        st.k_full[l].normal_(); st.v_full[l].normal_(); st.k_stream[l].normal_(); st.v_stream[l].normal_()
    err = torch.full((1,), 77, dtype=torch.int32, device="cuda")
    # first call: long rows (several KV chunks); second call: short rows and another q,
    # so stale partials of call 1 sit beyond what call 2 writes
    for lens in ([2900, 1500], [70, 3]):
        st.set_seq_lens(lens)
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        ref = st.attend(q, torch.float32)                                   # caller-owned workspace
        out = torch.full_like(ref, float("nan"))
        lt.hybrid_decode_attn_static(st.shape, q, st.tables, st.mask, st.seq_lens, out, dev_error=err)
        torch.cuda.synchronize()
        assert err.item() == 0
        assert torch.equal(out, ref), lens
    # the error word of a call is its own: a clamped length is reported, the next call starts clean
    st.set_seq_lens([cap + 5, 10])
    lt.hybrid_decode_attn_static(st.shape, q, st.tables, st.mask, st.seq_lens, out, dev_error=err)
    torch.cuda.synchronize()
    assert err.item() & 4
    st.set_seq_lens([20, 10])
    lt.hybrid_decode_attn_static(st.shape, q, st.tables, st.mask, st.seq_lens, out, dev_error=err)
    torch.cuda.synchronize()
    assert err.item() == 0
    # a call that is refused on the host leaves the caller's error word alone
    err.fill_(55)
    with pytest.raises(lt.LtError):
        lt.hybrid_decode_attn_static(st.shape, q, st.tables, st.mask, st.seq_lens, out, layer_begin=2, layer_count=5,
                                     dev_error=err)
    torch.cuda.synchronize()
    assert err.item() == 55
