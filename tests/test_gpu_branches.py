"""GPU parity on the branches of the decode step that ordinary shapes never
reach: the merge of a unit with more (max, sum) pairs than its shared-memory
staging area holds, the split of one call into several launches when the stack
has more (layer, batch row) pairs than one work list takes, and the mapping of
the device error word's bits to lt_check's status."""
import ctypes as C

import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, bits, f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True])
def test_merge_of_a_unit_with_more_pairs_than_the_staging_area(fused):
    """One layer, one batch row, one kv head with a group of 8 and 70 000 keys: the
    launch has so few keys that it takes 512-key chunks, 137 of them, so the unit's
    merge handles 137 x 8 = 1096 (max, sum) pairs - more than the 512 it can stage
    in shared memory - and reads them from global memory instead."""
    torch.manual_seed(71)
    L, B, Hq, Hkv, D, S, R = 1, 1, 8, 1, 128, 4, 60
    n = 70000
    cap = n + 8
    st = Stack(L, B, Hq, Hkv, D, S, R, cap)
    st.set_mask([0])
    K = torch.randn(B, Hkv, cap, D).bfloat16(); V = torch.randn(B, Hkv, cap, D).bfloat16()
    st.k_full[0].copy_(K); st.v_full[0].copy_(V)
    q = (1.5 * torch.randn(L, B, Hq, D)).bfloat16().cuda()
    if fused:
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda(); v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        st.set_seq_lens([n - 1])
        out = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
        K[0, :, n - 1] = k[0, 0].cpu(); V[0, :, n - 1] = v[0, 0].cpu()
        assert st.seq_lens.item() == n
        assert np.array_equal(bits(st.k_full[0][0, 0, n - 1]), bits(k[0, 0, 0]))
    else:
        st.set_seq_lens([n])
        out = st.attend(q, torch.float32)
    assert lt.check(st.ws) == 0
    ref = O.full_attention(f64(q[0, 0]), f64(K[0, :, :n]), f64(V[0, :, :n]))
    mx, rel = attn_errors(f64(out[0, 0]), ref)
    assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (mx, rel)
    # run-to-run identical bits: the chunks are merged in chunk order whichever CTA finishes last
    if not fused:
        assert torch.equal(st.attend(q, torch.float32), out)


def test_stack_with_more_layer_batch_pairs_than_one_launch_takes():
    """128 layers x 32 batch rows = 4096 (layer, batch row) pairs: the call is split
    on the host into two launches of 64 layers.  Fused steps: every layer appends
    at the same position (seq_lens advances once per step, after the last launch)."""
    torch.manual_seed(72)
    g = np.random.default_rng(72)
    L, B, Hq, Hkv, D, S, R = 128, 32, 2, 1, 128, 2, 6
    steps = 3
    lens = [int(x) for x in g.integers(0, 12, size=B)]
    cap = max(lens) + steps + 1
    mask = (g.random(L) < 0.5).astype(np.uint8)
    mask[[0, 63, 64, 127]] = [0, 1, 0, 1]                        # both kinds on either side of the split
    st = Stack(L, B, Hq, Hkv, D, S, R, cap)
    st.set_mask(mask)
    hk = [torch.randn(B, Hkv, cap, D).bfloat16() for _ in range(L)]
    hv = [torch.randn(B, Hkv, cap, D).bfloat16() for _ in range(L)]
    for l in range(L):
        for b, n in enumerate(lens):
            st.k_full[l][b, :, :n] = hk[l][b, :, :n].cuda(); st.v_full[l][b, :, :n] = hv[l][b, :, :n].cuda()
    st.set_seq_lens(lens)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    out = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
        assert st.seq_lens.cpu().tolist() == [n + step + 1 for n in lens]          # advanced exactly once
        for l in range(L):
            for b, n in enumerate(lens):
                hk[l][b, :, n + step] = k[l, b].cpu(); hv[l][b, :, n + step] = v[l, b].cpu()
    assert lt.check(st.ws) == 0 and torch.isfinite(out).all()
    units = [(0, 0), (63, B - 1), (64, 0), (127, B - 1)] + [(int(g.integers(L)), int(g.integers(B))) for _ in range(40)]
    for l, b in units:
        n = lens[b] + steps
        Kh, Vh = f64(hk[l][b, :, :n]), f64(hv[l][b, :, :n])
        ref = O.streaming_attention(f64(q[l, b]), Kh, Vh, S, R) if mask[l] else O.full_attention(f64(q[l, b]), Kh, Vh)
        mx, rel = attn_errors(f64(out[l, b]), ref)
        assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, mx, rel)
        if mask[l]:
            ek, _ = O.stream_cache_after(bits(hk[l][b, 0, :n]), S, R)
            assert np.array_equal(bits(st.k_stream[l][b, 0]), ek)
        else:
            assert np.array_equal(bits(st.k_full[l][b, 0, :n]), bits(hk[l][b, 0, :n]))
    # the attention half alone takes the same split
    ref_out = st.attend(q, torch.float32)
    assert torch.equal(ref_out, out)


def test_error_word_bits_map_to_status_codes():
    """lt_check reports LT_ERR_TIMEOUT when the timeout bit is set (with or without
    other bits), LT_ERR_DEVICE_RANGE for the other bits, and clears the word.  The
    word is written from the host here: no kernel has to run out of patience."""
    st = Stack(1, 1, 1, 1, 128, 1, 1, 4)
    L = lt.lib()
    word = st.ws[:4].view(torch.int32)
    flags = C.c_uint32(0)
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for bits_set, status in [(8, 5), (8 | 1, 5), (8 | 4 | 2, 5), (1, 6), (2, 6), (4, 6), (0, 0)]:
        word.fill_(bits_set)
        assert L.lt_check(C.c_void_p(st.ws.data_ptr()), C.byref(flags), stream) == status
        assert flags.value == bits_set
        assert word.item() == 0                                  # cleared for the next call
    word.fill_(8)
    with pytest.raises(lt.LtError) as e:
        lt.check(st.ws)
    assert e.value.status == 5 and "timed out" in str(e.value)
    word.fill_(8)
    assert lt.check(st.ws, raise_on_error=False) == 8
