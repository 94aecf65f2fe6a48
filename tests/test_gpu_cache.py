"""GPU parity: lt_kv_append and lt_stream_init against the oracle's integer ring
model.  Everything here is bit-exact."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import Stack, bits

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,D", [(torch.bfloat16, 128), (torch.float32, 64), (torch.bfloat16, 64)])
@pytest.mark.parametrize("S,R", [(4, 12), (0, 5), (3, 1)])
def test_append_replay_matches_ring_model(dtype, D, S, R):
    """Many steps with per-row start lengths: rings wrap several times; the
    stream cache must hold exactly the owner token's bits in every slot and
    the full cache every token at its position."""
    torch.manual_seed(0)
    L, B, Hq, Hkv = 3, 3, 4, 2
    steps, start = 4 * (S + R) + 3, [0, 2, S + R + 1]
    cap = max(start) + steps
    st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype)
    st.set_mask([0, 1, 1])
    st.set_seq_lens(start)
    # history per (layer, b): list of rows; rows before `start` are zeros already "in" the cache
    hist_k = [[[np.zeros((Hkv, D), dtype=bits(torch.zeros(1, dtype=dtype)).dtype)] * start[b] for b in range(B)]
              for _ in range(L)]
    hist_v = [[list(x) for x in row] for row in hist_k]
    for step in range(steps):
        k = torch.randn(L, B, Hkv, D, device="cuda").to(dtype)
        v = torch.randn(L, B, Hkv, D, device="cuda").to(dtype)
        st.append(k, v)
        kb, vb = bits(k), bits(v)
        for l in range(L):
            for b in range(B):
                hist_k[l][b].append(kb[l, b]); hist_v[l][b].append(vb[l, b])
    assert st.seq_lens.cpu().tolist() == [s + steps for s in start]
    assert lt.check(st.ws) == 0
    for l in range(L):
        for b in range(B):
            hk = np.stack(hist_k[l][b]); hv = np.stack(hist_v[l][b])       # [n, Hkv, D]
            n = hk.shape[0]
            if l == 0:
                assert np.array_equal(bits(st.k_full[l][b, :, :n]).transpose(1, 0, 2), hk)
                assert np.array_equal(bits(st.v_full[l][b, :, :n]).transpose(1, 0, 2), hv)
                assert not bits(st.k_stream[l]).any()                     # a full layer's stream cache is untouched
            else:
                # rows that were "in the cache" before the test started were never written: compare only
                # slots whose owner was appended by the test
                ck = bits(st.k_stream[l][b]).transpose(1, 0, 2); cv = bits(st.v_stream[l][b]).transpose(1, 0, 2)
                for s_ in range(S + R):
                    p = O.ring_owner(s_, n, S, R)
                    if p is not None and p >= start[b]:
                        assert np.array_equal(ck[s_], hk[p]) and np.array_equal(cv[s_], hv[p]), (l, b, s_, p)
                    elif p is None:
                        assert not ck[s_].any()
                assert not bits(st.k_full[l]).any()


def test_append_out_of_capacity_is_flagged_not_written():
    st = Stack(2, 2, 2, 1, 64, 2, 4, 8, torch.float32)
    st.set_mask([0, 1])
    st.set_seq_lens([8, 3])                       # row 0 is full
    k = torch.ones(2, 2, 1, 64, device="cuda"); v = 2 * k
    st.append(k, v)
    flags = lt.check(st.ws, raise_on_error=False)
    assert flags & 1
    assert float(st.k_full[0][0].abs().sum()) == 0.0          # skipped
    assert float(st.k_full[0][1, 0, 3].sum()) == 64.0         # the in-range row was written
    assert float(st.k_stream[1][0, 0, 2 + (8 - 2) % 4].sum()) == 64.0   # the lazy layer has no capacity limit
    assert lt.check(st.ws) == 0                               # cleared by the read


def test_append_layer_range_and_no_advance():
    st = Stack(4, 1, 2, 2, 64, 1, 3, 16, torch.bfloat16)
    st.set_mask([0, 1, 0, 1])
    k = torch.randn(4, 1, 2, 64, device="cuda").bfloat16(); v = torch.randn_like(k)
    st.append(k, v, layer_begin=1, layer_count=2, advance_seq_lens=False)
    assert st.seq_lens.item() == 0
    assert not st.k_full[0].any() and not st.k_stream[3].any()
    assert torch.equal(st.k_stream[1][0, :, 0], k[1, 0]) and torch.equal(st.v_full[2][0, :, 0], v[2, 0])
    st.append(k, v, layer_begin=0, layer_count=1)
    assert st.seq_lens.item() == 1 and torch.equal(st.k_full[0][0, :, 0], k[0, 0])


@pytest.mark.parametrize("S,R,lens", [(4, 60, [512, 70, 64, 63, 3, 0]), (0, 16, [100, 16, 15, 1]), (6, 1, [9, 6, 7])])
def test_stream_init_matches_replay(S, R, lens):
    torch.manual_seed(1)
    L, B, Hkv, D = 3, len(lens), 2, 64
    cap = max(lens) + 4
    st = Stack(L, B, 2 * Hkv, Hkv, D, S, R, cap, torch.bfloat16)
    for l in range(L):
        st.k_full[l].copy_(torch.randn(B, Hkv, cap, D).bfloat16()); st.v_full[l].copy_(torch.randn(B, Hkv, cap, D).bfloat16())
        st.k_stream[l].fill_(7.0); st.v_stream[l].fill_(7.0)              # sentinel: untouched rows keep it
    st.set_mask([1, 0, 1]); st.set_seq_lens(lens)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    assert lt.check(st.ws) == 0
    sent = bits(torch.full((1,), 7.0).bfloat16())[0]
    for l in range(L):
        ks, vs = bits(st.k_stream[l]), bits(st.v_stream[l])
        if l == 1:
            assert (ks == sent).all() and (vs == sent).all()
            continue
        kf, vf = bits(st.k_full[l]), bits(st.v_full[l])
        for b, n in enumerate(lens):
            for h in range(Hkv):
                ek, valid = O.stream_cache_after(kf[b, h, :n], S, R)
                ev, _ = O.stream_cache_after(vf[b, h, :n], S, R)
                assert np.array_equal(ks[b, h, :valid], ek[:valid]) and np.array_equal(vs[b, h, :valid], ev[:valid])
                assert (ks[b, h, valid:] == sent).all() and (vs[b, h, valid:] == sent).all()


def test_init_then_append_continues_the_ring():
    """Compaction followed by appends equals a replay of the whole history."""
    torch.manual_seed(2)
    S, R, n0, steps = 2, 6, 20, 15
    st = Stack(1, 1, 1, 1, 64, S, R, n0 + steps, torch.float32)
    hist = torch.randn(n0 + steps, 64)
    st.k_full[0][0, 0, :n0] = hist[:n0].cuda(); st.v_full[0][0, 0, :n0] = -hist[:n0].cuda()
    st.set_mask([1]); st.set_seq_lens([n0])
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens)
    for i in range(steps):
        row = hist[n0 + i].cuda().reshape(1, 1, 1, 64)
        st.append(row.contiguous(), (-row).contiguous())
    ek, valid = O.stream_cache_after(bits(hist), S, R)
    assert valid == S + R
    assert np.array_equal(bits(st.k_stream[0][0, 0]), ek)
    assert np.array_equal(bits(st.v_stream[0][0, 0]), bits(-hist)[[O.ring_owner(s, n0 + steps, S, R) for s in range(S + R)]])
