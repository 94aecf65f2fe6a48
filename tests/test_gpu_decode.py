"""GPU parity: lt_hybrid_decode_attn against the oracle (O1 on full layers, O2 on
the logical history for lazy layers)."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, f64

pytestmark = pytest.mark.gpu


def _fill_from_history(st, hist_k, hist_v, lens):
    """hist_[l]: tensor [B, Hkv, n_max, D] (logical history).  Full caches get the
    history, stream caches the oracle ring replay of it."""
    s = st.shape
    for l in range(s.n_layers):
        for b, n in enumerate(lens):
            st.k_full[l][b, :, :n] = hist_k[l][b, :, :n].cuda(); st.v_full[l][b, :, :n] = hist_v[l][b, :, :n].cuda()
            for h in range(s.n_kv_heads):
                ck, valid = O.stream_cache_after(hist_k[l][b, h, :n].float().numpy(), s.n_sink, s.n_recent)
                cv, _ = O.stream_cache_after(hist_v[l][b, h, :n].float().numpy(), s.n_sink, s.n_recent)
                st.k_stream[l][b, h] = torch.from_numpy(ck).to(st.dtype).cuda()
                st.v_stream[l][b, h] = torch.from_numpy(cv).to(st.dtype).cuda()
    st.set_seq_lens(lens)


def _oracle_out(st, q, hist_k, hist_v, lens, mask):
    s = st.shape
    ref = np.zeros((s.n_layers, s.batch, s.n_q_heads, s.head_dim))
    scale = s.softmax_scale if s.softmax_scale > 0 else None
    for l in range(s.n_layers):
        for b, n in enumerate(lens):
            if n == 0:
                continue
            K, V = f64(hist_k[l][b, :, :n]), f64(hist_v[l][b, :, :n])
            ref[l, b] = (O.streaming_attention(f64(q[l, b]), K, V, s.n_sink, s.n_recent, scale) if mask[l]
                         else O.full_attention(f64(q[l, b]), K, V, scale))
    return ref


CASES = [
    # dtype, D, Hq, Hkv, S, R, lens, scale              (bf16, G <= 32 -> tensor-core path)
    (torch.bfloat16, 128, 8, 2, 4, 60, [300, 1, 64, 65, 17], 0.0),          # G=4, ragged, n<S+R, exactly S+R
    (torch.bfloat16, 128, 5, 1, 4, 28, [2049, 2048, 2047, 33], 0.0),        # G=5, chunk boundaries
    (torch.bfloat16, 128, 2, 2, 0, 16, [100, 16, 3], 0.11),                 # G=1, no sink, custom scale
    (torch.bfloat16, 128, 16, 2, 2, 6, [700, 5], 0.0),                      # G=8
    (torch.bfloat16, 128, 32, 2, 4, 12, [130, 40], 0.0),                    # G=16: warp pairs, eight heads per warp
    (torch.bfloat16, 128, 12, 1, 4, 28, [4200, 2049, 65], 0.0),             # G=12: warps of a pair serve 8 and 4 heads, several chunks
    (torch.bfloat16, 128, 40, 2, 4, 12, [130, 40], 0.0),                    # G=20: four warps per tile; the third serves 4 heads, the fourth none
    (torch.bfloat16, 128, 32, 1, 4, 28, [4200, 2049, 65, 0], 0.0),          # G=32: four warps per tile, eight heads each, several chunks
    (torch.bfloat16, 128, 17, 1, 0, 16, [300, 31], 0.0),                    # G=17: one head in the third warp
    (torch.bfloat16, 64, 24, 1, 4, 28, [2049, 2047, 33, 4500], 0.0),        # D=64, G=24: four warps over a twelve-stage ring
    (torch.bfloat16, 128, 40, 1, 4, 12, [130, 40], 0.0),                    # G=40 -> CUDA-core path, five passes of eight heads
    (torch.bfloat16, 64, 4, 2, 4, 60, [257, 90], 0.0),                      # D=64: 32-key tiles of 128-byte rows
    (torch.bfloat16, 64, 8, 1, 4, 28, [2049, 2048, 2047, 33, 4500], 0.0),   # D=64, G=8, chunk boundaries
    (torch.bfloat16, 64, 16, 1, 4, 28, [300, 2100], 0.0),                   # D=64, G=16: warp pairs
    (torch.float32, 128, 4, 4, 4, 20, [129, 77], 0.0),                      # fp32
    (torch.float32, 64, 4, 2, 4, 60, [513], 0.0),                           # toy shape
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,lens,scale", CASES)
def test_decode_matches_oracle(dtype, D, Hq, Hkv, S, R, lens, scale):
    torch.manual_seed(3)
    L, B = 3, len(lens)
    cap = max(lens) + 5
    mask = [0, 1, 0]
    st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype, scale)
    st.set_mask(mask)
    hist_k = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    hist_v = [torch.randn(B, Hkv, cap, D).to(dtype) for _ in range(L)]
    _fill_from_history(st, hist_k, hist_v, lens)
    # rows beyond the valid length hold NaN bit patterns: they must never be read into the result
    for l in range(L):
        for b, n in enumerate(lens):
            st.k_full[l][b, :, n:] = float("nan"); st.v_full[l][b, :, n:] = float("nan")
            valid = O.ring_valid_slots(n, S, R)
            st.k_stream[l][b, :, valid:] = float("nan"); st.v_stream[l][b, :, valid:] = float("nan")
    q = (1.5 * torch.randn(L, B, Hq, D)).to(dtype).cuda()
    ref = _oracle_out(st, q, hist_k, hist_v, lens, mask)
    out = st.attend(q, torch.float32)
    assert lt.check(st.ws) == 0
    got = f64(out)
    assert np.isfinite(got).all()
    mx, rel = attn_errors(got, ref)
    assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (mx, rel)
    # per-layer bound too, so that one bad layer kind cannot hide in the average
    for l in range(L):
        mxl, rell = attn_errors(got[l], ref[l])
        assert mxl <= ATTN_MAX_ABS and rell <= ATTN_REL_L2, (l, mxl, rell)
    # bf16 output option: the fp32 result rounded once
    out16 = st.attend(q, torch.bfloat16)
    assert torch.equal(out16, out.to(torch.bfloat16))
    # determinism: identical bits on a second run
    assert torch.equal(st.attend(q, torch.float32), out)


def test_empty_rows_give_zeros_and_hint_and_layer_range():
    torch.manual_seed(4)
    L, B, Hq, Hkv, D, S, R = 2, 3, 8, 2, 128, 4, 60
    lens = [0, 500, 64]
    cap = 4096
    st = Stack(L, B, Hq, Hkv, D, S, R, cap)
    st.set_mask([0, 1])
    hist_k = [torch.randn(B, Hkv, cap, D).bfloat16() for _ in range(L)]
    hist_v = [torch.randn(B, Hkv, cap, D).bfloat16() for _ in range(L)]
    _fill_from_history(st, hist_k, hist_v, lens)
    q = torch.randn(L, B, Hq, D).bfloat16().cuda()
    ref = _oracle_out(st, q, hist_k, hist_v, lens, [0, 1])
    full = st.attend(q)
    assert float(full[:, 0].abs().sum()) == 0.0
    hinted = st.attend(q, hint=500)
    assert torch.equal(hinted, full)                            # a true bound changes nothing
    mx, rel = attn_errors(f64(full), ref)
    assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2
    # one layer at a time writes only that layer
    s = st.shape
    out = torch.full((L, B, Hq, D), 9.0, dtype=torch.float32, device="cuda")
    lt.hybrid_decode_attn(s, q, st.tables, st.mask, st.seq_lens, out, st.ws, layer_begin=1, layer_count=1)
    assert torch.equal(out[1], full[1]) and bool((out[0] == 9.0).all())
    # the hint no longer sizes anything: a wrong one changes nothing either
    assert torch.equal(st.attend(q, hint=100), full)
    assert lt.check(st.ws) == 0


def test_seq_len_beyond_capacity_is_clamped_and_flagged():
    st = Stack(1, 1, 4, 1, 128, 4, 12, 32)
    st.k_full[0].normal_(); st.v_full[0].normal_()
    st.set_seq_lens([40])
    q = torch.randn(1, 1, 4, 128).bfloat16().cuda()
    out = st.attend(q)
    assert torch.isfinite(out).all()
    assert lt.check(st.ws, raise_on_error=False) & 4
    st.set_seq_lens([32])
    assert torch.equal(st.attend(q), out)


def test_null_layer_entry_is_flagged():
    st = Stack(2, 1, 4, 1, 128, 4, 12, 32)
    tabs = lt.LayerTables(st.shape, st.k_full, st.v_full, [None, None], [None, None])
    st.set_mask([0, 1]); st.set_seq_lens([8])
    q = torch.randn(2, 1, 4, 128).bfloat16().cuda()
    out = torch.zeros(2, 1, 4, 128, device="cuda")
    lt.hybrid_decode_attn(st.shape, q, tabs, st.mask, st.seq_lens, out, st.ws)
    assert lt.check(st.ws, raise_on_error=False) & 2
