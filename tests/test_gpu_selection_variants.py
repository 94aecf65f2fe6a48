"""GPU parity of the selection variants around the hot path: per-prompt masks,
the streaming priority queue of Figure 3 with immediate compaction, and the
per-row reading of X_recent in the scoring pass."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, SCORE_ABS, Stack, attn_errors, bits, f64

pytestmark = pytest.mark.gpu


def test_per_sequence_selection_fed_oracle_scores_is_bit_exact():
    g = np.random.default_rng(16)
    for L, B, Hq in [(2, 1, 4), (32, 8, 32), (64, 4, 40), (7, 3, 5)]:
        sc = g.random((L, B, Hq)).astype(np.float32)
        d = torch.from_numpy(sc).cuda()
        for n_lazy in sorted({0, 1, L // 2, L}):
            mask = torch.full((B, L), 9, dtype=torch.uint8, device="cuda")
            ratio = torch.zeros((B, L), dtype=torch.float32, device="cuda")
            lt.select_lazy_per_seq(d, L, B, Hq, n_lazy, mask, ratio)
            em, er = O.select_lazy_per_sequence(sc, n_lazy)
            assert np.array_equal(mask.cpu().numpy(), em)
            assert np.allclose(ratio.cpu().numpy(), er, rtol=0, atol=1e-7)


def test_frequency_choice_over_per_sample_masks_is_bit_exact():
    """Section 5.2: per-sample masks (here from lt_select_lazy_per_seq over several
    batches of samples) are counted per layer and the most frequent layers chosen."""
    g = np.random.default_rng(26)
    L, B, Hq, n_lazy = 12, 5, 4, 5
    rows = []
    for _ in range(3):                                            # three batches of five samples
        sc = g.random((L, B, Hq)).astype(np.float32)
        sc[[2, 7, 9]] += 0.5                                      # layers that most samples find lazy
        m = torch.zeros((B, L), dtype=torch.uint8, device="cuda")
        lt.select_lazy_per_seq(torch.from_numpy(sc).cuda(), L, B, Hq, n_lazy, m)
        assert np.array_equal(m.cpu().numpy(), O.select_lazy_per_sequence(sc, n_lazy)[0])
        rows.append(m)
    masks = torch.cat(rows).contiguous()                          # [15][L]
    for k in (0, 3, 5, L):
        out = torch.full((L,), 9, dtype=torch.uint8, device="cuda")
        cnt = torch.zeros(L, dtype=torch.int32, device="cuda")
        lt.select_lazy_frequency(masks, masks.shape[0], L, k, out, cnt)
        em, ec = O.select_lazy_by_frequency(masks.cpu().numpy(), k)
        assert np.array_equal(out.cpu().numpy(), em) and np.array_equal(cnt.cpu().numpy(), ec)
    assert {2, 7, 9} <= set(np.nonzero(O.select_lazy_by_frequency(masks.cpu().numpy(), 5)[0])[0].tolist())


def test_per_sequence_masks_through_compaction_and_decode():
    """Every prompt of the batch has its own lazy layers: compaction, fused decode
    steps (ring wraps) and the separate append/attend calls follow the [B][L] mask."""
    torch.manual_seed(17)
    L, B, Hq, Hkv, D, S, R = 4, 3, 8, 2, 128, 3, 13
    n0, steps = 30, 24
    cap = n0 + steps
    mask = np.array([[1, 0, 0, 1], [0, 1, 1, 0], [1, 1, 0, 0]], dtype=np.uint8)          # [B][L]
    stacks = []
    for _ in range(2):
        st = Stack(L, B, Hq, Hkv, D, S, R, cap)
        st.shape.per_sequence_mask = 1
        st.mask = torch.from_numpy(mask).cuda().contiguous()
        stacks.append(st)
    fus, sep = stacks
    hk = [torch.randn(B, Hkv, n0, D).bfloat16() for _ in range(L)]
    hv = [torch.randn(B, Hkv, n0, D).bfloat16() for _ in range(L)]
    for st in stacks:
        for l in range(L):
            st.k_full[l][:, :, :n0] = hk[l].cuda(); st.v_full[l][:, :, :n0] = hv[l].cuda()
        st.set_seq_lens([n0] * B)
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    replays = []
    for b in range(B):
        rp = O.HybridReplay(mask[b], S, R)
        for l in range(L):
            rp.load_prompt(l, f64(hk[l][b]), f64(hv[l][b]))
        replays.append(rp)
    # compaction touched exactly the (layer, prompt) pairs whose mask is 1
    for l in range(L):
        for b in range(B):
            assert bool(fus.k_stream[l][b].any()) == bool(mask[b, l])
    hist = [[bits(hk[l][b]) for b in range(B)] for l in range(L)]
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(fus.shape, q, k, v, fus.tables, fus.mask, fus.seq_lens, out, fus.ws)
        sep.append(k, v)
        assert torch.equal(sep.attend(q, torch.float32), out)
        for l in range(L):
            for b in range(B):
                replays[b].append(l, f64(k[l, b]), f64(v[l, b]))
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
                hist[l][b] = np.concatenate([hist[l][b], bits(k[l, b])[:, None]], axis=1)
    assert lt.check(fus.ws) == 0 and lt.check(sep.ws) == 0
    for l in range(L):
        for b in range(B):
            for h in range(Hkv):
                if mask[b, l]:
                    ek, _ = O.stream_cache_after(hist[l][b][h], S, R)
                    assert np.array_equal(bits(fus.k_stream[l][b, h]), ek)
                    assert not fus.k_full[l][b, h, n0:].any()            # a lazy (layer, prompt) never grows its full cache
                else:
                    assert np.array_equal(bits(fus.k_full[l][b, h]), hist[l][b][h])
            assert torch.equal(fus.k_stream[l][b], sep.k_stream[l][b]) and torch.equal(fus.k_full[l][b], sep.k_full[l][b])


def test_streaming_queue_pops_like_figure_3_and_compacts_at_once():
    g = np.random.default_rng(18)
    torch.manual_seed(18)
    L, B, Hq, Hkv, D, S, R, n0 = 9, 2, 4, 2, 64, 2, 6, 20
    st = Stack(L, B, Hq, Hkv, D, S, R, n0 + 2, torch.float32)
    for l in range(L):
        st.k_full[l].normal_(); st.v_full[l].normal_()
    st.set_seq_lens([n0, n0 - 3])
    for P in (0, 3, 5, 9):
        sc = np.round(g.random((L, B, Hq)), 1).astype(np.float32)          # coarse: ties occur
        d = torch.from_numpy(sc).cuda()
        state = torch.zeros(L, dtype=torch.float64, device="cuda")
        mask = torch.full((L,), 7, dtype=torch.uint8, device="cuda")
        popped = torch.full((1,), -5, dtype=torch.int32, device="cuda")
        for l in range(L):
            st.k_stream[l].zero_(); st.v_stream[l].zero_()
        emask, epopped = O.select_lazy_priority_queue_trace(O.layer_ratios(sc), P)
        for l in range(L):
            lt.select_lazy_push(d[l], l, L, B, Hq, P, state, mask, popped)
            lt.stream_init_layer(st.shape, mask, popped, st.tables, st.seq_lens, ws=st.ws)
            assert popped.item() == epopped[l], (P, l)
            # layers that have not arrived are untouched; exactly the popped layers are compacted so far
            done = set(int(x) for x in epopped[: l + 1] if x >= 0)
            for m in range(L):
                assert bool(st.k_stream[m].any()) == (m in done)
        assert np.array_equal(mask.cpu().numpy(), emask)
        assert np.array_equal(emask, O.select_lazy(sc, L - P)[0])
        # same stream caches as the one-shot compaction with the final mask
        ref = Stack(L, B, Hq, Hkv, D, S, R, n0 + 2, torch.float32)
        for l in range(L):
            ref.k_full[l].copy_(st.k_full[l]); ref.v_full[l].copy_(st.v_full[l])
        ref.seq_lens.copy_(st.seq_lens); ref.mask.copy_(mask)
        lt.stream_init(ref.shape, ref.mask, ref.tables, ref.seq_lens, ws=ref.ws)
        for l in range(L):
            assert torch.equal(ref.k_stream[l], st.k_stream[l]) and torch.equal(ref.v_stream[l], st.v_stream[l])
    assert lt.check(st.ws) == 0


PER_ROW_CASES = [
    # dtype, D, Hq, Hkv, S, R, n_ctx, T
    (torch.float32, 64, 4, 2, 4, 60, 512, 16),
    (torch.bfloat16, 128, 8, 2, 4, 60, 777, 64),
    (torch.bfloat16, 128, 2, 2, 0, 16, 130, 64),          # T > R, no sink
    (torch.bfloat16, 128, 4, 1, 4, 252, 2500, 64),
    (torch.bfloat16, 128, 4, 1, 4, 60, 40, 40),           # covers everything
    (torch.bfloat16, 64, 8, 2, 4, 60, 777, 64),           # head_dim 64 on the tensor-core route
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,n_ctx,T", PER_ROW_CASES)
def test_per_row_window_scores_both_routes(dtype, D, Hq, Hkv, S, R, n_ctx, T):
    torch.manual_seed(19)
    L, B = 2, 2
    st = Stack(L, B, Hq, Hkv, D, S, R, n_ctx + 1, dtype, n_ctx_max=n_ctx, w_last_max=T)
    st.shape.recent_per_row = 1
    for l in range(L):
        st.k_full[l][:, :, :n_ctx] = torch.randn(B, Hkv, n_ctx, D).to(dtype).cuda()
    q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
    ref = np.array([[O.lazy_scores_per_row_window(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx]), S, R)
                     for b in range(B)] for l in range(L)])
    fixed = np.array([[O.lazy_scores(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx]), S, R)
                       for b in range(B)] for l in range(L)])
    got = torch.zeros((L, B, Hq), dtype=torch.float32, device="cuda")
    lt.lazy_scores(st.shape, q_tail, st.tables, n_ctx, T, got, st.ws)
    assert np.max(np.abs(f64(got) - ref)) <= SCORE_ABS
    if S + R < n_ctx - T and T > 1:
        assert np.max(np.abs(ref - fixed)) > 10 * SCORE_ABS          # the two readings really differ on this input
    lse = torch.from_numpy(np.array([[O.causal_lse(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx]))
                                      for b in range(B)] for l in range(L)])).float().cuda().contiguous()
    got2 = torch.zeros_like(got)
    lt.lazy_scores_lse(st.shape, q_tail, st.tables, lse, n_ctx, T, got2, st.ws)
    assert np.max(np.abs(f64(got2) - ref)) <= SCORE_ABS
    assert lt.check(st.ws) == 0
