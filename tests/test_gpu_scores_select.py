"""GPU parity: lt_lazy_scores (Eq. 1) and lt_select_lazy against the oracle."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import SCORE_ABS, Stack, f64

pytestmark = pytest.mark.gpu


def _run_scores(st, q_tail, n_ctx, T):
    s = st.shape
    scores = torch.full((s.n_layers, s.batch, s.n_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    lt.lazy_scores(s, q_tail, st.tables, n_ctx, T, scores, st.ws)
    return scores


def _oracle_scores(st, q_tail, n_ctx):
    s = st.shape
    scale = s.softmax_scale if s.softmax_scale > 0 else None
    ref = np.zeros((s.n_layers, s.batch, s.n_q_heads))
    for l in range(s.n_layers):
        for b in range(s.batch):
            ref[l, b] = O.lazy_scores(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx]), s.n_sink, s.n_recent, scale)
    return ref


CASES = [
    # dtype, D, Hq, Hkv, S, R, n_ctx, T, scale
    (torch.float32, 64, 4, 2, 4, 60, 512, 16, 0.0),        # toy
    (torch.bfloat16, 128, 8, 2, 4, 60, 777, 64, 0.0),      # GQA 4, odd length
    (torch.bfloat16, 128, 5, 1, 4, 28, 1300, 8, 0.0),      # GQA 5
    (torch.bfloat16, 128, 2, 2, 0, 16, 130, 64, 0.2),      # MHA, no sink, T > R, custom scale
    (torch.bfloat16, 128, 4, 1, 4, 2044, 2500, 64, 0.0),   # paper defaults
    (torch.bfloat16, 128, 4, 1, 4, 60, 40, 40, 0.0),       # window covers everything -> 1.0
    (torch.bfloat16, 64, 4, 2, 2, 9, 300, 5, 0.0),         # D=64
    (torch.bfloat16, 64, 16, 2, 4, 60, 1500, 64, 0.0),     # D=64, GQA 8: two 256-row blocks per (b, h)
    (torch.bfloat16, 64, 8, 2, 6, 252, 4100, 32, 0.3),     # D=64, several key splits, custom scale
    (torch.bfloat16, 128, 8, 2, 6, 252, 4100, 32, 0.0),    # several key splits
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,n_ctx,T,scale", CASES)
def test_scores_match_oracle(dtype, D, Hq, Hkv, S, R, n_ctx, T, scale):
    torch.manual_seed(5)
    L, B = 2, 2
    cap = n_ctx + 3
    st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype, scale, n_ctx_max=n_ctx, w_last_max=T)
    for l in range(L):
        st.k_full[l][:, :, :n_ctx] = torch.randn(B, Hkv, n_ctx, D).to(dtype).cuda()
        st.k_full[l][:, :, n_ctx:] = float("nan")               # never read
    q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
    got = f64(_run_scores(st, q_tail, n_ctx, T))
    ref = _oracle_scores(st, q_tail, n_ctx)
    assert np.isfinite(got).all()
    assert np.max(np.abs(got - ref)) <= SCORE_ABS, np.max(np.abs(got - ref))
    if S + R >= n_ctx:
        assert np.max(np.abs(got - 1.0)) <= 1e-5
    assert torch.equal(_run_scores(st, q_tail, n_ctx, T), torch.from_numpy(got).float().cuda())   # deterministic


@pytest.mark.parametrize("dtype,D", [(torch.float32, 64), (torch.bfloat16, 128), (torch.bfloat16, 64)])
def test_scoring_a_layer_range_equals_the_whole_stack_call(dtype, D):
    """Layer by layer, in ranges and all at once: the same scores up to the rounding of another split of the keys
    (the split depends on how many layers share the launch), only the scored layers' slices are written, and
    table entries outside the range may be missing (both kernels: CUDA-core and tensor-core path)."""
    torch.manual_seed(8)
    L, B, Hq, Hkv, S, R, n_ctx, T = 5, 2, 4, 2, 4, 60, 700, 16
    st = Stack(L, B, Hq, Hkv, D, S, R, n_ctx + 1, dtype, n_ctx_max=n_ctx, w_last_max=T)
    for l in range(L):
        st.k_full[l][:, :, :n_ctx] = torch.randn(B, Hkv, n_ctx, D).to(dtype).cuda()
    q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
    whole = _run_scores(st, q_tail, n_ctx, T)
    assert np.max(np.abs(f64(whole) - _oracle_scores(st, q_tail, n_ctx))) <= SCORE_ABS
    for ranges in ([(l, 1) for l in range(L)], [(0, 2), (2, 3)], [(3, 2), (0, 3)]):
        got = torch.full_like(whole, float("nan"))
        for begin, count in ranges:
            before = got.clone()
            only = [st.k_full[l] if begin <= l < begin + count else None for l in range(L)]     # the rest is "freed"
            tabs = lt.LayerTables(st.shape, only, None, None, None)
            lt.lazy_scores(st.shape, q_tail, tabs, n_ctx, T, got, st.ws, layer_begin=begin, layer_count=count)
            untouched = [l for l in range(L) if not begin <= l < begin + count]
            assert torch.equal(torch.nan_to_num(got[untouched], nan=-7.0), torch.nan_to_num(before[untouched], nan=-7.0))
        assert float((got - whole).abs().max()) <= 2e-6, ranges
        assert np.max(np.abs(f64(got) - _oracle_scores(st, q_tail, n_ctx))) <= SCORE_ABS
    assert lt.check(st.ws) == 0


def test_select_fed_oracle_scores_is_bit_exact():
    g = np.random.default_rng(6)
    for L, B, Hq in [(2, 1, 4), (32, 8, 32), (64, 4, 40), (7, 3, 5), (128, 1, 1)]:
        sc = g.random((L, B, Hq)).astype(np.float32)
        d = torch.from_numpy(sc).cuda()
        for n_lazy in sorted({0, 1, L // 4, L // 2, L - 1, L}):
            mask = torch.full((L,), 9, dtype=torch.uint8, device="cuda")
            ratio = torch.zeros(L, dtype=torch.float32, device="cuda")
            lt.select_lazy(d, L, B, Hq, n_lazy, mask, ratio)
            em, er = O.select_lazy(sc, n_lazy)
            assert np.array_equal(mask.cpu().numpy(), em)
            assert np.allclose(ratio.cpu().numpy(), er, rtol=0, atol=1e-7)
            assert np.array_equal(O.select_lazy_priority_queue(er, L - n_lazy), em)


def test_select_ties_go_to_lower_index():
    sc = np.array([0.5, 0.9, 0.5, 0.9, 0.1, 0.9], dtype=np.float32).reshape(6, 1, 1).repeat(3, axis=2)
    d = torch.from_numpy(sc).cuda()
    for n_lazy in range(7):
        mask = torch.zeros(6, dtype=torch.uint8, device="cuda")
        lt.select_lazy(d, 6, 1, 3, n_lazy, mask)
        assert np.array_equal(mask.cpu().numpy(), O.select_lazy(sc, n_lazy)[0])


# ---- the deployed form: denominator given, only the kept keys are read ---------------
def _oracle_lse(st, q_tail, n_ctx):
    s = st.shape
    scale = s.softmax_scale if s.softmax_scale > 0 else None
    return np.array([[O.causal_lse(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx]), scale)
                      for b in range(s.batch)] for l in range(s.n_layers)])          # [L, B, Hq, T]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,n_ctx,T,scale", CASES)
def test_scores_from_lse_match_eq1(dtype, D, Hq, Hkv, S, R, n_ctx, T, scale):
    """lt_lazy_scores_lse against the DEFINITION (O3, Eq. 1 over all keys), with the
    log-sum-exp an fp64 prefill would hand over rounded to fp32.  Keys outside the
    kept set hold NaN: the call must not read them."""
    torch.manual_seed(7)
    L, B = 2, 2
    cap = n_ctx + 3
    st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype, scale, n_ctx_max=n_ctx, w_last_max=T)
    for l in range(L):
        st.k_full[l][:, :, :n_ctx] = torch.randn(B, Hkv, n_ctx, D).to(dtype).cuda()
        st.k_full[l][:, :, n_ctx:] = float("nan")
    q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
    ref = _oracle_scores(st, q_tail, n_ctx)
    lse = torch.from_numpy(_oracle_lse(st, q_tail, n_ctx)).float().cuda().contiguous()
    for l in range(L):                                   # poison everything a lazy layer would discard
        lo, hi = min(S, n_ctx), max(S, n_ctx - R)
        st.k_full[l][:, :, lo:hi] = float("nan")
    s = st.shape
    got = torch.full((L, B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    lt.lazy_scores_lse(s, q_tail, st.tables, lse, n_ctx, T, got, st.ws)
    assert lt.check(st.ws) == 0
    g = f64(got)
    assert np.isfinite(g).all()
    assert np.max(np.abs(g - ref)) <= SCORE_ABS, np.max(np.abs(g - ref))
    ref2 = np.array([[O.lazy_scores_from_lse(f64(q_tail[l, b]), np.nan_to_num(f64(st.k_full[l][b, :, :n_ctx])),
                                             f64(lse[l, b]), S, R, s.softmax_scale if s.softmax_scale > 0 else None)
                      for b in range(B)] for l in range(L)])
    assert np.max(np.abs(g - ref2)) <= SCORE_ABS


def test_both_scoring_routes_give_the_same_mask_on_a_planted_stack():
    from synth import CONFIGS
    from tests.gpu_util import build_stack
    cfg = CONFIGS["llama3_8b_32k"].scaled(name="mini", n_layers=6, batch=2, n_ctx=3000, n_recent=252, n_lazy=3, steps=1)
    st, q_tail, planted = build_stack(cfg)
    s = st.shape
    L, B, Hq = cfg.n_layers, cfg.batch, cfg.n_q_heads
    a = torch.zeros((L, B, Hq), dtype=torch.float32, device="cuda")
    b = torch.zeros_like(a)
    lt.lazy_scores(s, q_tail, st.tables, cfg.n_ctx, cfg.w_last, a, st.ws)
    lse = torch.from_numpy(_oracle_lse(st, q_tail, cfg.n_ctx)).float().cuda().contiguous()
    lt.lazy_scores_lse(s, q_tail, st.tables, lse, cfg.n_ctx, cfg.w_last, b, st.ws)
    assert float((a - b).abs().max()) <= 2e-4
    ma = torch.zeros(L, dtype=torch.uint8, device="cuda"); mb = torch.zeros_like(ma)
    lt.select_lazy(a, L, B, Hq, cfg.n_lazy, ma); lt.select_lazy(b, L, B, Hq, cfg.n_lazy, mb)
    assert torch.equal(ma, mb) and sorted(torch.nonzero(ma).flatten().tolist()) == planted


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,n_ctx,T", [
    (torch.float32, 64, 4, 2, 4, 60, 512, 16),           # CUDA-core kernel
    (torch.bfloat16, 128, 8, 2, 4, 60, 1777, 64),        # tensor-core kernel, several pieces per unit
    (torch.bfloat16, 64, 5, 1, 0, 28, 900, 8),           # one row block, tiles alternate between the accumulators
])
def test_scores_pass_hands_out_the_log_sum_exp(dtype, D, Hq, Hkv, S, R, n_ctx, T):
    """lt_lazy_scores_with_lse: the denominators of the same pass against the oracle's causal log-sum-exp (what
    Table 1 takes from the prefill), the scores unchanged, and the pair (lse, kept keys) through the constant-size
    route reproducing Eq. 1."""
    torch.manual_seed(15)
    L, B = 3, 2
    st = Stack(L, B, Hq, Hkv, D, S, R, n_ctx, dtype, n_ctx_max=n_ctx, w_last_max=T)
    for l in range(L):
        st.k_full[l][:, :, :n_ctx] = torch.randn(B, Hkv, n_ctx, D).to(dtype).cuda()
    q_tail = (1.3 * torch.randn(L, B, Hq, T, D)).to(dtype).cuda()
    plain = _run_scores(st, q_tail, n_ctx, T)
    scores = torch.full_like(plain, float("nan"))
    lse = torch.full((L, B, Hq, T), float("nan"), dtype=torch.float32, device="cuda")
    lt.lazy_scores_with_lse(st.shape, q_tail, st.tables, n_ctx, T, scores, lse, st.ws)
    assert torch.equal(scores, plain)
    ref_lse = np.stack([np.stack([O.causal_lse(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :n_ctx])) for b in range(B)])
                        for l in range(L)])
    assert np.max(np.abs(f64(lse) - ref_lse)) <= 1e-4, np.max(np.abs(f64(lse) - ref_lse))
    # a layer range writes only its slices
    part = torch.full_like(lse, float("nan"))
    lt.lazy_scores_with_lse(st.shape, q_tail, st.tables, n_ctx, T, scores, part, st.ws, layer_begin=1, layer_count=1)
    assert torch.isnan(part[0]).all() and torch.isnan(part[2]).all()
    assert np.max(np.abs(f64(part[1]) - ref_lse[1])) <= 1e-4
    # the denominators feed the route that reads the kept keys only
    again = torch.full_like(plain, float("nan"))
    lt.lazy_scores_lse(st.shape, q_tail, st.tables, lse, n_ctx, T, again, st.ws)
    assert np.max(np.abs(f64(again) - _oracle_scores(st, q_tail, n_ctx))) <= SCORE_ABS
    assert lt.check(st.ws) == 0
