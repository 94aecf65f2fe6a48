"""GPU edge cases of the decode step (maximum layer count, degenerate windows,
one-token caches, all-lazy and all-full stacks) and replay of a captured step."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, bits, f64

pytestmark = pytest.mark.gpu


def _replay_check(L, B, Hq, Hkv, D, S, R, n0, steps, mask, dtype=torch.bfloat16, seed=0):
    torch.manual_seed(seed)
    cap = n0 + steps
    st = Stack(L, B, Hq, Hkv, D, S, R, cap, dtype)
    st.set_mask(mask)
    hk = [torch.randn(B, Hkv, max(n0, 1), D).to(dtype) for _ in range(L)]
    hv = [torch.randn(B, Hkv, max(n0, 1), D).to(dtype) for _ in range(L)]
    for l in range(L):
        st.k_full[l][:, :, :n0] = hk[l][:, :, :n0].cuda(); st.v_full[l][:, :, :n0] = hv[l][:, :, :n0].cuda()
    st.set_seq_lens([n0] * B)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    reps = []
    for b in range(B):
        rp = O.HybridReplay(mask, S, R)
        for l in range(L):
            rp.load_prompt(l, f64(hk[l][b, :, :n0]), f64(hv[l][b, :, :n0]))
        reps.append(rp)
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).to(dtype).cuda()
        k = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        v = torch.randn(L, B, Hkv, D).to(dtype).cuda()
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
        for l in range(L):
            for b in range(B):
                reps[b].append(l, f64(k[l, b]), f64(v[l, b]))
                mx, rel = attn_errors(f64(out[l, b]), reps[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
    assert lt.check(st.ws) == 0 and st.seq_lens.cpu().tolist() == [n0 + steps] * B
    return st


def test_maximum_layer_count():
    g = np.random.default_rng(1)
    mask = (g.random(128) < 0.5).astype(np.uint8)
    _replay_check(128, 1, 4, 2, 128, 2, 6, 5, 10, mask)


def test_window_of_one_and_no_sink():
    # S = 0, R = 1: a lazy layer sees only the newest token -> the output is that token's value row
    st = _replay_check(2, 2, 2, 2, 128, 0, 1, 3, 4, [1, 0])
    assert st.k_stream[0].shape[2] == 1


def test_empty_prompt_single_head_and_one_token():
    _replay_check(2, 1, 1, 1, 128, 4, 4, 0, 9, [0, 1])           # starts from an empty cache; the ring wraps
    _replay_check(1, 3, 1, 1, 64, 1, 1, 0, 1, [1], dtype=torch.float32)   # one step from nothing: n = 1 everywhere


def test_all_lazy_and_all_full_stacks():
    _replay_check(3, 2, 8, 2, 128, 4, 12, 40, 6, [1, 1, 1], seed=2)
    _replay_check(3, 2, 8, 2, 128, 4, 12, 40, 6, [0, 0, 0], seed=3)


def test_captured_decode_step_replays():
    """The step reads lengths, mask and block state from the device, so one captured
    launch serves every later token: replay against eager calls, bit for bit."""
    torch.manual_seed(5)
    L, B, Hq, Hkv, D, S, R, n0, steps = 4, 2, 8, 2, 128, 4, 28, 100, 40
    cap = n0 + steps + 2
    eager = Stack(L, B, Hq, Hkv, D, S, R, cap)
    graph = Stack(L, B, Hq, Hkv, D, S, R, cap)
    for st in (eager, graph):
        st.set_mask([0, 1, 1, 0]); st.set_seq_lens([n0, n0 - 37])
    for l in range(L):
        k0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda(); v0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda()
        for st in (eager, graph):
            st.k_full[l].copy_(k0); st.v_full[l].copy_(v0)
    for st in (eager, graph):
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    sq = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    sk = torch.zeros(L, B, Hkv, D, dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros_like(sk)
    so = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    # one eager call on scratch state first: per-device launch attributes are looked up outside the capture
    warm = Stack(L, B, Hq, Hkv, D, S, R, cap)
    warm.set_seq_lens([1, 1])
    lt.decode_step(warm.shape, sq, sk, sv, warm.tables, warm.mask, warm.seq_lens, so, warm.ws)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        seq_before = graph.seq_lens.clone()
        with torch.cuda.graph(g, stream=side):
            lt.decode_step(graph.shape, sq, sk, sv, graph.tables, graph.mask, graph.seq_lens, so, graph.ws)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    assert torch.equal(graph.seq_lens, seq_before)              # capturing runs nothing
    ref = torch.zeros_like(so)
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(eager.shape, q, k, v, eager.tables, eager.mask, eager.seq_lens, ref, eager.ws)
        sq.copy_(q); sk.copy_(k); sv.copy_(v)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(so, ref), step
    assert torch.equal(graph.seq_lens, eager.seq_lens) and lt.check(graph.ws) == 0
    for l in range(L):
        assert torch.equal(graph.k_full[l], eager.k_full[l]) and torch.equal(graph.k_stream[l], eager.k_stream[l])


def test_captured_per_layer_step_replays():
    """A step issued layer by layer (launches that carry the programmatic-serialization attribute) captured
    as one CUDA graph: every replay equals an eager whole-stack step, bit for bit."""
    torch.manual_seed(6)
    L, B, Hq, Hkv, D, S, R, n0, steps = 5, 2, 8, 2, 128, 4, 28, 700, 12
    cap = n0 + steps + 2
    eager = Stack(L, B, Hq, Hkv, D, S, R, cap)
    graph = Stack(L, B, Hq, Hkv, D, S, R, cap)
    for st in (eager, graph):
        st.set_mask([0, 1, 0, 1, 0]); st.set_seq_lens([n0, n0 - 300])
    for l in range(L):
        k0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda(); v0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda()
        for st in (eager, graph):
            st.k_full[l].copy_(k0); st.v_full[l].copy_(v0)
    for st in (eager, graph):
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    sq = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    sk = torch.zeros(L, B, Hkv, D, dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros_like(sk)
    so = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")

    def per_layer_step(st):
        for l in range(L):
            lt.decode_step(st.shape, sq, sk, sv, st.tables, st.mask, st.seq_lens, so, st.ws, layer_begin=l,
                           layer_count=1, advance_seq_lens=(l == L - 1))

    warm = Stack(L, B, Hq, Hkv, D, S, R, cap)                    # per-device lookups happen outside the capture
    warm.set_seq_lens([1, 1])
    per_layer_step(warm)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            per_layer_step(graph)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    ref = torch.zeros_like(so)
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(eager.shape, q, k, v, eager.tables, eager.mask, eager.seq_lens, ref, eager.ws)
        sq.copy_(q); sk.copy_(k); sv.copy_(v)
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(so, ref), step
    assert torch.equal(graph.seq_lens, eager.seq_lens) and lt.check(graph.ws) == 0
    for l in range(L):
        assert torch.equal(graph.k_full[l], eager.k_full[l]) and torch.equal(graph.k_stream[l], eager.k_stream[l])
