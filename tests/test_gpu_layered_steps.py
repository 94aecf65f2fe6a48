"""GPU parity of lt_decode_step_layers: a step issued as launches over disjoint layer ranges that may run under
one another's tails.  Bit-identical to the same launches in plain stream order (lt_decode_step layer by
layer), and equal to the oracle (O1 / O2 on the logical history) on units sampled at the last step."""
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, f64

pytestmark = pytest.mark.gpu


def _layered_ws(st):
    nbytes = lt.workspace_bytes_layers(st.shape, 0, 0)
    assert nbytes >= lt.workspace_bytes(st.shape, 0, 0)
    st.ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    assert st.ws.data_ptr() % 256 == 0
    lt.workspace_init(st.ws)


def _two_stacks(L, B, Hq, Hkv, D, S, R, cap, dtype, lens, mask, seed):
    g = torch.Generator().manual_seed(seed)
    stacks = [Stack(L, B, Hq, Hkv, D, S, R, cap, dtype) for _ in range(2)]
    prompts = []
    for l in range(L):
        k = torch.randn(B, Hkv, cap, D, generator=g).to(dtype)
        v = torch.randn(B, Hkv, cap, D, generator=g).to(dtype)
        prompts.append((k, v))
        for st in stacks:
            st.k_full[l].copy_(k); st.v_full[l].copy_(v)
    for st in stacks:
        st.set_mask(mask); st.set_seq_lens(lens)
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    _layered_ws(stacks[1])
    return stacks[0], stacks[1], prompts


CASES = [
    # dtype, D, Hq, Hkv, S, R, lens, mask, range length, steps
    (torch.bfloat16, 128, 16, 4, 4, 60, [9000, 4100, 700, 0], [0, 1, 0, 0, 1, 1, 0, 0], 1, 10),   # several chunks per unit
    (torch.bfloat16, 128, 16, 4, 4, 28, [3000, 1500, 31], [1, 0, 0, 1, 0, 1], 2, 40),             # ranges of two layers; rings wrap
    (torch.bfloat16, 64, 24, 2, 0, 16, [5000, 2047], [0, 0, 1, 0], 1, 6),                         # head_dim 64, warp pairs (G = 12)
    (torch.float32, 64, 4, 2, 4, 60, [513, 3], [0, 1, 0], 1, 5),                                  # CUDA-core path: plain order inside
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,lens,mask,span,steps", CASES)
def test_overlapped_layer_launches_equal_plain_stream_order(dtype, D, Hq, Hkv, S, R, lens, mask, span, steps):
    """No host synchronisation inside the chain, so that launches really are in flight together; every output,
    every cache row and seq_lens must carry the bits of the plain-order chain, step boundaries included."""
    L, B = len(mask), len(lens)
    cap = max(lens) + steps + 3
    plain, over, prompts = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, dtype, lens, mask, seed=21)
    g = torch.Generator().manual_seed(22)
    qs = [torch.randn(L, B, Hq, D, generator=g).to(dtype).cuda() for _ in range(steps)]
    ks = [torch.randn(L, B, Hkv, D, generator=g).to(dtype).cuda() for _ in range(steps)]
    vs = [torch.randn(L, B, Hkv, D, generator=g).to(dtype).cuda() for _ in range(steps)]
    ref = [torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda") for _ in range(steps)]
    got = [torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda") for _ in range(steps)]
    begins = list(range(0, L, span))
    for t in range(steps):
        for l0 in begins:
            lt.decode_step(plain.shape, qs[t], ks[t], vs[t], plain.tables, plain.mask, plain.seq_lens, ref[t], plain.ws,
                           layer_begin=l0, layer_count=min(span, L - l0), advance_seq_lens=(l0 == begins[-1]))
    torch.cuda.synchronize()
    for t in range(steps):
        for l0 in begins:
            lt.decode_step_layers(over.shape, qs[t], ks[t], vs[t], over.tables, over.mask, over.seq_lens, got[t], over.ws,
                                  layer_begin=l0, layer_count=min(span, L - l0), advance_seq_lens=(l0 == begins[-1]),
                                  independent_of_previous=(l0 != 0))
    torch.cuda.synchronize()
    for t in range(steps):
        assert torch.equal(got[t], ref[t]), t
    assert torch.equal(over.seq_lens, plain.seq_lens) and over.seq_lens.cpu().tolist() == [n + steps for n in lens]
    for l in range(L):
        assert torch.equal(over.k_full[l], plain.k_full[l]) and torch.equal(over.v_full[l], plain.v_full[l])
        assert torch.equal(over.k_stream[l], plain.k_stream[l]) and torch.equal(over.v_stream[l], plain.v_stream[l])
    assert lt.check(over.ws) == 0 and lt.check(plain.ws) == 0
    # the oracle on the logical history (prompt + the appended rows, all made on the host side of this test):
    # the last step's output of one full and one lazy layer, first and last batch row
    t = steps - 1
    for l in (mask.index(0), mask.index(1)):
        for b in (0, B - 1):
            n0 = lens[b]
            K = torch.cat([prompts[l][0][b, :, :n0]] + [ks[i][l, b].cpu()[:, None] for i in range(steps)], dim=1)
            V = torch.cat([prompts[l][1][b, :, :n0]] + [vs[i][l, b].cpu()[:, None] for i in range(steps)], dim=1)
            if mask[l]:
                want = O.streaming_attention(f64(qs[t][l, b]), f64(K), f64(V), S, R)
            else:
                want = O.full_attention(f64(qs[t][l, b]), f64(K), f64(V))
            mx, rel = attn_errors(f64(got[t][l, b]), want)
            assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, mx, rel)


def test_whole_stack_through_the_layered_entry_and_a_split_call():
    """One call over the whole stack is legal too (one launch, slot regions side by side); with more (layer,
    batch row) pairs than a launch's work list holds the call splits by layers and its later launches overlap
    the earlier ones.  Same bits as lt_decode_step either way."""
    for (L, B, Hq, Hkv, D, S, R, cap, dtype) in [(5, 3, 8, 2, 128, 4, 12, 700, torch.bfloat16),
                                                 (9, 600, 4, 1, 128, 2, 6, 24, torch.bfloat16)]:
        torch.manual_seed(31)
        lens = torch.randint(0, cap - 4, (B,)).tolist()
        mask = [(l % 3 == 1) * 1 for l in range(L)]
        plain, over, _ = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, dtype, lens, mask, seed=32)
        for _ in range(3):
            q = torch.randn(L, B, Hq, D).to(dtype).cuda()
            k = torch.randn(L, B, Hkv, D).to(dtype).cuda()
            v = torch.randn(L, B, Hkv, D).to(dtype).cuda()
            ref = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
            out = torch.full_like(ref, float("nan"))
            lt.decode_step(plain.shape, q, k, v, plain.tables, plain.mask, plain.seq_lens, ref, plain.ws)
            lt.decode_step_layers(over.shape, q, k, v, over.tables, over.mask, over.seq_lens, out, over.ws,
                                  layer_begin=0, layer_count=L, advance_seq_lens=True)
            assert torch.equal(out, ref) and torch.equal(over.seq_lens, plain.seq_lens)
        assert lt.check(over.ws) == 0


def test_layered_entry_refuses_a_workspace_without_per_layer_slots():
    st = Stack(8, 2, 8, 2, 128, 4, 60, 40000)
    q = torch.zeros(8, 2, 8, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(8, 2, 2, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, 2, 8, 128, device="cuda")
    need = lt.workspace_bytes_layers(st.shape, 0, 0)
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(lt.LtError) as e:
        lt.decode_step_layers(st.shape, q, k, k, st.tables, st.mask, st.seq_lens, out, small, layer_begin=0)
    assert e.value.status == 3      # LT_ERR_WORKSPACE: nothing was enqueued


def test_captured_overlapped_step_replays():
    """A step of overlapped per-layer launches captured as one CUDA graph and replayed back to back: every
    replay equals an eager whole-stack step, bit for bit (the programmatic edges between the kernel nodes are
    part of the graph; a replay's first launch waits for the replay before it)."""
    torch.manual_seed(41)
    L, B, Hq, Hkv, D, S, R, n0, steps = 6, 2, 8, 2, 128, 4, 28, 700, 12
    cap = n0 + steps + 2
    mask = [0, 1, 0, 1, 0, 0]
    eager = Stack(L, B, Hq, Hkv, D, S, R, cap)
    graph = Stack(L, B, Hq, Hkv, D, S, R, cap)
    for st in (eager, graph):
        st.set_mask(mask); st.set_seq_lens([n0, n0 - 300])
    for l in range(L):
        k0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda(); v0 = torch.randn(B, Hkv, cap, D).bfloat16().cuda()
        for st in (eager, graph):
            st.k_full[l].copy_(k0); st.v_full[l].copy_(v0)
    for st in (eager, graph):
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    _layered_ws(graph)
    sq = torch.zeros(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    sk = torch.zeros(L, B, Hkv, D, dtype=torch.bfloat16, device="cuda")
    sv = torch.zeros_like(sk)
    so = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")

    def layered_step(st):
        for l in range(L):
            lt.decode_step_layers(st.shape, sq, sk, sv, st.tables, st.mask, st.seq_lens, so, st.ws, layer_begin=l,
                                  advance_seq_lens=(l == L - 1), independent_of_previous=(l > 0))

    warm = Stack(L, B, Hq, Hkv, D, S, R, cap)                    # per-device lookups happen outside the capture
    warm.set_seq_lens([1, 1])
    _layered_ws(warm)
    layered_step(warm)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            layered_step(graph)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    refs, gots = [], []
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        ref = torch.zeros_like(so)
        lt.decode_step(eager.shape, q, k, v, eager.tables, eager.mask, eager.seq_lens, ref, eager.ws)
        sq.copy_(q); sk.copy_(k); sv.copy_(v)
        g.replay()
        refs.append(ref); gots.append(so.clone())               # stream-ordered: no host synchronisation in the loop
    torch.cuda.synchronize()
    for step in range(steps):
        assert torch.equal(gots[step], refs[step]), step
    assert torch.equal(graph.seq_lens, eager.seq_lens) and lt.check(graph.ws) == 0
    for l in range(L):
        assert torch.equal(graph.k_full[l], eager.k_full[l]) and torch.equal(graph.k_stream[l], eager.k_stream[l])


def test_overlapped_launches_with_paged_fp8_caches_and_per_prompt_masks():
    """The deployment options together (block tables, 8-bit caches, a mask row per prompt): overlapped per-layer
    launches still equal the plain-order chain bit for bit (their parity with the oracle is covered where each
    option is tested on its own)."""
    torch.manual_seed(51)
    L, B, Hq, Hkv, D, S, R, page, pps = 6, 3, 16, 2, 128, 4, 60, 128, 40
    cap, n_pages, steps = page * pps, 3 * 40 + 5, 8
    lens = [4990, 2100, 129]
    scales = torch.full((L, 2), 0.03, dtype=torch.float32, device="cuda")
    table = torch.randperm(n_pages)[: B * pps].view(B, pps).to(torch.int32).cuda().contiguous()
    mask = torch.tensor([[0, 1, 0, 0, 1, 0], [1, 0, 0, 1, 0, 0], [0, 0, 1, 1, 0, 1]], dtype=torch.uint8).cuda()
    pools = [torch.randint(0, 120, (n_pages, Hkv, page, D), dtype=torch.uint8) for _ in range(2 * L)]
    rings = [torch.randint(0, 120, (B, Hkv, S + R, D), dtype=torch.uint8) for _ in range(2 * L)]
    shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt.LT_BF16, 0.0, per_sequence_mask=1, page_size=page, pages_per_seq=pps,
                     n_pages=n_pages, block_table=table, kv_fp8=1, kv_scales=scales)
    state = []
    for layered in (False, True):
        kf = [p.clone().cuda() for p in pools[:L]]; vf = [p.clone().cuda() for p in pools[L:]]
        ks = [p.clone().cuda() for p in rings[:L]]; vs = [p.clone().cuda() for p in rings[L:]]
        tabs = lt.LayerTables(shape, kf, vf, ks, vs)
        nbytes = lt.workspace_bytes_layers(shape) if layered else lt.workspace_bytes(shape)
        ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda"); lt.workspace_init(ws)
        seq = torch.tensor(lens, dtype=torch.int32, device="cuda")
        state.append((kf, vf, ks, vs, tabs, ws, seq))
    g = torch.Generator().manual_seed(52)
    outs = ([], [])
    for t in range(steps):
        q = torch.randn(L, B, Hq, D, generator=g).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D, generator=g).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D, generator=g).bfloat16().cuda()
        for which, (kf, vf, ks, vs, tabs, ws, seq) in enumerate(state):
            out = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda")
            for l in range(L):
                if which:
                    lt.decode_step_layers(shape, q, k, v, tabs, mask, seq, out, ws, layer_begin=l,
                                          advance_seq_lens=(l == L - 1), independent_of_previous=(l > 0))
                else:
                    lt.decode_step(shape, q, k, v, tabs, mask, seq, out, ws, layer_begin=l, layer_count=1,
                                   advance_seq_lens=(l == L - 1))
            outs[which].append(out)
    torch.cuda.synchronize()
    for t in range(steps):
        assert torch.isfinite(outs[0][t]).all() and torch.equal(outs[1][t], outs[0][t]), t
    for a, b in zip(state[0][:4], state[1][:4]):
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    assert torch.equal(state[0][6], state[1][6]) and lt.check(state[0][5]) == 0 and lt.check(state[1][5]) == 0
