"""GPU parity of lt_decode_step (append + attend + advance in one launch):
bit-identical to lt_kv_append followed by lt_hybrid_decode_attn, and equal to the
oracle's replay on the logical history (O1 / O2 / O5)."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, Stack, attn_errors, bits, f64

pytestmark = pytest.mark.gpu


def _two_stacks(L, B, Hq, Hkv, D, S, R, cap, dtype, lens, mask, seed):
    """Two device stacks with identical contents: one for the separate calls, one for the fused call."""
    g = torch.Generator().manual_seed(seed)
    stacks = [Stack(L, B, Hq, Hkv, D, S, R, cap, dtype) for _ in range(2)]
    for l in range(L):
        k = torch.randn(B, Hkv, cap, D, generator=g).to(dtype)
        v = torch.randn(B, Hkv, cap, D, generator=g).to(dtype)
        for st in stacks:
            st.k_full[l].copy_(k); st.v_full[l].copy_(v)
    for st in stacks:
        st.set_mask(mask); st.set_seq_lens(lens)
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    return stacks


CASES = [
    # dtype, D, Hq, Hkv, S, R, lens, steps
    (torch.bfloat16, 128, 8, 2, 4, 28, [300, 1, 0, 31, 32, 2047], 40),      # tensor-core path; wraps; n = 0 start
    (torch.bfloat16, 128, 5, 1, 0, 16, [2040, 15], 20),                    # G=5, no sink, chunk boundary crossed
    (torch.bfloat16, 128, 32, 2, 4, 12, [130, 40, 2040], 20),              # G=16: warp pairs; the fused append stores the new row once
    (torch.bfloat16, 128, 40, 2, 4, 12, [130, 40, 2040], 20),              # G=20: four warps per tile (8, 8, 4, 0 heads); chunk boundary crossed
    (torch.bfloat16, 128, 32, 1, 4, 28, [300, 1, 0, 2047], 40),            # G=32: four warps per tile; wraps; the new row is stored once
    (torch.bfloat16, 64, 32, 1, 0, 16, [2040, 15], 20),                    # head_dim 64, G=32
    (torch.bfloat16, 128, 40, 1, 4, 12, [130, 40], 20),                    # G=40 -> CUDA-core path
    (torch.bfloat16, 64, 8, 2, 4, 28, [300, 1, 0, 31, 32, 2047], 40),      # head_dim 64 on the tensor-core path; wraps
    (torch.bfloat16, 64, 5, 1, 0, 16, [2040, 15], 20),                     # head_dim 64, G=5, chunk boundary crossed
    (torch.float32, 64, 4, 2, 4, 60, [513, 3], 70),                        # fp32, D=64
]


@pytest.mark.parametrize("dtype,D,Hq,Hkv,S,R,lens,steps", CASES)
def test_fused_step_is_bit_identical_to_append_then_attend(dtype, D, Hq, Hkv, S, R, lens, steps):
    L, B = 4, len(lens)
    mask = [0, 1, 1, 0]
    cap = max(lens) + steps + 3
    sep, fus = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, dtype, lens, mask, seed=5)
    g = torch.Generator().manual_seed(6)
    for step in range(steps):
        q = torch.randn(L, B, Hq, D, generator=g).to(dtype).cuda()
        k = torch.randn(L, B, Hkv, D, generator=g).to(dtype).cuda()
        v = torch.randn(L, B, Hkv, D, generator=g).to(dtype).cuda()
        sep.append(k, v)
        ref = sep.attend(q, torch.float32)
        out = torch.full_like(ref, float("nan"))
        lt.decode_step(fus.shape, q, k, v, fus.tables, fus.mask, fus.seq_lens, out, fus.ws)
        assert torch.equal(out, ref), step
        assert torch.equal(fus.seq_lens, sep.seq_lens)
    assert lt.check(fus.ws) == 0 and lt.check(sep.ws) == 0
    for l in range(L):
        assert torch.equal(fus.k_full[l], sep.k_full[l]) and torch.equal(fus.v_full[l], sep.v_full[l])
        assert torch.equal(fus.k_stream[l], sep.k_stream[l]) and torch.equal(fus.v_stream[l], sep.v_stream[l])


def test_fused_step_against_oracle_replay_with_ring_wraps():
    """Oracle replay on the logical history; the lazy layers' rings wrap several times."""
    torch.manual_seed(8)
    L, B, Hq, Hkv, D, S, R = 3, 2, 8, 2, 128, 3, 13
    n0, steps = 40, 45
    cap = n0 + steps
    mask = np.array([1, 0, 1], dtype=np.uint8)
    st = Stack(L, B, Hq, Hkv, D, S, R, cap)
    st.set_mask(mask)
    hk = [torch.randn(B, Hkv, n0, D).bfloat16() for _ in range(L)]
    hv = [torch.randn(B, Hkv, n0, D).bfloat16() for _ in range(L)]
    for l in range(L):
        st.k_full[l][:, :, :n0] = hk[l].cuda(); st.v_full[l][:, :, :n0] = hv[l].cuda()
    st.set_seq_lens([n0] * B)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    replays = []
    for b in range(B):
        rp = O.HybridReplay(mask, S, R)
        for l in range(L):
            rp.load_prompt(l, f64(hk[l][b]), f64(hv[l][b]))
        replays.append(rp)
    hist_bits = [[bits(hk[l][b]) for b in range(B)] for l in range(L)]         # [l][b] -> [Hkv, n, D]
    out = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    for step in range(steps):
        q = torch.randn(L, B, Hq, D).bfloat16().cuda()
        k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
        for l in range(L):
            for b in range(B):
                replays[b].append(l, f64(k[l, b]), f64(v[l, b]))
                mx, rel = attn_errors(f64(out[l, b]), replays[b].attend(l, f64(q[l, b])))
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, mx, rel)
                hist_bits[l][b] = np.concatenate([hist_bits[l][b], bits(k[l, b])[:, None]], axis=1)
    assert lt.check(st.ws) == 0 and st.seq_lens.cpu().tolist() == [n0 + steps] * B
    for l in np.nonzero(mask)[0]:
        for b in range(B):
            for h in range(Hkv):
                ek, valid = O.stream_cache_after(hist_bits[l][b][h], S, R)
                assert valid == S + R and np.array_equal(bits(st.k_stream[l][b, h]), ek)
    l = 1                                                               # the full layer kept every row
    for b in range(B):
        assert np.array_equal(bits(st.k_full[l][b]), hist_bits[l][b])


def test_per_layer_calls_advance_once():
    L, B, Hq, Hkv, D, S, R = 3, 2, 8, 2, 128, 4, 12
    lens, cap = [50, 9], 64
    sep, fus = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, torch.bfloat16, lens, [0, 1, 0], seed=9)
    q = torch.randn(L, B, Hq, D).bfloat16().cuda()
    k = torch.randn(L, B, Hkv, D).bfloat16().cuda()
    v = torch.randn(L, B, Hkv, D).bfloat16().cuda()
    sep.append(k, v)
    ref = sep.attend(q, torch.float32)
    out = torch.zeros_like(ref)
    for l in range(L):
        lt.decode_step(fus.shape, q, k, v, fus.tables, fus.mask, fus.seq_lens, out, fus.ws, layer_begin=l,
                       layer_count=1, advance_seq_lens=(l == L - 1))
        assert fus.seq_lens.cpu().tolist() == ([x + 1 for x in lens] if l == L - 1 else lens)
    assert torch.equal(out, ref)


def test_per_layer_launch_chain_without_host_syncs_matches_whole_stack_steps():
    """A model issues the step layer by layer.  Those launches carry the programmatic-serialization
    attribute: each may become resident under the tail of the one before and waits there until it has
    completed.  Twelve steps of six back-to-back per-layer launches, no host synchronisation anywhere in
    the chain (so that launches do overlap), against whole-stack steps: same bits in every output, every
    cache and seq_lens - including the step boundary, where the first launch of a step must see the
    lengths that the last launch of the previous step advanced."""
    L, B, Hq, Hkv, D, S, R = 6, 3, 8, 2, 128, 4, 60
    lens, steps = [3000, 1500, 700], 12
    cap = max(lens) + steps + 4
    whole, chain = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, torch.bfloat16, lens, [0, 1, 0, 0, 1, 0], seed=12)
    torch.manual_seed(13)
    qs = [torch.randn(L, B, Hq, D).bfloat16().cuda() for _ in range(steps)]
    ks = [torch.randn(L, B, Hkv, D).bfloat16().cuda() for _ in range(steps)]
    vs = [torch.randn(L, B, Hkv, D).bfloat16().cuda() for _ in range(steps)]
    ref = [torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda") for _ in range(steps)]
    got = [torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device="cuda") for _ in range(steps)]
    for t in range(steps):
        lt.decode_step(whole.shape, qs[t], ks[t], vs[t], whole.tables, whole.mask, whole.seq_lens, ref[t], whole.ws)
    torch.cuda.synchronize()
    for t in range(steps):
        for l in range(L):
            lt.decode_step(chain.shape, qs[t], ks[t], vs[t], chain.tables, chain.mask, chain.seq_lens, got[t], chain.ws,
                           layer_begin=l, layer_count=1, advance_seq_lens=(l == L - 1))
    torch.cuda.synchronize()
    for t in range(steps):
        assert torch.equal(got[t], ref[t]), t
    assert torch.equal(chain.seq_lens, whole.seq_lens) and chain.seq_lens.cpu().tolist() == [n + steps for n in lens]
    for l in range(L):
        assert torch.equal(chain.k_full[l], whole.k_full[l]) and torch.equal(chain.v_full[l], whole.v_full[l])
        assert torch.equal(chain.k_stream[l], whole.k_stream[l]) and torch.equal(chain.v_stream[l], whole.v_stream[l])
    assert lt.check(chain.ws) == 0
    # the attention half alone, layer by layer (no append): same chain, same bits
    out_whole = whole.attend(qs[0], torch.float32)
    out_chain = torch.full_like(out_whole, float("nan"))
    for l in range(L):
        lt.hybrid_decode_attn(chain.shape, qs[0], chain.tables, chain.mask, chain.seq_lens, out_chain, chain.ws,
                              layer_begin=l, layer_count=1)
    assert torch.equal(out_chain, out_whole)


def test_position_beyond_capacity_is_flagged_and_not_stored():
    st = Stack(2, 1, 4, 1, 128, 4, 12, 32)
    st.k_full[0].normal_(); st.v_full[0].normal_(); st.k_full[1].normal_(); st.v_full[1].normal_()
    st.set_mask([0, 1]); st.set_seq_lens([32])
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    before = st.k_full[0].clone()
    q = torch.randn(2, 1, 4, 128).bfloat16().cuda()
    k = torch.randn(2, 1, 1, 128).bfloat16().cuda()
    out = torch.zeros(2, 1, 4, 128, device="cuda")
    lt.decode_step(st.shape, q, k, k, st.tables, st.mask, st.seq_lens, out, st.ws)
    assert lt.check(st.ws, raise_on_error=False) & 1
    assert torch.equal(st.k_full[0], before) and torch.isfinite(out).all()
    # the lazy layer took its token: ring slot of position 32
    assert torch.equal(st.k_stream[1][0, 0, lt.ring_slot(32, 4, 12)], k[1, 0, 0])


def test_large_batch_is_split_into_launches_by_layers():
    """More (layer, batch row) pairs than one launch's work list holds."""
    L, B, Hq, Hkv, D, S, R, cap = 5, 600, 2, 1, 64, 2, 6, 24
    torch.manual_seed(10)
    lens = torch.randint(0, 20, (B,)).tolist()
    sep, fus = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, torch.float32, lens, [0, 1, 0, 1, 0], seed=11)
    for _ in range(3):
        q = torch.randn(L, B, Hq, D).cuda()
        k = torch.randn(L, B, Hkv, D).cuda()
        v = torch.randn(L, B, Hkv, D).cuda()
        sep.append(k, v)
        ref = sep.attend(q, torch.float32)
        out = torch.zeros_like(ref)
        lt.decode_step(fus.shape, q, k, v, fus.tables, fus.mask, fus.seq_lens, out, fus.ws)
        assert torch.equal(out, ref) and torch.equal(fus.seq_lens, sep.seq_lens)
    assert lt.check(fus.ws) == 0


def test_host_buffer_step_equals_device_step():
    """lt_decode_step_host: pinned host inputs in, host output back, same bits as the device-pointer call."""
    L, B, Hq, Hkv, D, S, R = 3, 2, 8, 2, 128, 4, 12
    lens, cap = [40, 9], 64
    dev, host = _two_stacks(L, B, Hq, Hkv, D, S, R, cap, torch.bfloat16, lens, [0, 1, 0], seed=12)
    g = torch.Generator().manual_seed(13)
    d_q = torch.empty(L, B, Hq, D, dtype=torch.bfloat16, device="cuda")
    d_k = torch.empty(L, B, Hkv, D, dtype=torch.bfloat16, device="cuda"); d_v = torch.empty_like(d_k)
    d_out = torch.empty(L, B, Hq, D, dtype=torch.float32, device="cuda")
    h_out = torch.empty(L, B, Hq, D, dtype=torch.float32).pin_memory()
    ref = torch.zeros(L, B, Hq, D, dtype=torch.float32, device="cuda")
    for step in range(5):
        q = torch.randn(L, B, Hq, D, generator=g).bfloat16().pin_memory()
        k = torch.randn(L, B, Hkv, D, generator=g).bfloat16().pin_memory()
        v = torch.randn(L, B, Hkv, D, generator=g).bfloat16().pin_memory()
        lt.decode_step(dev.shape, q.cuda(), k.cuda(), v.cuda(), dev.tables, dev.mask, dev.seq_lens, ref, dev.ws)
        lt.decode_step_host(host.shape, q, k, v, h_out, d_q, d_k, d_v, d_out, host.tables, host.mask, host.seq_lens,
                            host.ws)
        torch.cuda.synchronize()
        assert torch.equal(h_out, ref.cpu()), step
    assert torch.equal(host.seq_lens, dev.seq_lens) and lt.check(host.ws) == 0
    for l in range(L):
        assert torch.equal(host.k_full[l], dev.k_full[l]) and torch.equal(host.k_stream[l], dev.k_stream[l])
