"""GPU parity at the full sizes of the other workloads, on sampled units:
the Llama-2-7B-shaped MHA stack (G = 1), the QwQ-32B-shaped long generation
(G = 5, 16384 appended tokens, rings wrap four times) and the Llama-3.1-8B-shaped
128K stack with the lazy fraction swept over 0 / 25 / 50 / 75 %, and the
Llama-3-70B-shaped stack (80 layers, G = 8) with batch rows of different lengths
through the fused decode step."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from synth import CONFIGS, decode_inputs
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, SCORE_ABS, attn_errors, bits, build_stack, f64

pytestmark = pytest.mark.gpu


def _need_gb(gb):
    import gc
    gc.collect(); torch.cuda.empty_cache()          # earlier tests' blocks sit in torch's cache
    free, _ = torch.cuda.mem_get_info()
    if free < gb * 2**30:
        pytest.skip(f"needs ~{gb} GB of free device memory")


def _score_select(st, q_tail, cfg, n_lazy):
    s = st.shape
    scores = torch.zeros((cfg.n_layers, cfg.batch, cfg.n_q_heads), dtype=torch.float32, device="cuda")
    lt.lazy_scores(s, q_tail, st.tables, cfg.n_ctx, cfg.w_last, scores, st.ws)
    lt.select_lazy(scores, cfg.n_layers, cfg.batch, cfg.n_q_heads, n_lazy, st.mask)
    return scores


def _check_scores(st, q_tail, cfg, sc, g, n_units):
    G = cfg.group
    for _ in range(n_units):
        l, b, h = int(g.integers(cfg.n_layers)), int(g.integers(cfg.batch)), int(g.integers(cfg.n_kv_heads))
        ref = O.lazy_scores(f64(q_tail[l, b, h * G:(h + 1) * G]), f64(st.k_full[l][b, h:h + 1, :cfg.n_ctx]),
                            cfg.n_sink, cfg.n_recent)
        assert np.max(np.abs(sc[l, b, h * G:(h + 1) * G] - ref)) <= SCORE_ABS, (l, b, h)


def _check_units(st, cfg, mask, q, out, new_k, new_v, units):
    G, n0 = cfg.group, cfg.n_ctx
    for l, b, h in units:
        K = np.concatenate([f64(st.k_full[l][b, h, :n0]), np.stack([f64(x[l, b, h]) for x in new_k])])[None]
        V = np.concatenate([f64(st.v_full[l][b, h, :n0]), np.stack([f64(x[l, b, h]) for x in new_v])])[None]
        qh = f64(q[l, b, h * G:(h + 1) * G])
        ref = O.streaming_attention(qh, K, V, cfg.n_sink, cfg.n_recent) if mask[l] else O.full_attention(qh, K, V)
        mx, rel = attn_errors(f64(out[l, b, h * G:(h + 1) * G]), ref)
        assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, h, mx, rel)


def test_llama2_7b_mha_4k_sampled_units():
    _need_gb(110)
    cfg = CONFIGS["llama2_7b_4k"]
    steps = 2
    st, q_tail, planted = build_stack(cfg, steps)
    g = np.random.default_rng(31)
    sc = f64(_score_select(st, q_tail, cfg, cfg.n_lazy))
    _check_scores(st, q_tail, cfg, sc, g, 6)
    mask = st.mask.cpu().numpy()
    assert sorted(np.nonzero(mask)[0].tolist()) == planted
    assert np.array_equal(mask, O.select_lazy(sc, cfg.n_lazy)[0])
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    new_k, new_v = [], []
    for step in range(steps):
        q, k, v = decode_inputs(cfg, step, "cuda")
        st.append(k, v); new_k.append(k); new_v.append(v)
        out = st.attend(q, torch.float32)
    assert lt.check(st.ws) == 0
    lazy, full = np.nonzero(mask)[0], np.nonzero(mask == 0)[0]
    units = [(int(full[0]), 0, 0), (int(full[-1]), 31, 31), (int(lazy[0]), 0, 17), (int(lazy[-1]), 31, 5)]
    units += [(int(g.integers(32)), int(g.integers(32)), int(g.integers(32))) for _ in range(6)]
    _check_units(st, cfg, mask, q, out, new_k, new_v, units)
    # all-full mask on the same caches (the comparison the throughput ratio is quoted against)
    st.set_mask([0] * cfg.n_layers); st.set_seq_lens([cfg.n_ctx] * cfg.batch)
    out0 = st.attend(q, torch.float32)
    for l, b, h in units[:4]:
        ref = O.full_attention(f64(q[l, b, h:h + 1]), f64(st.k_full[l][b, h:h + 1, :cfg.n_ctx]),
                               f64(st.v_full[l][b, h:h + 1, :cfg.n_ctx]))
        mx, rel = attn_errors(f64(out0[l, b, h:h + 1]), ref)
        assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2


def test_qwq32b_long_generation_rings_wrap():
    """1024-token prompt, 16384 generated tokens with per-step append; the 4092-row
    rings wrap four times.  A fixed mask (the Train setting: no identification,
    the prompt is shorter than the window so every ratio is 1)."""
    _need_gb(40)
    cfg = CONFIGS["qwq32b_longgen"]
    L, B, Hkv, G, n0, steps = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.group, cfg.n_ctx, cfg.steps
    st, q_tail, _ = build_stack(cfg)
    sc = f64(_score_select(st, q_tail, cfg, cfg.n_lazy))
    assert np.max(np.abs(sc - 1.0)) <= 1e-5                     # window covers the prompt: ratio 1 everywhere
    assert st.mask.cpu().tolist() == [1] * 32 + [0] * 32        # all tie -> lower indices
    g = np.random.default_rng(41)
    mask = np.zeros(L, dtype=np.uint8); mask[g.permutation(L)[:32]] = 1
    st.set_mask(mask)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    lazy, full = np.nonzero(mask)[0], np.nonzero(mask == 0)[0]
    units = [(int(lazy[0]), 0, 0), (int(lazy[-1]), B - 1, Hkv - 1), (int(full[0]), 1, 3), (int(full[-1]), 2, 5)]
    rec_k = {u: [] for u in units}; rec_v = {u: [] for u in units}
    C = cfg.n_sink + cfg.n_recent
    check_steps = {0, C - n0 - 2, C - n0 - 1, C - n0, C - n0 + 1, 2 * C - n0, 9000, steps - 1}
    gen = torch.Generator(device="cuda").manual_seed(4242)
    dt = torch.bfloat16
    for step in range(steps):
        q = torch.randn((L, B, cfg.n_q_heads, 128), generator=gen, device="cuda", dtype=dt)
        k = torch.randn((L, B, Hkv, 128), generator=gen, device="cuda", dtype=dt)
        v = torch.randn((L, B, Hkv, 128), generator=gen, device="cuda", dtype=dt)
        st.append(k, v)
        out = st.attend(q, torch.float32, hint=n0 + step + 1)
        for (l, b, h) in units:
            rec_k[(l, b, h)].append(k[l, b, h]); rec_v[(l, b, h)].append(v[l, b, h])
        if step in check_steps:
            for (l, b, h) in units:
                K = np.concatenate([f64(st.k_full[l][b, h, :n0]), f64(torch.stack(rec_k[(l, b, h)]))])[None]
                V = np.concatenate([f64(st.v_full[l][b, h, :n0]), f64(torch.stack(rec_v[(l, b, h)]))])[None]
                qh = f64(q[l, b, h * G:(h + 1) * G])
                ref = (O.streaming_attention(qh, K, V, cfg.n_sink, cfg.n_recent) if mask[l]
                       else O.full_attention(qh, K, V))
                mx, rel = attn_errors(f64(out[l, b, h * G:(h + 1) * G]), ref)
                assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (step, l, b, h, mx, rel)
    assert lt.check(st.ws) == 0
    assert st.seq_lens.cpu().tolist() == [n0 + steps] * B
    for (l, b, h) in units:
        hist = np.concatenate([bits(st.k_full[l][b, h, :n0]), bits(torch.stack(rec_k[(l, b, h)]))])
        if mask[l]:
            ek, valid = O.stream_cache_after(hist, cfg.n_sink, cfg.n_recent)
            assert valid == C and np.array_equal(bits(st.k_stream[l][b, h]), ek)          # ring bit-exact
            hv = np.concatenate([bits(st.v_full[l][b, h, :n0]), bits(torch.stack(rec_v[(l, b, h)]))])
            assert np.array_equal(bits(st.v_stream[l][b, h]), O.stream_cache_after(hv, cfg.n_sink, cfg.n_recent)[0])
        else:
            assert np.array_equal(bits(st.k_full[l][b, h, :n0 + steps]), hist)


def test_llama31_8b_128k_lazy_fraction_sweep():
    _need_gb(60)
    cfg = CONFIGS["llama31_8b_128k"]
    L, B, Hkv = cfg.n_layers, cfg.batch, cfg.n_kv_heads
    st, q_tail, planted = build_stack(cfg, 4)
    g = np.random.default_rng(51)
    scores = _score_select(st, q_tail, cfg, cfg.n_lazy)
    sc = f64(scores)
    _check_scores(st, q_tail, cfg, sc, g, 4)
    assert sorted(np.nonzero(st.mask.cpu().numpy())[0].tolist()) == planted
    for frac_idx, n_lazy in enumerate([0, L // 4, L // 2, 3 * L // 4]):
        lt.select_lazy(scores, L, B, cfg.n_q_heads, n_lazy, st.mask)
        mask = st.mask.cpu().numpy()
        assert np.array_equal(mask, O.select_lazy(sc, n_lazy)[0]) and mask.sum() == n_lazy
        if n_lazy <= len(planted):
            assert set(np.nonzero(mask)[0]) <= set(planted)
        else:
            assert set(planted) <= set(np.nonzero(mask)[0])
        st.set_seq_lens([cfg.n_ctx] * B)
        lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
        q, k, v = decode_inputs(cfg, frac_idx, "cuda")
        st.append(k, v)
        out = st.attend(q, torch.float32)
        assert lt.check(st.ws) == 0
        units = [(int(g.integers(L)), int(g.integers(B)), int(g.integers(Hkv))) for _ in range(3)]
        if n_lazy:
            units.append((int(np.nonzero(mask)[0][0]), 1, 7))
        units.append((int(np.nonzero(mask == 0)[0][-1]), 0, 2))
        _check_units(st, cfg, mask, q, out, [k], [v], units)


def test_llama3_70b_gqa8_ragged_rows_fused_steps():
    """80 layers, 64 query / 8 kv heads: 512 query rows per scoring unit (two row
    blocks), group of 8 in the decode kernel; after identification the two batch
    rows continue from different lengths."""
    _need_gb(30)
    cfg = CONFIGS["llama3_70b_16k"]
    L, B, Hkv, G, n0 = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.group, cfg.n_ctx
    steps = 3
    st, q_tail, planted = build_stack(cfg, steps)
    g = np.random.default_rng(61)
    sc = f64(_score_select(st, q_tail, cfg, cfg.n_lazy))
    _check_scores(st, q_tail, cfg, sc, g, 4)
    mask = st.mask.cpu().numpy()
    assert sorted(np.nonzero(mask)[0].tolist()) == planted
    assert np.array_equal(mask, O.select_lazy(sc, cfg.n_lazy)[0])
    lens = [n0, 9001]                                            # row 1 is a shorter prompt
    st.set_seq_lens(lens)
    lt.stream_init(st.shape, st.mask, st.tables, st.seq_lens, ws=st.ws)
    out = torch.zeros((L, B, cfg.n_q_heads, 128), dtype=torch.float32, device="cuda")
    new_k, new_v = [], []
    for step in range(steps):
        q, k, v = decode_inputs(cfg, step, "cuda")
        new_k.append(k); new_v.append(v)
        lt.decode_step(st.shape, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
    assert lt.check(st.ws) == 0 and st.seq_lens.cpu().tolist() == [x + steps for x in lens]
    lazy, full = np.nonzero(mask)[0], np.nonzero(mask == 0)[0]
    units = [(int(full[0]), 0, 0), (int(full[-1]), 1, 7), (int(lazy[0]), 1, 1), (int(lazy[-1]), 0, 6)]
    units += [(int(g.integers(L)), int(g.integers(B)), int(g.integers(Hkv))) for _ in range(4)]
    for l, b, h in units:
        nb = lens[b]
        kb = torch.stack([x[l, b, h] for x in new_k]); vb = torch.stack([x[l, b, h] for x in new_v])
        # row 1's appended tokens overwrote prompt rows nb.. of a full layer's cache; a lazy layer's full cache still holds the prompt
        K = np.concatenate([f64(st.k_full[l][b, h, :nb]), f64(kb)])[None]
        V = np.concatenate([f64(st.v_full[l][b, h, :nb]), f64(vb)])[None]
        qh = f64(q[l, b, h * G:(h + 1) * G])
        ref = O.streaming_attention(qh, K, V, cfg.n_sink, cfg.n_recent) if mask[l] else O.full_attention(qh, K, V)
        mx, rel = attn_errors(f64(out[l, b, h * G:(h + 1) * G]), ref)
        assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, h, mx, rel)
        hist = np.concatenate([bits(st.k_full[l][b, h, :nb]), bits(kb)])
        if mask[l]:
            ek, _ = O.stream_cache_after(hist, cfg.n_sink, cfg.n_recent)
            assert np.array_equal(bits(st.k_stream[l][b, h]), ek)
        else:
            assert np.array_equal(bits(st.k_full[l][b, h, nb:nb + steps]), bits(kb))
