"""GPU parity end to end on the seeded workloads: scores -> select -> compaction
-> decode steps with append, replayed by the oracle on the logical history.
The toy stack is checked on every element; the Llama-3-8B-shaped 32K stack in
the launch configuration the benchmark times, on sampled units."""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from synth import CONFIGS, decode_inputs
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, SCORE_ABS, attn_errors, bits, build_stack as _build, f64

pytestmark = pytest.mark.gpu


def test_toy_stack_every_element():
    cfg = CONFIGS["toy"]
    steps = 70                                             # > n_recent: the ring wraps
    st, q_tail, planted = _build(cfg, steps)
    s = st.shape
    L, B = cfg.n_layers, cfg.batch
    # scores
    scores = torch.zeros((L, B, cfg.n_q_heads), dtype=torch.float32, device="cuda")
    lt.lazy_scores(s, q_tail, st.tables, cfg.n_ctx, cfg.w_last, scores, st.ws)
    ref_sc = np.array([[O.lazy_scores(f64(q_tail[l, b]), f64(st.k_full[l][b, :, :cfg.n_ctx]), cfg.n_sink, cfg.n_recent)
                        for b in range(B)] for l in range(L)])
    assert np.max(np.abs(f64(scores) - ref_sc)) <= SCORE_ABS
    # select: planted layer recovered, equal to the oracle fed GPU scores and fed its own scores
    lt.select_lazy(scores, L, B, cfg.n_q_heads, cfg.n_lazy, st.mask)
    mask = st.mask.cpu().numpy()
    assert mask.tolist() == [0, 1] == [int(l in planted) for l in range(L)]
    assert np.array_equal(mask, O.select_lazy(ref_sc, cfg.n_lazy)[0])
    assert np.array_equal(mask, O.select_lazy(f64(scores), cfg.n_lazy)[0])
    # compaction
    lt.stream_init(s, st.mask, st.tables, st.seq_lens, ws=st.ws)
    # oracle replay on the logical history
    rp = O.HybridReplay(mask, cfg.n_sink, cfg.n_recent)
    for l in range(L):
        rp.load_prompt(l, f64(st.k_full[l][0, :, :cfg.n_ctx]), f64(st.v_full[l][0, :, :cfg.n_ctx]))
    for step in range(steps):
        q, k, v = decode_inputs(cfg, step, "cuda")
        st.append(k, v)
        out = st.attend(q, torch.float32)
        for l in range(L):
            rp.append(l, f64(k[l, 0]), f64(v[l, 0]))
            mx, rel = attn_errors(f64(out[l, 0]), rp.attend(l, f64(q[l, 0])))
            assert mx <= 1e-4 and rel <= 1e-5, (step, l, mx, rel)          # fp32 inputs: far inside the bf16 bar
    assert st.seq_lens.item() == cfg.n_ctx + steps and lt.check(st.ws) == 0
    # ring contents of the lazy layer, bit for bit, after wrapping
    n = cfg.n_ctx + steps
    for h in range(cfg.n_kv_heads):
        hist = np.concatenate([bits(st.k_full[1][0, h, :cfg.n_ctx]),
                               np.stack([bits(decode_inputs(cfg, t, "cuda")[1][1, 0, h]) for t in range(steps)])])
        ek, valid = O.stream_cache_after(hist, cfg.n_sink, cfg.n_recent)
        assert valid == cfg.n_sink + cfg.n_recent and np.array_equal(bits(st.k_stream[1][0, h]), ek)
    # the full layer never wrote its stream cache; the lazy layer never appended to its full cache
    assert not st.k_stream[0].any() and not st.k_full[1][0, :, cfg.n_ctx:].any()


def test_llama3_8b_32k_sampled_units():
    """Full-size target configuration (about 40 GB on the device)."""
    import gc
    gc.collect(); torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2**30:
        pytest.skip("needs ~40 GB of free device memory")
    cfg = CONFIGS["llama3_8b_32k"]
    steps = 3
    st, q_tail, planted = _build(cfg, steps)
    s = st.shape
    L, B, Hkv, G, n0 = cfg.n_layers, cfg.batch, cfg.n_kv_heads, cfg.group, cfg.n_ctx
    # ---- scoring + selection --------------------------------------------------
    scores = torch.zeros((L, B, cfg.n_q_heads), dtype=torch.float32, device="cuda")
    lt.lazy_scores(s, q_tail, st.tables, n0, cfg.w_last, scores, st.ws)
    sc = f64(scores)
    assert np.isfinite(sc).all() and sc.min() >= 0 and sc.max() <= 1 + 1e-6
    # scoring units (layer, b, kv head; all G heads of each): a fixed sample that covers every kv head, the
    # first and the last batch row, and planted as well as unplanted layers (first, middle, last of each)
    unplanted = [l for l in range(L) if l not in planted]
    score_units = [(planted[0], 0, 0), (unplanted[0], B - 1, 1), (planted[-1], B - 1, 2), (unplanted[-1], 0, 3),
                   (planted[len(planted) // 2], B // 2, 4), (unplanted[len(unplanted) // 2], 1, 5),
                   (planted[1], B - 1, 6), (unplanted[1], 0, 7)]
    assert {u[2] for u in score_units} == set(range(Hkv))
    for l, b, h in score_units:
        ref = O.lazy_scores(f64(q_tail[l, b, h * G:(h + 1) * G]), f64(st.k_full[l][b, h:h + 1, :n0]), cfg.n_sink,
                            cfg.n_recent)
        assert np.max(np.abs(sc[l, b, h * G:(h + 1) * G] - ref)) <= SCORE_ABS, (l, b, h)
    lt.select_lazy(scores, L, B, cfg.n_q_heads, cfg.n_lazy, st.mask)
    mask = st.mask.cpu().numpy()
    r = O.layer_ratios(sc)
    assert sorted(np.nonzero(mask)[0].tolist()) == planted            # planted layers recovered
    assert np.array_equal(mask, O.select_lazy(sc, cfg.n_lazy)[0])
    assert r[mask == 1].min() - r[mask == 0].max() > 1e-3             # the margin is far from a tie
    # ---- compaction + decode steps ----------------------------------------------
    lt.stream_init(s, st.mask, st.tables, st.seq_lens, ws=st.ws)
    new_k, new_v = [], []
    out = torch.zeros((L, B, cfg.n_q_heads, cfg.head_dim), dtype=torch.float32, device="cuda")
    for step in range(steps):
        q, k, v = decode_inputs(cfg, step, "cuda")
        new_k.append(k); new_v.append(v)
        # the call the benchmark times: append + attend + merge + advance in one launch over the whole stack
        lt.decode_step(s, q, k, v, st.tables, st.mask, st.seq_lens, out, st.ws)
    assert lt.check(st.ws) == 0 and st.seq_lens.cpu().tolist() == [n0 + steps] * B
    assert torch.isfinite(out).all()
    n = n0 + steps
    lazy_layers, full_layers = np.nonzero(mask)[0], np.nonzero(mask == 0)[0]
    # decode units: a fixed sample with every kv head at least once and the first and last batch row of both layer kinds
    fl, lz = [int(x) for x in full_layers], [int(x) for x in lazy_layers]
    units = [(fl[0], 0, 0), (fl[-1], B - 1, Hkv - 1), (lz[0], 0, 1), (lz[-1], B - 1, Hkv - 2),
             (fl[len(fl) // 2], B // 2, 2), (lz[len(lz) // 2], 1, 3), (fl[1], B - 1, 4), (lz[1], 0, 5)]
    assert {u[2] for u in units} == set(range(Hkv))
    for l, b, h in units:
        # logical history of this unit: prompt rows (still in the full cache of every layer) + appended rows
        K = np.concatenate([f64(st.k_full[l][b, h, :n0]), np.stack([f64(x[l, b, h]) for x in new_k])])[None]
        V = np.concatenate([f64(st.v_full[l][b, h, :n0]), np.stack([f64(x[l, b, h]) for x in new_v])])[None]
        qh = f64(q[l, b, h * G:(h + 1) * G])
        ref = O.streaming_attention(qh, K, V, cfg.n_sink, cfg.n_recent) if mask[l] else O.full_attention(qh, K, V)
        mx, rel = attn_errors(f64(out[l, b, h * G:(h + 1) * G]), ref)
        assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, h, mx, rel)
        if mask[l]:                                           # ring contents bit-exact
            hist = np.concatenate([bits(st.k_full[l][b, h, :n0]), np.stack([bits(x[l, b, h]) for x in new_k])])
            ek, valid = O.stream_cache_after(hist, cfg.n_sink, cfg.n_recent)
            assert np.array_equal(bits(st.k_stream[l][b, h]), ek)
        else:
            assert np.array_equal(bits(st.k_full[l][b, h, n0:n]), np.stack([bits(x[l, b, h]) for x in new_k]))
