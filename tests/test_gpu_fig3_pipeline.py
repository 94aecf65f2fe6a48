"""Figure 3 end to end on the GPU: the layers are prefetched, scored, queued,
popped, compacted and FREED one at a time, so that no more than P + 1 full
caches exist at any moment (P = capacity of the priority queue = layers that
stay full; Section 5.1 and the caption of Figure 3).

For l = 0 .. L-1: allocate layer l's full cache and fill it with the prompt's
K/V, score layer l alone (lt_lazy_scores with a one-layer range; the table
entries of layers that are not resident are NULL), push its ratio into the
device queue, compact the popped layer at once and free its full cache.  At the
end the mask must equal the one-shot selection over all scores, the stream
caches the one-shot compaction bit for bit, and a decode step over the
surviving caches must match the oracle.
"""
import numpy as np
import pytest
import torch

import paper_2410_13846_b200 as lt
from oracle import lt_oracle as O
from synth import Config, decode_inputs, make_layer, planted_layers
from tests.gpu_util import ATTN_MAX_ABS, ATTN_REL_L2, SCORE_ABS, attn_errors, bits, f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("use_lse", [False, True])
def test_layer_by_layer_identification_keeps_at_most_p_plus_one_full_caches(use_lse):
    cfg = Config("fig3", n_layers=12, n_q_heads=8, n_kv_heads=2, head_dim=128, batch=2, n_ctx=3000, n_sink=4,
                 n_recent=252, w_last=64, n_lazy=7, dtype="bf16", steps=2)
    L, B, Hq, Hkv, D, n, T = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_ctx, cfg.w_last
    P = L - cfg.n_lazy
    S, R, C = cfg.n_sink, cfg.n_recent, cfg.n_sink + cfg.n_recent
    cap = n + cfg.steps
    dev = "cuda"
    planted = planted_layers(cfg)
    shape = lt.Shape(L, B, Hq, Hkv, D, S, R, cap, lt.LT_BF16)
    ws = torch.empty(lt.workspace_bytes(shape, n, T), dtype=torch.uint8, device=dev)
    lt.workspace_init(ws)
    k_stream = [torch.zeros((B, Hkv, C, D), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    v_stream = [torch.zeros((B, Hkv, C, D), dtype=torch.bfloat16, device=dev) for _ in range(L)]
    k_full, v_full = [None] * L, [None] * L                      # resident full caches only
    q_tail = torch.zeros((L, B, Hq, T, D), dtype=torch.bfloat16, device=dev)
    scores = torch.full((L, B, Hq), float("nan"), dtype=torch.float32, device=dev)
    lse = torch.zeros((L, B, Hq, T), dtype=torch.float32, device=dev)
    seq = torch.full((B,), n, dtype=torch.int32, device=dev)
    mask = torch.full((L,), 9, dtype=torch.uint8, device=dev)
    state = torch.zeros(L, dtype=torch.float64, device=dev)
    popped = torch.full((1,), -7, dtype=torch.int32, device=dev)
    most_resident, pops = 0, []
    ref_scores = np.zeros((L, B, Hq))
    host_k, host_v = [], []                                      # the test's own record of every layer's prompt (host memory)
    for l in range(L):
        # "prefill" of layer l: its K/V arrive, with the tail queries (and the rows' log-sum-exp for the LSE route)
        qt, K, V = make_layer(cfg, l, l in planted, dev, capacity=cap)
        q_tail[l].copy_(qt); k_full[l], v_full[l] = K, V
        host_k.append(K.cpu()); host_v.append(V.cpu())
        most_resident = max(most_resident, sum(t is not None for t in k_full))
        for b in range(B):
            ref_scores[l, b] = O.lazy_scores(f64(qt[b]), f64(K[b, :, :n]), S, R)
            if use_lse:
                lse[l, b] = torch.from_numpy(O.causal_lse(f64(qt[b]), f64(K[b, :, :n]))).float().to(dev)
        tabs = lt.LayerTables(shape, k_full, v_full, k_stream, v_stream)
        if use_lse:
            lt.lazy_scores_lse(shape, q_tail, tabs, lse, n, T, scores, ws, layer_begin=l, layer_count=1)
        else:
            lt.lazy_scores(shape, q_tail, tabs, n, T, scores, ws, layer_begin=l, layer_count=1)
        lt.select_lazy_push(scores[l], l, L, B, Hq, P, state, mask, popped)
        lt.stream_init_layer(shape, mask, popped, tabs, seq, ws=ws)
        p = popped.item()                                         # the host learns which cache it may free
        pops.append(p)
        if p >= 0:
            assert k_full[p] is not None
            k_full[p], v_full[p] = None, None                     # freed: at most P full caches remain
        assert sum(t is not None for t in k_full) <= P
        # only layer l's slice was written by this call
        assert torch.isfinite(scores[: l + 1]).all() and torch.isnan(scores[l + 1:]).all()
    assert lt.check(ws) == 0
    assert most_resident <= P + 1
    got_scores = f64(scores)
    assert np.max(np.abs(got_scores - ref_scores)) <= SCORE_ABS
    m = mask.cpu().numpy()
    # the queue leaves the same set as the one-shot selection on all scores, on the device and in the oracle
    one_shot = torch.zeros(L, dtype=torch.uint8, device=dev)
    lt.select_lazy(scores, L, B, Hq, cfg.n_lazy, one_shot)
    assert np.array_equal(m, one_shot.cpu().numpy())
    emask, epops = O.select_lazy_priority_queue_trace(O.layer_ratios(got_scores), P)
    assert np.array_equal(m, emask) and pops == list(epops)
    assert sorted(np.nonzero(m)[0].tolist()) == planted
    assert [t is None for t in k_full] == [bool(x) for x in m]   # exactly the full layers are still resident
    # stream caches: bit for bit what a one-shot compaction with the final mask gives
    for l in range(L):
        if not m[l]:
            assert not k_stream[l].any() and not v_stream[l].any()
            continue
        K, V = host_k[l], host_v[l]
        for b in range(B):
            for h in range(Hkv):
                ek, valid = O.stream_cache_after(bits(K[b, h, :n]), S, R)
                ev, _ = O.stream_cache_after(bits(V[b, h, :n]), S, R)
                assert valid == C
                assert np.array_equal(bits(k_stream[l][b, h]), ek) and np.array_equal(bits(v_stream[l][b, h]), ev)
    # a decode step over what is left: full layers read their full caches, lazy layers have none
    tabs = lt.LayerTables(shape, k_full, v_full, k_stream, v_stream)
    q, k, v = decode_inputs(cfg, 0, dev)
    out = torch.full((L, B, Hq, D), float("nan"), dtype=torch.float32, device=dev)
    lt.decode_step(shape, q, k, v, tabs, mask, seq, out, ws)
    assert lt.check(ws) == 0 and seq.cpu().tolist() == [n + 1] * B
    for l in range(L):
        K, V = host_k[l], host_v[l]
        for b in range(B):
            Kh = np.concatenate([f64(K[b, :, :n]), f64(k[l, b])[:, None]], axis=1)
            Vh = np.concatenate([f64(V[b, :, :n]), f64(v[l, b])[:, None]], axis=1)
            ref = (O.streaming_attention(f64(q[l, b]), Kh, Vh, S, R) if m[l] else O.full_attention(f64(q[l, b]), Kh, Vh))
            mx, rel = attn_errors(f64(out[l, b]), ref)
            assert mx <= ATTN_MAX_ABS and rel <= ATTN_REL_L2, (l, b, mx, rel)
